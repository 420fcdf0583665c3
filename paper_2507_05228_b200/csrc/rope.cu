// The rotary steps of the Pre-Pass algorithm (q <- rotary_pos_emb(q, p^{R_i}), k <- rotary_pos_emb(k, p^{R_i})) as a pass
// of its own, for the rows that no fused staging covers: fp32 tensors, head_dim 64, and above all the decode step,
// where one new token's q row is rotated for immediate use and its k row once, on its way into the token-sharded
// cache ("Caching" in the appendix on cost optimizations), so that cached key rows are never touched again.
// A row's angle depends on its original position only (the rows of the positional table p are sharded with the
// tokens, Section 5.1), so the rotation commutes with any sharding.
// Pairing (i, i + d/2), angles from the table written by cascade_rope_table: y_lo = x_lo cos - x_hi sin,
// y_hi = x_hi cos + x_lo sin, in fp32, rounded once to the I/O type.  Bandwidth-bound, 16-byte accesses.
#include "cascade_internal.cuh"

namespace cascade {

template <typename T>
struct RopeVec;
template <>
struct RopeVec<float> {
  static constexpr int N = 4;
  using Raw = float4;
  static __device__ __forceinline__ void unpack(const Raw& r, float (&x)[4]) { x[0] = r.x; x[1] = r.y; x[2] = r.z; x[3] = r.w; }
  static __device__ __forceinline__ Raw pack(const float (&x)[4]) { return make_float4(x[0], x[1], x[2], x[3]); }
};
template <>
struct RopeVec<__nv_bfloat16> {
  static constexpr int N = 8;
  using Raw = uint4;
  static __device__ __forceinline__ void unpack(const Raw& r, float (&x)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ Raw pack(const float (&x)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// Rotates the N pairs (lo[e], hi[e]) by the angles whose (cos, sin) start at cs.
template <typename T>
__device__ __forceinline__ void rotate_pairs(typename RopeVec<T>::Raw& lo, typename RopeVec<T>::Raw& hi,
                                             const float2* __restrict__ cs) {
  constexpr int N = RopeVec<T>::N;
  float a[N], b[N], ya[N], yb[N];
  RopeVec<T>::unpack(lo, a);
  RopeVec<T>::unpack(hi, b);
#pragma unroll
  for (int e = 0; e < N; e += 2) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(cs + e));  // (cos, sin) of pairs e and e + 1
    ya[e] = a[e] * t.x - b[e] * t.y;
    yb[e] = b[e] * t.x + a[e] * t.y;
    ya[e + 1] = a[e + 1] * t.z - b[e + 1] * t.w;
    yb[e + 1] = b[e + 1] * t.z + a[e + 1] * t.w;
  }
  lo = RopeVec<T>::pack(ya);
  hi = RopeVec<T>::pack(yb);
}

struct RopeApplyParams {
  const void* x;
  void* y;
  Strides xs, ys;
  const float2* rope;
  int32_t batch, n_rows, n_heads, half, first_position;
};

// One thread per 16-byte piece of the lower half of a (row, head) vector and its partner in the upper half.
template <typename T>
__global__ void __launch_bounds__(256) rope_apply_kernel(RopeApplyParams p) {
  constexpr int N = RopeVec<T>::N;
  const int pieces = p.half / N;  // threads per (row, head)
  const int64_t total = (int64_t)p.batch * p.n_rows * p.n_heads * pieces;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % pieces);
  int64_t rest = idx / pieces;
  const int h = (int)(rest % p.n_heads);
  rest /= p.n_heads;
  const int r = (int)(rest % p.n_rows);
  const int b = (int)(rest / p.n_rows);
  const T* src = static_cast<const T*>(p.x) + (int64_t)b * p.xs.batch + (int64_t)r * p.xs.token + (int64_t)h * p.xs.head +
                 c * N;
  T* dst = static_cast<T*>(p.y) + (int64_t)b * p.ys.batch + (int64_t)r * p.ys.token + (int64_t)h * p.ys.head + c * N;
  using Raw = typename RopeVec<T>::Raw;
  Raw lo = *reinterpret_cast<const Raw*>(src);
  Raw hi = *reinterpret_cast<const Raw*>(src + p.half);
  rotate_pairs<T>(lo, hi, p.rope + (int64_t)(p.first_position + r) * p.half + c * N);
  *reinterpret_cast<Raw*>(dst) = lo;
  *reinterpret_cast<Raw*>(dst + p.half) = hi;
}

cudaError_t launch_rope_apply(cascade_dtype_t dtype, int32_t batch, int32_t n_rows, int32_t n_heads, int32_t head_dim,
                              const void* x, Strides xs, int32_t first_position, const float2* table, void* y, Strides ys,
                              cudaStream_t stream) {
  RopeApplyParams p;
  p.x = x;
  p.y = y;
  p.xs = xs;
  p.ys = ys;
  p.rope = table;
  p.batch = batch;
  p.n_rows = n_rows;
  p.n_heads = n_heads;
  p.half = head_dim / 2;
  p.first_position = first_position;
  const int n = dtype == CASCADE_BF16 ? 8 : 4;
  const int64_t total = (int64_t)batch * n_rows * n_heads * (p.half / n);
  const unsigned grid = (unsigned)((total + 255) / 256);
  if (dtype == CASCADE_BF16) rope_apply_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(p);
  else rope_apply_kernel<float><<<grid, 256, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

// Decode-step append (bf16, head_dim 128): for every sequence, the new token's q row is rotated into q_rot, its k row
// is rotated and written at row `position` of the key cache, and its v row is copied to the value cache.
// grid = (H + 2 Hkv, batch), 8 threads per head vector.
struct AppendParams {
  const __nv_bfloat16 *q_new, *k_new, *v_new;
  __nv_bfloat16 *q_rot, *k_cache, *v_cache;
  Strides qs, kns, vns, kcs, vcs;
  const float2* rope;
  int32_t H, Hkv, position;
};

__global__ void __launch_bounds__(32) append_rope_kernel(AppendParams p) {
  constexpr int D = 128;
  const int b = blockIdx.y, which = blockIdx.x, c = threadIdx.x;
  if (c >= 8) return;
  const float2* cs = p.rope + (int64_t)p.position * (D / 2) + c * 8;
  if (which < p.H) {  // a query head
    const __nv_bfloat16* src = p.q_new + (int64_t)b * p.qs.batch + (int64_t)which * p.qs.head + c * 8;
    __nv_bfloat16* dst = p.q_rot + ((int64_t)b * p.H + which) * D + c * 8;
    uint4 lo = *reinterpret_cast<const uint4*>(src), hi = *reinterpret_cast<const uint4*>(src + 64);
    rotate_pairs<__nv_bfloat16>(lo, hi, cs);
    *reinterpret_cast<uint4*>(dst) = lo;
    *reinterpret_cast<uint4*>(dst + 64) = hi;
  } else if (which < p.H + p.Hkv) {  // a key head: rotated, then into the cache
    const int g = which - p.H;
    const __nv_bfloat16* src = p.k_new + (int64_t)b * p.kns.batch + (int64_t)g * p.kns.head + c * 8;
    __nv_bfloat16* dst = p.k_cache + (int64_t)b * p.kcs.batch + (int64_t)p.position * p.kcs.token +
                         (int64_t)g * p.kcs.head + c * 8;
    uint4 lo = *reinterpret_cast<const uint4*>(src), hi = *reinterpret_cast<const uint4*>(src + 64);
    rotate_pairs<__nv_bfloat16>(lo, hi, cs);
    *reinterpret_cast<uint4*>(dst) = lo;
    *reinterpret_cast<uint4*>(dst + 64) = hi;
  } else {  // a value head: copied
    const int g = which - p.H - p.Hkv;
    const __nv_bfloat16* src = p.v_new + (int64_t)b * p.vns.batch + (int64_t)g * p.vns.head + c * 8;
    __nv_bfloat16* dst = p.v_cache + (int64_t)b * p.vcs.batch + (int64_t)p.position * p.vcs.token +
                         (int64_t)g * p.vcs.head + c * 8;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
    *reinterpret_cast<uint4*>(dst + 64) = *reinterpret_cast<const uint4*>(src + 64);
  }
}

cudaError_t launch_append_rope(int32_t batch, int32_t H, int32_t Hkv, const void* q_new, Strides qs, const void* k_new,
                               Strides kns, const void* v_new, Strides vns, void* q_rot, void* k_cache, Strides kcs,
                               void* v_cache, Strides vcs, int32_t position, const float2* table, cudaStream_t stream) {
  AppendParams p;
  p.q_new = static_cast<const __nv_bfloat16*>(q_new);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.q_rot = static_cast<__nv_bfloat16*>(q_rot);
  p.k_cache = static_cast<__nv_bfloat16*>(k_cache);
  p.v_cache = static_cast<__nv_bfloat16*>(v_cache);
  p.qs = qs;
  p.kns = kns;
  p.vns = vns;
  p.kcs = kcs;
  p.vcs = vcs;
  p.rope = table;
  p.H = H;
  p.Hkv = Hkv;
  p.position = position;
  append_rope_kernel<<<dim3(H + 2 * Hkv, batch), 32, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cascade
