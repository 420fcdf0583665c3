// Post-pass combine (the Post-Pass algorithm): a log-sum-exp weighted average of the per-shard partials.
// Bandwidth-bound: every partial is read exactly once with 16-byte loads; one thread owns 16 bytes of one
// (row, head) output vector and loops over the parts with several loads in flight.
#include "cascade_internal.cuh"

namespace cascade {

template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  using Raw = float4;
  static __device__ __forceinline__ Raw load(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
  static __device__ __forceinline__ void fma(float (&acc)[4], const Raw& t, float w) {
    acc[0] = fmaf(w, t.x, acc[0]); acc[1] = fmaf(w, t.y, acc[1]);
    acc[2] = fmaf(w, t.z, acc[2]); acc[3] = fmaf(w, t.w, acc[3]);
  }
  static __device__ __forceinline__ void store(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  using Raw = uint4;
  static __device__ __forceinline__ Raw load(const __nv_bfloat16* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
  static __device__ __forceinline__ void fma(float (&acc)[8], const Raw& t, float w) {
    const uint32_t x[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[2 * i] = fmaf(w, __uint_as_float(x[i] << 16), acc[2 * i]);
      acc[2 * i + 1] = fmaf(w, __uint_as_float(x[i] & 0xffff0000u), acc[2 * i + 1]);
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&x)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// A group of TPR = D / (16 / sizeof(T)) lanes owns one (row, head) output vector.  The lanes share the work on the
// statistics (lane `sub` evaluates the weights of parts sub, sub + TPR, ...; weights travel by shuffle) and each lane
// streams its own 16 bytes of every partial, two loads in flight per thread at full occupancy (8 CTAs of 256 threads
// per SM at 32 registers).  Measured on the batched / long prefill partials: 8 loads in flight at 3-4 CTAs per SM
// 5.4 / 5.9 TB/s, 4 at 6 CTAs 6.0 / 6.4, 2 at 8 CTAs 6.4 / 6.7, 1 at 8 CTAs 5.8 / 6.2.
template <typename T, int D>
__global__ void __launch_bounds__(256, 8) merge_kernel(MergeParams p) {
  using VT = Vec16<T>;
  constexpr int V = VT::N;
  constexpr int TPR = D / V;
  constexpr int ITEMS = 256 / TPR;
  constexpr int CH = 2;  // partial rows in flight per thread
  const int sub = threadIdx.x % TPR;
  const int lane = threadIdx.x & 31;
  const int group_lane0 = lane - sub;
  const int64_t per_batch = (int64_t)p.n_rows * p.H;
  const int64_t total = per_batch * p.batch;
  int64_t item = (int64_t)blockIdx.x * ITEMS + threadIdx.x / TPR;
  const bool active = item < total;
  if (!active) item = total - 1;  // keep the lane in the shuffles; it stores nothing
  const int b = (int)(item / per_batch);
  const int64_t rh = item - (int64_t)b * per_batch;  // r * H + h
  const int r = (int)(rh / p.H);
  const int h = (int)(rh - (int64_t)r * p.H);
  const int P = p.n_parts;
  const int64_t part_stride = per_batch;
  const float* mp = p.m_part + (int64_t)b * P * part_stride + rh;
  const float* lp = p.l_part + (int64_t)b * P * part_stride + rh;
  const T* up = static_cast<const T*>(p.o_part) + ((int64_t)b * P * part_stride + rh) * D + sub * V;

  // n = max over parts of m
  float n = -INFINITY;
  for (int k = sub; k < P; k += TPR) n = fmaxf(n, __ldg(mp + (int64_t)k * part_stride));
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) n = fmaxf(n, __shfl_xor_sync(0xffffffffu, n, off));

  float acc[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = 0.f;
  float w = 0.f;
  for (int base = 0; base < P; base += TPR) {
    // weight exp(m_k - n) * l_k of part base + sub (an empty part has l = 0)
    float wt = 0.f;
    if (base + sub < P) {
      const float mk = __ldg(mp + (int64_t)(base + sub) * part_stride);
      const float lk = __ldg(lp + (int64_t)(base + sub) * part_stride);
      wt = lk > 0.f ? expf(mk - n) * lk : 0.f;
    }
    w += wt;
    const int cnt = min(TPR, P - base);  // warp-uniform
    for (int c0 = 0; c0 < cnt; c0 += CH) {
      typename VT::Raw u[CH];
#pragma unroll
      for (int c = 0; c < CH; ++c)
        if (c0 + c < cnt) u[c] = VT::load(up + (int64_t)(base + c0 + c) * part_stride * D);
#pragma unroll
      for (int c = 0; c < CH; ++c)
        if (c0 + c < cnt) {
          const float wc = __shfl_sync(0xffffffffu, wt, group_lane0 + c0 + c);
          VT::fma(acc, u[c], wc);
        }
    }
  }
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) w += __shfl_xor_sync(0xffffffffu, w, off);
  if (!active) return;
  const float inv = w > 0.f ? 1.f / w : 0.f;  // the final division by w
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] *= inv;
  const int out_row = p.row_scatter ? __ldg(p.row_scatter + (int64_t)b * p.row_scatter_batch_stride + r) : r;
  T* op = static_cast<T*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)out_row * p.os.token +
          (int64_t)h * p.os.head + sub * V;
  VT::store(op, acc);
  if (p.lse_out && sub == 0)
    p.lse_out[((int64_t)b * p.n_rows + out_row) * p.H + h] = w > 0.f ? n + logf(w) : -INFINITY;
}

// The same combine with the parts left where they were computed: source s (a party's partial buffers, possibly in
// another GPU's memory mapped into this process) holds parts[s] parts of every row; output row r combines row
// row_gather[r] of every source.  Stage B of the layer and the post-pass in one kernel: each 16-byte piece of a part
// crosses the link once, straight into the registers that accumulate it, with plain loads (no staging copy, no
// multicast).  Same thread mapping as merge_kernel.
template <typename T, int D>
__global__ void __launch_bounds__(256, 8) merge_peers_kernel(const __grid_constant__ MergePeersParams p) {
  using VT = Vec16<T>;
  constexpr int V = VT::N;
  constexpr int TPR = D / V;
  constexpr int ITEMS = 256 / TPR;
  constexpr int CH = 2;
  const int sub = threadIdx.x % TPR;
  const int lane = threadIdx.x & 31;
  const int group_lane0 = lane - sub;
  const int64_t per_batch = (int64_t)p.n_rows * p.H;
  const int64_t total = per_batch * p.batch;
  int64_t item = (int64_t)blockIdx.x * ITEMS + threadIdx.x / TPR;
  const bool active = item < total;
  if (!active) item = total - 1;
  const int b = (int)(item / per_batch);
  const int64_t rh = item - (int64_t)b * per_batch;
  const int r = (int)(rh / p.H);
  const int h = (int)(rh - (int64_t)r * p.H);
  const int src_row = p.row_gather ? __ldg(p.row_gather + r) : r;
  const int64_t part_stride = (int64_t)p.n_src_rows * p.H;       // elements of m / l between two parts of a source
  const int64_t row_off = (int64_t)src_row * p.H + h;

  float n = -INFINITY;
  for (int s = 0; s < p.n_src; ++s) {
    const float* mp = p.m_src[s] + (int64_t)b * p.parts[s] * part_stride + row_off;
    for (int k = sub; k < p.parts[s]; k += TPR) n = fmaxf(n, __ldg(mp + (int64_t)k * part_stride));
  }
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) n = fmaxf(n, __shfl_xor_sync(0xffffffffu, n, off));

  float acc[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = 0.f;
  float w = 0.f;
  for (int s = 0; s < p.n_src; ++s) {
    const int P = p.parts[s];
    const float* mp = p.m_src[s] + (int64_t)b * P * part_stride + row_off;
    const float* lp = p.l_src[s] + (int64_t)b * P * part_stride + row_off;
    const T* up = static_cast<const T*>(p.o_src[s]) + ((int64_t)b * P * part_stride + row_off) * D + sub * V;
    for (int base = 0; base < P; base += TPR) {
      float wt = 0.f;
      if (base + sub < P) {
        const float mk = __ldg(mp + (int64_t)(base + sub) * part_stride);
        const float lk = __ldg(lp + (int64_t)(base + sub) * part_stride);
        wt = lk > 0.f ? expf(mk - n) * lk : 0.f;
      }
      w += wt;
      const int cnt = min(TPR, P - base);  // warp-uniform
      for (int c0 = 0; c0 < cnt; c0 += CH) {
        typename VT::Raw u[CH];
#pragma unroll
        for (int c = 0; c < CH; ++c)
          if (c0 + c < cnt) u[c] = VT::load(up + (int64_t)(base + c0 + c) * part_stride * D);
#pragma unroll
        for (int c = 0; c < CH; ++c)
          if (c0 + c < cnt) {
            const float wc = __shfl_sync(0xffffffffu, wt, group_lane0 + c0 + c);
            VT::fma(acc, u[c], wc);
          }
      }
    }
  }
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) w += __shfl_xor_sync(0xffffffffu, w, off);
  if (!active) return;
  const float inv = w > 0.f ? 1.f / w : 0.f;
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] *= inv;
  T* op = static_cast<T*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)r * p.os.token + (int64_t)h * p.os.head + sub * V;
  VT::store(op, acc);
  if (p.lse_out && sub == 0) p.lse_out[((int64_t)b * p.n_rows + r) * p.H + h] = w > 0.f ? n + logf(w) : -INFINITY;
}

cudaError_t launch_merge_peers(const MergePeersParams& p, cascade_dtype_t dtype, cudaStream_t stream) {
  const int64_t items = (int64_t)p.batch * p.n_rows * p.H;
  auto go = [&](auto kern, int items_per_cta) {
    const int64_t grid = (items + items_per_cta - 1) / items_per_cta;
    kern<<<(unsigned)grid, 256, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
  };
  if (dtype == CASCADE_BF16) {
    if (p.d == 128) return go(merge_peers_kernel<__nv_bfloat16, 128>, 256 / 16);
    return go(merge_peers_kernel<__nv_bfloat16, 64>, 256 / 8);
  }
  if (p.d == 128) return go(merge_peers_kernel<float, 128>, 256 / 32);
  return go(merge_peers_kernel<float, 64>, 256 / 16);
}

cudaError_t launch_merge(const MergeParams& p, cascade_dtype_t dtype, cudaStream_t stream) {
  const int64_t items = (int64_t)p.batch * p.n_rows * p.H;
  auto go = [&](auto kern, int items_per_cta) {
    const int64_t grid = (items + items_per_cta - 1) / items_per_cta;
    kern<<<(unsigned)grid, 256, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
  };
  if (dtype == CASCADE_BF16) {
    if (p.d == 128) return go(merge_kernel<__nv_bfloat16, 128>, 256 / 16);
    return go(merge_kernel<__nv_bfloat16, 64>, 256 / 8);
  }
  if (p.d == 128) return go(merge_kernel<float, 128>, 256 / 32);
  return go(merge_kernel<float, 64>, 256 / 16);
}

}  // namespace cascade
