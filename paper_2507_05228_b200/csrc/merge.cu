// Post-pass combine (Algorithm 4 lines 1-8): a log-sum-exp weighted average of the per-shard partials.
// Bandwidth-bound: every partial is read exactly once with 16-byte loads; one thread owns 16 bytes of one
// (row, head) output vector and loops over the parts with several loads in flight.
#include "cascade_internal.cuh"

namespace cascade {

template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float (&x)[4]) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&x)[8]) {
    const uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
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

template <typename T, int D>
__global__ void __launch_bounds__(256) merge_kernel(MergeParams p) {
  constexpr int V = Vec16<T>::N;
  constexpr int TPR = D / V;       // threads per (row, head) vector
  constexpr int ITEMS = 256 / TPR; // vectors per CTA
  constexpr int CH = 4;            // parts fetched together
  const int sub = threadIdx.x % TPR;
  const int64_t item = (int64_t)blockIdx.x * ITEMS + threadIdx.x / TPR;
  const int64_t per_batch = (int64_t)p.n_rows * p.H;
  if (item >= per_batch * p.batch) return;
  const int b = (int)(item / per_batch);
  const int64_t rh = item - (int64_t)b * per_batch;  // r * H + h
  const int r = (int)(rh / p.H);
  const int h = (int)(rh - (int64_t)r * p.H);
  const int64_t part_stride = per_batch;  // statistics per part
  const float* mp = p.m_part + (int64_t)b * p.n_parts * part_stride + rh;
  const float* lp = p.l_part + (int64_t)b * p.n_parts * part_stride + rh;
  const T* up = static_cast<const T*>(p.o_part) + ((int64_t)b * p.n_parts * part_stride + rh) * D + sub * V;

  // line 3: n = max over parts of m
  float n = -INFINITY;
  for (int k = 0; k < p.n_parts; ++k) n = fmaxf(n, __ldg(mp + (int64_t)k * part_stride));

  float acc[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = 0.f;
  float w = 0.f;
  for (int k0 = 0; k0 < p.n_parts; k0 += CH) {
    float u[CH][V];
    float wt[CH];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      const int k = k0 + c;
      if (k < p.n_parts) {
        Vec16<T>::load(up + (int64_t)k * part_stride * D, u[c]);
        const float mk = __ldg(mp + (int64_t)k * part_stride);
        const float lk = __ldg(lp + (int64_t)k * part_stride);
        wt[c] = lk > 0.f ? expf(mk - n) * lk : 0.f;  // lines 5-6 weight; an empty part has l = 0
      } else {
        wt[c] = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i) u[c][i] = 0.f;
      }
    }
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      w += wt[c];
      if (wt[c] != 0.f) {
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = fmaf(wt[c], u[c][i], acc[i]);
      }
    }
  }
  const float inv = w > 0.f ? 1.f / w : 0.f;  // line 8
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] *= inv;
  const int out_row = p.row_scatter ? __ldg(p.row_scatter + (int64_t)b * p.row_scatter_batch_stride + r) : r;
  T* op = static_cast<T*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)out_row * p.os.token +
          (int64_t)h * p.os.head + sub * V;
  Vec16<T>::store(op, acc);
  if (p.lse_out && sub == 0)
    p.lse_out[((int64_t)b * p.n_rows + out_row) * p.H + h] = w > 0.f ? n + logf(w) : -INFINITY;
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
