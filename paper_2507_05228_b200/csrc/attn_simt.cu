// Attention-pass on the fp32 ALUs (the Attention-Pass algorithm), used for fp32 inputs and for shapes the tensor-core kernel
// does not take.  One CTA owns a tile of up to 32 query slots of one shard and one head; KV rows of a shard are
// gathered through the plan's index list into shared memory 32 at a time; each warp owns 8 query rows, one
// lane per key for the logits and one lane per output column group for the value product.  Statistics follow
// the printed steps with the usual streaming form: running max m, running sum l, running output.
#include "cascade_internal.cuh"

namespace cascade {

template <typename T>
__device__ __forceinline__ void load_row_chunk(const T* src, float* dst);
template <>
__device__ __forceinline__ void load_row_chunk<float>(const float* src, float* dst) {
  const float4 t = __ldg(reinterpret_cast<const float4*>(src));
  dst[0] = t.x; dst[1] = t.y; dst[2] = t.z; dst[3] = t.w;
}
template <>
__device__ __forceinline__ void load_row_chunk<__nv_bfloat16>(const __nv_bfloat16* src, float* dst) {
  const uint2 t = __ldg(reinterpret_cast<const uint2*>(src));
  dst[0] = __uint_as_float(t.x << 16);
  dst[1] = __uint_as_float(t.x & 0xffff0000u);
  dst[2] = __uint_as_float(t.y << 16);
  dst[3] = __uint_as_float(t.y & 0xffff0000u);
}

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(128) attn_simt_kernel(AttnParams p) {
  constexpr int R = 32;    // query slots per CTA
  constexpr int TK = 32;   // keys per shared-memory tile
  constexpr int RPW = 8;   // query rows per warp
  constexpr int DPL = D / 32;
  constexpr int KP = D + 4;  // padded K row (floats): conflict-free float4 reads across lanes
  extern __shared__ __align__(16) float smem_f[];
  float (*sQ)[D] = reinterpret_cast<float (*)[D]>(smem_f);
  float (*sK)[KP] = reinterpret_cast<float (*)[KP]>(smem_f + R * D);
  float (*sV)[D] = reinterpret_cast<float (*)[D]>(smem_f + R * D + TK * KP);
  int* sVis = reinterpret_cast<int*>(smem_f + R * D + TK * KP + TK * D);

  const PlanDev& pl = p.plan;
  const int P = pl.n_kv_shards;
  const int n_parts = p.fused ? 1 : P;
  const int b = blockIdx.z / n_parts;
  const int part = blockIdx.z % n_parts;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int h = blockIdx.y;
  const int g = h / p.G;
  const int4 qt = pl.qtiles[0][(size_t)map * pl.n_qtiles[0] + blockIdx.x];
  const int row0 = qt.x, nrows = qt.y;
  if (nrows == 0) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* q_idx = pl.q_idx + (size_t)map * pl.n_q;
  const int32_t* kv_idx = pl.kv_idx + (size_t)map * pl.n_kv;
  const int32_t* kv_off = pl.kv_off + (size_t)map * (P + 1);
  const int32_t* vis = pl.vis + (size_t)map * pl.n_q * P;
  const T* qb = static_cast<const T*>(p.q) + (int64_t)b * p.qs.batch + (int64_t)h * p.qs.head;
  const T* kb = static_cast<const T*>(p.k) + (int64_t)b * p.ks.batch + (int64_t)g * p.ks.head;
  const T* vb = static_cast<const T*>(p.v) + (int64_t)b * p.vs.batch + (int64_t)g * p.vs.head;

  // gather the query rows of this tile
  for (int i = tid; i < R * (D / 4); i += 128) {
    const int r = i / (D / 4), c4 = (i % (D / 4)) * 4;
    if (r < nrows)
      load_row_chunk<T>(qb + CASCADE_CHECKED((int64_t)q_idx[row0 + r], pl.n_q, pl.status, 104) * p.qs.token + c4,
                        &sQ[r][c4]);
    else sQ[r][c4] = sQ[r][c4 + 1] = sQ[r][c4 + 2] = sQ[r][c4 + 3] = 0.f;
  }

  float m_run[RPW], l_run[RPW], acc[RPW][DPL];
#pragma unroll
  for (int i = 0; i < RPW; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int j = 0; j < DPL; ++j) acc[i][j] = 0.f;
  }

  const int k_begin = p.fused ? 0 : part, k_end = p.fused ? P : part + 1;
  for (int kk = k_begin; kk < k_end; ++kk) {
    __syncthreads();  // previous shard's tiles and sVis fully consumed
    if (tid < R) sVis[tid] = tid < nrows ? vis[(size_t)(row0 + tid) * P + kk] : 0;
    // rows ascend in position, so the last row of the tile has the longest visible prefix
    const int need = vis[(size_t)(row0 + nrows - 1) * P + kk];
    const int base = kv_off[kk];
    for (int t0 = 0; t0 < need; t0 += TK) {
      __syncthreads();
      for (int i = tid; i < TK * (D / 4); i += 128) {
        const int r = i / (D / 4), c4 = (i % (D / 4)) * 4;
        if (t0 + r < need) {
          const int64_t tok = CASCADE_CHECKED((int64_t)kv_idx[base + t0 + r], pl.n_kv, pl.status, 105);
          load_row_chunk<T>(kb + tok * p.ks.token + c4, &sK[r][c4]);
          load_row_chunk<T>(vb + tok * p.vs.token + c4, &sV[r][c4]);
        } else {
          sK[r][c4] = sK[r][c4 + 1] = sK[r][c4 + 2] = sK[r][c4 + 3] = 0.f;
          sV[r][c4] = sV[r][c4 + 1] = sV[r][c4 + 2] = sV[r][c4 + 3] = 0.f;
        }
      }
      __syncthreads();
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        const int r = warp * RPW + rr;
        const int my_vis = sVis[r];
        if (t0 >= my_vis) continue;  // warp-uniform: nothing of this tile is visible to the row
        // logits a = scale q k^T, lane = key
        float dot = 0.f;
#pragma unroll
        for (int c = 0; c < D; c += 4) {
          const float4 qv = *reinterpret_cast<const float4*>(&sQ[r][c]);
          const float4 kv = *reinterpret_cast<const float4*>(&sK[lane][c]);
          dot = fmaf(qv.x, kv.x, dot);
          dot = fmaf(qv.y, kv.y, dot);
          dot = fmaf(qv.z, kv.z, dot);
          dot = fmaf(qv.w, kv.w, dot);
        }
        const bool valid = t0 + lane < my_vis;
        const float s = valid ? dot * p.scale : -INFINITY;
        float mx = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_new = fmaxf(m_run[rr], mx);  // finite: key t0 is visible
        const float pexp = valid ? expf(s - m_new) : 0.f;
        float ps = pexp;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        const float alpha = expf(m_run[rr] - m_new);  // exp(-inf) = 0 on the first tile
        l_run[rr] = l_run[rr] * alpha + ps;
        m_run[rr] = m_new;
#pragma unroll
        for (int j = 0; j < DPL; ++j) acc[rr][j] *= alpha;
        for (int c = 0; c < TK; ++c) {
          const float pc = __shfl_sync(0xffffffffu, pexp, c);
#pragma unroll
          for (int j = 0; j < DPL; ++j) acc[rr][j] = fmaf(pc, sV[c][lane + 32 * j], acc[rr][j]);
        }
      }
    }
    if (!p.fused) {
      // write the pair's (u, m, l): u normalised inside the shard (the Attention-Pass algorithm)
#pragma unroll
      for (int rr = 0; rr < RPW; ++rr) {
        const int r = warp * RPW + rr;
        if (r >= nrows) continue;
        const int64_t stat = (((int64_t)b * P + kk) * pl.n_q + (row0 + r)) * p.H + h;
        const float inv = l_run[rr] > 0.f ? 1.f / l_run[rr] : 0.f;
        T* op = static_cast<T*>(p.o_part) + stat * D;
#pragma unroll
        for (int j = 0; j < DPL; ++j) op[lane + 32 * j] = from_float<T>(acc[rr][j] * inv);
        if (lane == 0) {
          p.m_part[stat] = m_run[rr];
          p.l_part[stat] = l_run[rr];
        }
      }
    }
  }
  if (p.fused) {
#pragma unroll
    for (int rr = 0; rr < RPW; ++rr) {
      const int r = warp * RPW + rr;
      if (r >= nrows) continue;
      const int tok = (int)CASCADE_CHECKED((int64_t)q_idx[row0 + r], pl.n_q, pl.status, 104);
      const float inv = l_run[rr] > 0.f ? 1.f / l_run[rr] : 0.f;
      T* op = static_cast<T*>(p.o_out) + (int64_t)b * p.os.batch + (int64_t)tok * p.os.token +
              (int64_t)h * p.os.head;
#pragma unroll
      for (int j = 0; j < DPL; ++j) op[lane + 32 * j] = from_float<T>(acc[rr][j] * inv);
      if (lane == 0 && p.lse_out)
        p.lse_out[((int64_t)b * pl.n_q + tok) * p.H + h] =
            l_run[rr] > 0.f ? m_run[rr] + logf(l_run[rr]) : -INFINITY;
    }
  }
}

template <typename T, int D>
static cudaError_t launch_one(const AttnParams& p, dim3 grid, cudaStream_t stream) {
  constexpr size_t smem = sizeof(float) * (32 * D + 32 * (D + 4) + 32 * D) + sizeof(int) * 32;
  // per function and per device; cheap enough to repeat on every launch
  cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  attn_simt_kernel<T, D><<<grid, 128, smem, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_attn_simt(const AttnParams& p, cascade_dtype_t dtype, cudaStream_t stream) {
  const int n_parts = p.fused ? 1 : p.plan.n_kv_shards;
  dim3 grid(p.plan.n_qtiles[0], p.H, p.batch * n_parts);
  if (dtype == CASCADE_BF16) {
    if (p.d == 128) return launch_one<__nv_bfloat16, 128>(p, grid, stream);
    return launch_one<__nv_bfloat16, 64>(p, grid, stream);
  }
  if (p.d == 128) return launch_one<float, 128>(p, grid, stream);
  return launch_one<float, 64>(p, grid, stream);
}

}  // namespace cascade
