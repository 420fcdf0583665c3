// Decode step with a token-sharded KV cache (Appendix F, "Caching"): one new query row per sequence against
// every KV shard.  Each shard is an independent partial (Algorithm 3 with a single query row) and the K/V rows
// of the cache are read exactly once, so the kernel is bound by HBM reads of gathered 256-byte rows.
//
// One CTA = (KV shard, KV head, sequence).  A half-warp owns one gathered row at a time: 16 lanes x 16 bytes.
// The G query heads that share the KV head ("repeat_kv") are applied to each loaded row.  Partial dot products
// are combined with a transposing shuffle reduction so that each lane ends up owning one (row, head) logit and
// evaluates one exponential; probabilities are then broadcast back for the value accumulation.
#include "cascade_internal.cuh"

namespace cascade {

__device__ __forceinline__ void unpack_bf16x8(const uint4& t, float (&x)[8]) {
  const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(w[i] << 16);
    x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

template <int G>
__global__ void __launch_bounds__(128) decode_kernel(AttnParams p) {
  constexpr int D = 128;
  constexpr int U = (G >= 4) ? 16 / G : 4;  // rows per half-warp per step
  constexpr int NV = U * G;                 // logits per half-warp per step (4, 8 or 16)
  constexpr int LOG_NV = NV == 16 ? 4 : (NV == 8 ? 3 : 2);
  constexpr int SH = 4 - LOG_NV;            // lane (within the half-warp) holding logit idx is idx << SH
  constexpr int STEP = 8 * U;               // rows per CTA step
  __shared__ float s_m[8][G], s_l[8][G];
  __shared__ __align__(16) float s_acc[8][G][D];

  const PlanDev& pl = p.plan;
  const int P = pl.n_kv_shards;
  const int kk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int tid = threadIdx.x, lane = tid & 31, sub = lane & 15;
  const int hw = tid >> 4;  // half-warp 0..7
  const int32_t* kv_idx = pl.kv_idx + (size_t)map * pl.n_kv + pl.kv_off[(size_t)map * (P + 1) + kk];
  const int n_vis = pl.vis[(size_t)map * pl.n_q * P + kk];  // the single query slot
  const int64_t stat0 = (((int64_t)b * P + kk) * pl.n_q) * p.H + (int64_t)g * G;
  __nv_bfloat16* o_part = static_cast<__nv_bfloat16*>(p.o_part);
  if (n_vis == 0) {  // nothing of this shard is visible: m = -inf, l = 0, u = 0
    for (int gg = 0; gg < G; ++gg) {
      o_part[(stat0 + gg) * D + tid] = __float2bfloat16_rn(0.f);
      if (tid == 0) {
        p.m_part[stat0 + gg] = -INFINITY;
        p.l_part[stat0 + gg] = 0.f;
      }
    }
    return;
  }
  const int tok_q = pl.q_idx[(size_t)map * pl.n_q];
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(p.q) + (int64_t)b * p.qs.batch +
                            (int64_t)tok_q * p.qs.token + (int64_t)g * G * p.qs.head + sub * 8;
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(p.k) + (int64_t)b * p.ks.batch +
                            (int64_t)g * p.ks.head + sub * 8;
  const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(p.v) + (int64_t)b * p.vs.batch +
                            (int64_t)g * p.vs.head + sub * 8;

  // query chunk of every head of the group, pre-multiplied by scale * log2(e): logits live in base 2
  float qf[G][8];
  const float qscale = p.scale * 1.4426950408889634f;
#pragma unroll
  for (int gg = 0; gg < G; ++gg) {
    unpack_bf16x8(__ldg(reinterpret_cast<const uint4*>(qb + (int64_t)gg * p.qs.head)), qf[gg]);
#pragma unroll
    for (int i = 0; i < 8; ++i) qf[gg][i] *= qscale;
  }
  float acc[G][8];
#pragma unroll
  for (int gg = 0; gg < G; ++gg)
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[gg][i] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;  // statistics of the head this lane owns: my_idx % G
  const int my_idx = sub >> SH;
  const int my_u = my_idx / G;

  for (int r0 = 0; r0 < n_vis; r0 += STEP) {
    uint4 kx[U], vx[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int row = min(r0 + u * 8 + hw, n_vis - 1);  // clamped; masked below
      const int64_t tok = __ldg(kv_idx + row);
      kx[u] = __ldcs(reinterpret_cast<const uint4*>(kb + tok * p.ks.token));
      vx[u] = __ldcs(reinterpret_cast<const uint4*>(vb + tok * p.vs.token));
    }
    float val[NV];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float kf[8];
      unpack_bf16x8(kx[u], kf);
#pragma unroll
      for (int gg = 0; gg < G; ++gg) {
        float d0 = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) d0 = fmaf(qf[gg][i], kf[i], d0);
        val[u * G + gg] = d0;
      }
    }
    // transposing reduction over the 16 lanes of the half-warp: lane L ends with logit index L >> SH
    {
      int n = NV;
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) {
        if (n > 1) {
          n >>= 1;
          const bool upper = (lane & off) != 0;
#pragma unroll
          for (int i = 0; i < n; ++i) {
            const float send = upper ? val[i] : val[i + n];
            const float keep = upper ? val[i + n] : val[i];
            val[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        } else {
          val[0] += __shfl_xor_sync(0xffffffffu, val[0], off);
        }
      }
    }
    const bool mine_ok = r0 + my_u * 8 + hw < n_vis;
    const float s = mine_ok ? val[0] : -INFINITY;
    float mx = s;
#pragma unroll
    for (int off = G << SH; off < 16; off <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    const float m_new = fmaxf(m_run, mx);
    const float pr = (s == -INFINITY) ? 0.f : exp2f(s - m_new);
    const float alpha = (m_run == -INFINITY) ? 0.f : exp2f(m_run - m_new);
    l_run = l_run * alpha + pr;
    m_run = m_new;
#pragma unroll
    for (int gg = 0; gg < G; ++gg) {
      const float a = __shfl_sync(0xffffffffu, alpha, (lane & 16) | (gg << SH));
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[gg][i] *= a;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float vf[8];
      unpack_bf16x8(vx[u], vf);
#pragma unroll
      for (int gg = 0; gg < G; ++gg) {
        const float pp = __shfl_sync(0xffffffffu, pr, (lane & 16) | ((u * G + gg) << SH));
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[gg][i] = fmaf(pp, vf[i], acc[gg][i]);
      }
    }
  }
  // sum of exponentials over the rows this half-warp saw
#pragma unroll
  for (int off = G << SH; off < 16; off <<= 1) l_run += __shfl_xor_sync(0xffffffffu, l_run, off);
  if (my_idx < G && (sub & ((1 << SH) - 1)) == 0) {
    s_m[hw][my_idx] = m_run;
    s_l[hw][my_idx] = l_run;
  }
#pragma unroll
  for (int gg = 0; gg < G; ++gg) {
    *reinterpret_cast<float4*>(&s_acc[hw][gg][sub * 8]) = make_float4(acc[gg][0], acc[gg][1], acc[gg][2], acc[gg][3]);
    *reinterpret_cast<float4*>(&s_acc[hw][gg][sub * 8 + 4]) =
        make_float4(acc[gg][4], acc[gg][5], acc[gg][6], acc[gg][7]);
  }
  __syncthreads();
  // combine the 8 half-warps; thread = output column
#pragma unroll
  for (int gg = 0; gg < G; ++gg) {
    float n = -INFINITY;
#pragma unroll
    for (int x = 0; x < 8; ++x) n = fmaxf(n, s_m[x][gg]);
    float w = 0.f, o = 0.f;
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      const float f = s_m[x][gg] == -INFINITY ? 0.f : exp2f(s_m[x][gg] - n);
      w = fmaf(f, s_l[x][gg], w);
      o = fmaf(f, s_acc[x][gg][tid], o);
    }
    o_part[(stat0 + gg) * D + tid] = __float2bfloat16_rn(o / w);
    if (tid == 0) {
      p.m_part[stat0 + gg] = n * 0.6931471805599453f;  // back to natural-log units
      p.l_part[stat0 + gg] = w;
    }
  }
}

cudaError_t launch_decode(const AttnParams& p, cudaStream_t stream) {
  dim3 grid(p.plan.n_kv_shards, p.Hkv, p.batch);
  switch (p.G) {
    case 1: decode_kernel<1><<<grid, 128, 0, stream>>>(p); break;
    case 2: decode_kernel<2><<<grid, 128, 0, stream>>>(p); break;
    case 4: decode_kernel<4><<<grid, 128, 0, stream>>>(p); break;
    case 8: decode_kernel<8><<<grid, 128, 0, stream>>>(p); break;
    default: return cudaErrorInvalidValue;
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace cascade
