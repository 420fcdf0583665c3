// Decode step with a token-sharded KV cache (Appendix F, "Caching"): one new query row per sequence against
// every KV shard.  Each shard is an independent partial (the Attention-Pass algorithm with a single query row) and the K/V rows
// of the cache are read exactly once, so the kernel must be bound by HBM reads of gathered 256-byte rows.
//
// One CTA = (KV shard, KV head, sequence); each of its 4 warps walks blocks of 16 gathered keys.  The G query
// heads that share the KV head ("repeat_kv") form the M rows of warp-level mma.m16n8k16 products, which keeps the
// instruction count per loaded byte low enough for the memory system to be the limit (plain FMA code was
// issue-bound at ~60 % of the HBM rate).  No shared-memory staging is needed because the contraction order is
// free: the k index of an MMA may be any fixed permutation of head_dim / of the keys as long as both operands
// use the same one, so every thread loads contiguous 16-byte pieces straight from global memory into fragments:
//   logits  S[head, key]   : A = Q (heads x d), B = K (keys x d);   thread (x = lane/4, j = lane%4) holds
//                            d = 32j .. 32j+31 of Q row x and of K row x of the 8-key block
//   output  O[head, d]     : A = P (heads x 16 keys, taken directly from two S accumulators), B = V; the thread
//                            holds d = 16x .. 16x+15 of V rows 2j, 2j+1, 2j+8, 2j+9 and pairs them with PRMT
#include "cascade_internal.cuh"

namespace cascade {

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Same product when rows 8-15 of A are zero: their accumulators never change, so a few shared dummy registers can
// stand in for them (saves registers; callers rotate the dummies to keep the dependency chains short).
__device__ __forceinline__ void mma_16816_top(float& c0, float& c1, float& z0, float& z1, uint32_t a0, uint32_t a2,
                                              uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c0), "+f"(c1), "+f"(z0), "+f"(z1)
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

__device__ __forceinline__ void load64(const __nv_bfloat16* p, uint32_t (&r)[16], int o) {
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint4 t = __ldcs(reinterpret_cast<const uint4*>(p) + c);
    r[o + 4 * c] = t.x; r[o + 4 * c + 1] = t.y; r[o + 4 * c + 2] = t.z; r[o + 4 * c + 3] = t.w;
  }
}

template <int G>
// Four CTAs per SM (128 registers per thread, a few spilled values): 5.78 TB/s on the decode workload against 5.59 with
// three (168 registers); five or six spill too much (3.9 / 3.6 TB/s).
__global__ void __launch_bounds__(128, 4) decode_kernel(AttnParams p) {
  constexpr int D = 128;
  constexpr int NW = 4;  // warps per CTA
  __shared__ float s_m[NW][8], s_l[NW][8];
  __shared__ float s_o[NW][G * 4][33];  // [warp][head * 4 + j][32 columns + 1 pad]: conflict-free both ways

  const PlanDev& pl = p.plan;
  const int P = pl.n_kv_shards;
  const int kk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int x = lane >> 2, j = lane & 3;
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
  const int tok_q = (int)CASCADE_CHECKED((int64_t)pl.q_idx[(size_t)map * pl.n_q], pl.n_q, pl.status, 107);
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(p.k) + (int64_t)b * p.ks.batch +
                            (int64_t)g * p.ks.head + 32 * j;
  const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(p.v) + (int64_t)b * p.vs.batch +
                            (int64_t)g * p.vs.head + 16 * x;

  // A fragments of Q: row x = head g*G + x (rows >= G are zero), this thread's 32 d-values
  uint32_t qf[16];
  if (x < G) {
    const __nv_bfloat16* qp = static_cast<const __nv_bfloat16*>(p.q) + (int64_t)b * p.qs.batch +
                              (int64_t)tok_q * p.qs.token + (int64_t)(g * G + x) * p.qs.head + 32 * j;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint4 t = __ldg(reinterpret_cast<const uint4*>(qp) + c);
      qf[4 * c] = t.x; qf[4 * c + 1] = t.y; qf[4 * c + 2] = t.z; qf[4 * c + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int c = 0; c < 16; ++c) qf[c] = 0u;
  }
  const float cs = p.scale * 1.4426950408889634f;  // logits in log2 units

  float o[16][2];
#pragma unroll
  for (int t = 0; t < 16; ++t) o[t][0] = o[t][1] = 0.f;
  float zz[4][2] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};  // accumulators of the unused rows 8-15
  float m_run = -INFINITY, l_run = 0.f;  // for head x; l is this thread's share (its 4 key columns)

  for (int k0 = warp * 16; k0 < n_vis; k0 += NW * 16) {
    const int last = n_vis - 1;
    // gathered rows: K rows x and x+8 of the block, V rows 2j, 2j+1, 2j+8, 2j+9 (clamped; masked below)
    uint32_t ka[16], kbv[16];
    load64(kb + CASCADE_CHECKED((int64_t)__ldg(kv_idx + min(k0 + x, last)), pl.n_kv, pl.status, 106) * p.ks.token, ka, 0);
    load64(kb + CASCADE_CHECKED((int64_t)__ldg(kv_idx + min(k0 + 8 + x, last)), pl.n_kv, pl.status, 106) * p.ks.token, kbv, 0);
    uint32_t vr[4][8];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      const int key = k0 + 2 * j + (rr & 1) + (rr >> 1) * 8;
      const uint4* src = reinterpret_cast<const uint4*>(vb + CASCADE_CHECKED((int64_t)__ldg(kv_idx + min(key, last)), pl.n_kv, pl.status, 106) * p.vs.token);
      const uint4 t0 = __ldcs(src), t1 = __ldcs(src + 1);
      vr[rr][0] = t0.x; vr[rr][1] = t0.y; vr[rr][2] = t0.z; vr[rr][3] = t0.w;
      vr[rr][4] = t1.x; vr[rr][5] = t1.y; vr[rr][6] = t1.z; vr[rr][7] = t1.w;
    }
    // S = Q K^T for the two 8-key blocks; 8 k-steps of 16 over the (permuted) head_dim
    float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      mma_16816(sa, qf[2 * i], 0u, qf[2 * i + 1], 0u, ka[2 * i], ka[2 * i + 1]);
      mma_16816(sb, qf[2 * i], 0u, qf[2 * i + 1], 0u, kbv[2 * i], kbv[2 * i + 1]);
    }
    // this thread: head x, keys k0 + 2j, +1 (block a) and k0 + 8 + 2j, +1 (block b)
    float t[4];
    t[0] = (k0 + 2 * j < n_vis) ? sa[0] * cs : -INFINITY;
    t[1] = (k0 + 2 * j + 1 < n_vis) ? sa[1] * cs : -INFINITY;
    t[2] = (k0 + 8 + 2 * j < n_vis) ? sb[0] * cs : -INFINITY;
    t[3] = (k0 + 9 + 2 * j < n_vis) ? sb[1] * cs : -INFINITY;
    float mx = fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3]));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m_run, mx);  // finite: key k0 is visible
    const float alpha = ex2f(m_run - m_new);  // ex2(-inf) = 0 on the first block
    const float p0 = ex2f(t[0] - m_new), p1 = ex2f(t[1] - m_new), p2 = ex2f(t[2] - m_new), p3 = ex2f(t[3] - m_new);
    l_run = l_run * alpha + (p0 + p1) + (p2 + p3);
    m_run = m_new;
    const uint32_t pa = pack2_bf16(p0, p1), pb = pack2_bf16(p2, p3);
    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
      for (int tt = 0; tt < 16; ++tt) {
        o[tt][0] *= alpha;
        o[tt][1] *= alpha;
      }
    }
    // O += P V : 16 n-tiles of 8 columns; column n of tile tt is d = 16 n + tt
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const uint32_t b0lo = __byte_perm(vr[0][e], vr[1][e], 0x5410), b1lo = __byte_perm(vr[2][e], vr[3][e], 0x5410);
      const uint32_t b0hi = __byte_perm(vr[0][e], vr[1][e], 0x7632), b1hi = __byte_perm(vr[2][e], vr[3][e], 0x7632);
      mma_16816_top(o[2 * e][0], o[2 * e][1], zz[(2 * e) & 3][0], zz[(2 * e) & 3][1], pa, pb, b0lo, b1lo);
      mma_16816_top(o[2 * e + 1][0], o[2 * e + 1][1], zz[(2 * e + 1) & 3][0], zz[(2 * e + 1) & 3][1], pa, pb, b0hi,
                    b1hi);
    }
  }
  // this thread's share of the sum of exponentials -> whole row
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if (x < G) {
    if (j == 0) {
      s_m[warp][x] = m_run;
      s_l[warp][x] = l_run;
    }
    // accumulator (tile tt, c0) is column n = 2j -> d = 32j + tt; (tile tt, c1) is n = 2j+1 -> d = 32j + 16 + tt
#pragma unroll
    for (int tt = 0; tt < 16; ++tt) {
      s_o[warp][x * 4 + j][tt] = o[tt][0];
      s_o[warp][x * 4 + j][16 + tt] = o[tt][1];
    }
  }
  __syncthreads();
  // combine the warps (each saw a disjoint quarter of the keys); thread = output column
#pragma unroll
  for (int gg = 0; gg < G; ++gg) {
    float n = -INFINITY;
#pragma unroll
    for (int w2 = 0; w2 < NW; ++w2) n = fmaxf(n, s_m[w2][gg]);
    float wsum = 0.f, acc = 0.f;
#pragma unroll
    for (int w2 = 0; w2 < NW; ++w2) {
      const float f = ex2f(s_m[w2][gg] - n);  // 0 for a warp that saw no key
      wsum = fmaf(f, s_l[w2][gg], wsum);
      acc = fmaf(f, s_o[w2][gg * 4 + (tid >> 5)][tid & 31], acc);
    }
    o_part[(stat0 + gg) * D + tid] = __float2bfloat16_rn(acc / wsum);
    if (tid == 0) {
      p.m_part[stat0 + gg] = n * 0.6931471805599453f;  // back to natural-log units
      p.l_part[stat0 + gg] = wsum;
    }
  }
}

cudaError_t launch_decode(const AttnParams& p, cudaStream_t stream) {
  dim3 grid(p.plan.n_kv_shards, p.Hkv, p.batch);
  TimedLaunch timed(stream);
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
