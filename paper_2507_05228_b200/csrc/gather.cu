// Shard gather of the key/value rows (the paper's stage-A hand-over: every AttnNode receives k^{T_k}, v^{T_k}, the
// rows of its KV shard in ascending token order, the Single Layer Forward Pass algorithm / Appendix D): copies K and V from token order into
// shard-major order [batch][kv_head][slot][head_dim], slot = position in the plan's KV_IDX list.  After this pass
// the visible prefix of a shard is a contiguous run of rows, which the attention kernel fetches with large TMA tile
// loads; an index-mapped gather straight into shared memory could not feed the tensor cores (one 512-byte request
// per ~36 cycles per SM with TMA row gathers, less with cp.async).  Bandwidth-bound: every K/V byte is read once
// and written once, 16 bytes per thread.
// Positions of a shard's list that no query row of the plan sees (keys later than the last query position: the unwritten
// tail of a preallocated cache) are written as zeros instead of copied.  The attention kernel loads whole 16-key
// chunks and multiplies the rows past a prefix by zero weights, so what it loads there must be finite, whatever the
// caller's tensors hold at those positions.
#include "cascade_internal.cuh"

namespace cascade {

constexpr int kGatherRowsPerCta = 64;

// True if position `slot` of the shard-major order lies inside the longest visible prefix of its shard, i.e. the
// prefix seen by the query row with the largest position (the last token of the query block).
__device__ __forceinline__ bool slot_is_visible(const PlanDev& pl, int map, int slot) {
  const int P = pl.n_kv_shards;
  const int kk = (int)CASCADE_CHECKED((int64_t)__ldg(pl.kv_slot_shard + (size_t)map * pl.n_kv + slot), P, pl.status, 102);
  const int last_slot =
      (int)CASCADE_CHECKED((int64_t)__ldg(pl.q_inv + (size_t)map * pl.n_q + pl.n_q - 1), pl.n_q, pl.status, 103);
  const int longest = __ldg(pl.vis + ((size_t)map * pl.n_q + last_slot) * P + kk);
  return slot - __ldg(pl.kv_off + (size_t)map * (P + 1) + kk) < longest;
}

__global__ void __launch_bounds__(256) gather_kv_kernel(AttnParams p, __nv_bfloat16* k_out, __nv_bfloat16* v_out) {
  constexpr int D = 128;
  // The attention kernel that follows may be launched as a programmatic dependent: its CTAs may start their set-up
  // (query loads, shard tables, TMEM) now; they wait for this grid to finish before they touch the copies.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const PlanDev& pl = p.plan;
  const int g = blockIdx.y, b = blockIdx.z;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int32_t* kv_idx = pl.kv_idx + (size_t)map * pl.n_kv;
  const int chunk = threadIdx.x & 15, r0 = threadIdx.x >> 4;  // 16 rows per pass, 16 bytes per thread
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(p.k) + (int64_t)b * p.ks.batch + (int64_t)g * p.ks.head;
  const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(p.v) + (int64_t)b * p.vs.batch + (int64_t)g * p.vs.head;
  const int64_t out_base = ((int64_t)b * p.Hkv + g) * pl.n_kv;
  const int slot0 = blockIdx.x * kGatherRowsPerCta;
  uint4 kr[kGatherRowsPerCta / 16], vr[kGatherRowsPerCta / 16];
#pragma unroll
  for (int i = 0; i < kGatherRowsPerCta / 16; ++i) {
    const int slot = slot0 + 16 * i + r0;
    kr[i] = vr[i] = make_uint4(0u, 0u, 0u, 0u);
    if (slot < pl.n_kv && slot_is_visible(pl, map, slot)) {
      const int64_t tok = CASCADE_CHECKED((int64_t)__ldg(kv_idx + slot), pl.n_kv, pl.status, 101);
      kr[i] = __ldcs(reinterpret_cast<const uint4*>(kb + tok * p.ks.token + chunk * 8));
      vr[i] = __ldcs(reinterpret_cast<const uint4*>(vb + tok * p.vs.token + chunk * 8));
    }
  }
#pragma unroll
  for (int i = 0; i < kGatherRowsPerCta / 16; ++i) {
    const int slot = slot0 + 16 * i + r0;
    if (slot < pl.n_kv) {
      *reinterpret_cast<uint4*>(k_out + (out_base + slot) * D + chunk * 8) = kr[i];
      *reinterpret_cast<uint4*>(v_out + (out_base + slot) * D + chunk * 8) = vr[i];
    }
  }
}

// Turns the 8 pairs (lo[e], hi[e]) by the angles whose (cos, sin) are cs[0..7]: lo' = lo cos - hi sin,
// hi' = hi cos + lo sin, in fp32, rounded once to bf16.
__device__ __forceinline__ void rotate8(uint4& lo, uint4& hi, const float2* __restrict__ cs) {
  const float4* cs4 = reinterpret_cast<const float4*>(cs);
  __nv_bfloat162* l2 = reinterpret_cast<__nv_bfloat162*>(&lo);
  __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&hi);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float4 t = __ldg(cs4 + e);  // (cos, sin) of pairs 2e and 2e + 1
    const float2 a = __bfloat1622float2(l2[e]), b = __bfloat1622float2(h2[e]);
    l2[e] = __floats2bfloat162_rn(a.x * t.x - b.x * t.y, a.y * t.z - b.y * t.w);
    h2[e] = __floats2bfloat162_rn(b.x * t.x + a.x * t.y, b.y * t.z + a.y * t.w);
  }
}

// The same gather with the rotary step of the pre-pass (the Pre-Pass algorithm: k <- rotary_pos_emb(k, p^{R_i})) applied to the
// key rows on the way: a key row is turned by the angles of its own token index, so the rotation needs nothing but
// the row and its row of the positional table.  A thread holds both halves of 8 rotation pairs (columns 8c.. and
// 64 + 8c..), 8 threads per row; V rows are copied as they are.
__global__ void __launch_bounds__(256) gather_kv_rope_kernel(AttnParams p, __nv_bfloat16* k_out, __nv_bfloat16* v_out) {
  constexpr int D = 128;
  constexpr int kPasses = kGatherRowsPerCta / 32;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // as in gather_kv_kernel
  const PlanDev& pl = p.plan;
  const int g = blockIdx.y, b = blockIdx.z;
  const int map = pl.n_maps == 1 ? 0 : b;
  const int32_t* kv_idx = pl.kv_idx + (size_t)map * pl.n_kv;
  const int chunk = threadIdx.x & 7, r0 = threadIdx.x >> 3;  // 32 rows per pass
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(p.k) + (int64_t)b * p.ks.batch + (int64_t)g * p.ks.head;
  const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(p.v) + (int64_t)b * p.vs.batch + (int64_t)g * p.vs.head;
  const int64_t out_base = ((int64_t)b * p.Hkv + g) * pl.n_kv;
  const int slot0 = blockIdx.x * kGatherRowsPerCta;
  uint4 klo[kPasses], khi[kPasses], vlo[kPasses], vhi[kPasses];
  int tok[kPasses];
#pragma unroll
  for (int i = 0; i < kPasses; ++i) {
    const int slot = slot0 + 32 * i + r0;
    klo[i] = khi[i] = vlo[i] = vhi[i] = make_uint4(0u, 0u, 0u, 0u);
    tok[i] = -1;
    if (slot < pl.n_kv && slot_is_visible(pl, map, slot)) {
      tok[i] = (int)CASCADE_CHECKED((int64_t)__ldg(kv_idx + slot), pl.n_kv, pl.status, 101);
      const __nv_bfloat16* kr = kb + (int64_t)tok[i] * p.ks.token + chunk * 8;
      const __nv_bfloat16* vr = vb + (int64_t)tok[i] * p.vs.token + chunk * 8;
      klo[i] = __ldcs(reinterpret_cast<const uint4*>(kr));
      khi[i] = __ldcs(reinterpret_cast<const uint4*>(kr + 64));
      vlo[i] = __ldcs(reinterpret_cast<const uint4*>(vr));
      vhi[i] = __ldcs(reinterpret_cast<const uint4*>(vr + 64));
    }
  }
#pragma unroll
  for (int i = 0; i < kPasses; ++i) {
    const int slot = slot0 + 32 * i + r0;
    if (slot < pl.n_kv) {
      if (tok[i] >= 0) rotate8(klo[i], khi[i], p.rope + (int64_t)tok[i] * (D / 2) + chunk * 8);
      __nv_bfloat16* ko = k_out + (out_base + slot) * D + chunk * 8;
      __nv_bfloat16* vo = v_out + (out_base + slot) * D + chunk * 8;
      *reinterpret_cast<uint4*>(ko) = klo[i];
      *reinterpret_cast<uint4*>(ko + 64) = khi[i];
      *reinterpret_cast<uint4*>(vo) = vlo[i];
      *reinterpret_cast<uint4*>(vo + 64) = vhi[i];
    }
  }
}

cudaError_t launch_gather_kv(const AttnParams& p, void* k_out, void* v_out, cudaStream_t stream) {
  dim3 grid((p.plan.n_kv + kGatherRowsPerCta - 1) / kGatherRowsPerCta, p.Hkv, p.batch);
  if (p.rope) {
    gather_kv_rope_kernel<<<grid, 256, 0, stream>>>(p, static_cast<__nv_bfloat16*>(k_out),
                                                    static_cast<__nv_bfloat16*>(v_out));
  } else {
    gather_kv_kernel<<<grid, 256, 0, stream>>>(p, static_cast<__nv_bfloat16*>(k_out),
                                               static_cast<__nv_bfloat16*>(v_out));
  }
  count_launch();
  return cudaGetLastError();
}

// Positional table p of the rotary embedding (Section 5.1: p is set up before inference; the Pre-Pass algorithm takes its rows
// p^{R_i}): table[t * d/2 + i] = (cos, sin)(t * base^(-2 i / d)), angles formed and evaluated in fp64, stored as fp32.
__global__ void __launch_bounds__(256) rope_table_kernel(int32_t n_positions, int32_t half, double base,
                                                         float2* __restrict__ table) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n_positions * half) return;
  const int i = (int)(idx % half);
  const double t = (double)(idx / half);
  const double theta = pow(base, -(double)i / (double)half);
  double s, c;
  sincos(t * theta, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

cudaError_t launch_rope_table(int32_t n_positions, int32_t head_dim, double base, float2* table, cudaStream_t stream) {
  const int half = head_dim / 2;
  const int64_t n = (int64_t)n_positions * half;
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(n_positions, half, base, table);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cascade
