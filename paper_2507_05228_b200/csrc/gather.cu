// Shard gather of the key/value rows (the paper's stage-A hand-over: every AttnNode receives k^{T_k}, v^{T_k}, the
// rows of its KV shard in ascending token order, Algorithm 1 / Appendix D): copies K and V from token order into
// shard-major order [batch][kv_head][slot][head_dim], slot = position in the plan's KV_IDX list.  After this pass
// the visible prefix of a shard is a contiguous run of rows, which the attention kernel fetches with large TMA tile
// loads; an index-mapped gather straight into shared memory could not feed the tensor cores (one 512-byte request
// per ~36 cycles per SM with TMA row gathers, less with cp.async).  Bandwidth-bound: every K/V byte is read once
// and written once, 16 bytes per thread.
#include "cascade_internal.cuh"

namespace cascade {

constexpr int kGatherRowsPerCta = 64;

__global__ void __launch_bounds__(256) gather_kv_kernel(AttnParams p, __nv_bfloat16* k_out, __nv_bfloat16* v_out) {
  constexpr int D = 128;
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
    if (slot < pl.n_kv) {
      const int64_t tok = __ldg(kv_idx + slot);
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

cudaError_t launch_gather_kv(const AttnParams& p, void* k_out, void* v_out, cudaStream_t stream) {
  dim3 grid((p.plan.n_kv + kGatherRowsPerCta - 1) / kGatherRowsPerCta, p.Hkv, p.batch);
  gather_kv_kernel<<<grid, 256, 0, stream>>>(p, static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out));
  count_launch();
  return cudaGetLastError();
}

}  // namespace cascade
