// cascade_plan_advance on the device: the visible-prefix lengths and pair classes of a plan for a new position of
// its first query row, recomputed from the plan's own index arrays (appendix "Cost Optimizations", Caching: the
// cache grows by one row per generated token, the shard lists do not change).  No host work and no upload per call;
// used for plans with more than a few hundred (row, shard) entries, where the host pass would cost more than two launches.
#include "cascade_internal.cuh"

namespace cascade {

namespace {

// vis[map][r][k] = number of keys of shard k (positions ascending in kv_idx) at or before the position of query
// slot r.  One thread per entry, a binary search each.
__device__ __forceinline__ void advance_vis(const PlanDev& d, int32_t q_pos_offset, int32_t* vis,
                                            int64_t first, int64_t step) {
  const int P = d.n_kv_shards;
  const int64_t n = (int64_t)d.n_maps * d.n_q * P;
  for (int64_t t = first; t < n; t += step) {
    const int k = (int)(t % P);
    const int64_t mr = t / P;
    const int r = (int)(mr % d.n_q);
    const int mp = (int)(mr / d.n_q);
    const int32_t* ko = d.kv_off + (size_t)mp * (P + 1);
    const int32_t begin = ko[k], len = ko[k + 1] - begin;
    int32_t c = len;  // every key of the shard, unless the mask is causal and cuts the list
    if (d.causal) {
      const int64_t pos = (int64_t)d.q_idx[(size_t)mp * d.n_q + r] + q_pos_offset;
      if (pos < 0) {
        c = 0;
      } else if (pos < d.n_kv) {
        const int32_t* list = d.kv_idx + (size_t)mp * d.n_kv + begin;
        int lo = 0, hi = len;  // first entry greater than pos
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (list[mid] <= (int32_t)pos) lo = mid + 1;
          else hi = mid;
        }
        c = lo;
      }
    }
    vis[t] = c;
  }
}

// EMPTY / PARTIAL / FULL per (query shard, KV shard) from the prefix lengths of the shard's first and last row (rows
// ascend in position, so the first row has the shortest prefix and the last the longest).
__device__ __forceinline__ void advance_class(const PlanDev& d, const int32_t* vis, uint8_t* __restrict__ pair_class,
                                              int64_t first, int64_t step) {
  const int J = d.n_q_shards, P = d.n_kv_shards;
  const int64_t n = (int64_t)d.n_maps * J * P;
  for (int64_t t = first; t < n; t += step) {
    const int k = (int)(t % P);
    const int64_t mj = t / P;
    const int j = (int)(mj % J);
    const int mp = (int)(mj / J);
    const int32_t* qo = d.q_off + (size_t)mp * (J + 1);
    const int32_t* ko = d.kv_off + (size_t)mp * (P + 1);
    const int32_t* v = vis + (size_t)mp * d.n_q * P;
    const int len = ko[k + 1] - ko[k];
    uint8_t cls = CASCADE_PAIR_EMPTY;
    if (qo[j + 1] > qo[j] && len > 0) {
      const int lo = v[(size_t)qo[j] * P + k], hi = v[(size_t)(qo[j + 1] - 1) * P + k];
      cls = hi == 0 ? CASCADE_PAIR_EMPTY : (lo == len ? CASCADE_PAIR_FULL : CASCADE_PAIR_PARTIAL);
    }
    pair_class[t] = cls;
  }
}

__global__ void plan_advance_vis_kernel(PlanDev d, int32_t q_pos_offset, int32_t* __restrict__ vis) {
  advance_vis(d, q_pos_offset, vis, blockIdx.x * (int64_t)blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x);
}
__global__ void plan_advance_class_kernel(PlanDev d, const int32_t* __restrict__ vis, uint8_t* __restrict__ pair_class) {
  advance_class(d, vis, pair_class, blockIdx.x * (int64_t)blockDim.x + threadIdx.x, (int64_t)gridDim.x * blockDim.x);
}

}  // namespace

cudaError_t launch_plan_advance(const PlanDev& d, int32_t q_pos_offset, cudaStream_t stream) {
  const int64_t n_vis = (int64_t)d.n_maps * d.n_q * d.n_kv_shards;
  const int64_t n_cls = (int64_t)d.n_maps * d.n_q_shards * d.n_kv_shards;
  const int threads = 256;
  const int max_blocks = 8 * 1024;
  if (n_vis > 0) {
    const int blocks = (int)std::min<int64_t>((n_vis + threads - 1) / threads, max_blocks);
    plan_advance_vis_kernel<<<blocks, threads, 0, stream>>>(d, q_pos_offset, const_cast<int32_t*>(d.vis));
  }
  if (n_cls > 0) {
    const int blocks = (int)std::min<int64_t>((n_cls + threads - 1) / threads, max_blocks);
    plan_advance_class_kernel<<<blocks, threads, 0, stream>>>(d, d.vis, const_cast<uint8_t*>(d.pair_class));
  }
  count_launch(2);
  return cudaGetLastError();
}

}  // namespace cascade
