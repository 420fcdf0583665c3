// Internal declarations shared by the translation units of the CUDA library (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "cascade.h"

namespace cascade {

constexpr int kNumTileSizes = 4;  // query-tile heights 32, 64, 128, 256

// Device-side view of a plan.  All arrays have a leading n_maps dimension.
struct PlanDev {
  const int32_t* q_off;
  const int32_t* q_idx;
  const int32_t* q_inv;
  const int32_t* kv_off;
  const int32_t* kv_idx;
  const int32_t* kv_inv;
  const int32_t* kv_slot_shard;  // [n_kv]: the shard whose list holds this position of kv_idx
  const int32_t* vis;
  const uint8_t* pair_class;
  // Query tiles that never cross a shard boundary: {first slot, rows, shard, unused}; rows == 0 pads.
  // Ordered by decreasing work (longest visible prefix first) so late CTAs are the short ones.
  // One list per tile height: qtiles[i] holds tiles of up to (32 << i) slots.
  const int4* qtiles[kNumTileSizes];
  int32_t n_qtiles[kNumTileSizes];  // per map (padded to the maximum over maps)
  int32_t* status;      // device status word, 0 = fine
  int32_t n_maps, n_q, n_kv, n_q_shards, n_kv_shards, q_pos_offset, causal;
  int32_t max_kv_shard_len;
};

struct Strides {
  int64_t batch, token, head;
};

struct AttnParams {
  PlanDev plan;
  const void* q;
  const void* k;
  const void* v;
  Strides qs, ks, vs;
  int32_t batch, H, Hkv, G, d;
  float scale;
  int32_t fused;  // 0: one job per KV shard, write (u, m, l); 1: walk all KV shards, write o (+lse)
  void* o_part;
  float* m_part;
  float* l_part;
  void* o_out;
  Strides os;
  float* lse_out;
  // Rotary step of the pre-pass fused into the staging of Q and K rows (the Pre-Pass algorithm): rows of the positional table,
  // rope[position * 64 + i] = (cos, sin) of position * theta_i; null = rows are used as given.  A query row sits at
  // position q_pos_offset + token, a key row at its token index.
  const float2* rope;
};

// Debug build (-DCASCADE_DEBUG, libcascade_b200_debug.so): every row index that a kernel reads out of a plan array
// before it forms an address is checked against the tensor it indexes; a bad one is recorded in the plan's status word
// (codes 101..; cascade_plan_device_status then fails) and replaced by row 0, so the access itself stays in bounds.
// The release build compiles the checks away.
#ifdef CASCADE_DEBUG
__device__ __forceinline__ int64_t cascade_checked_index(int64_t i, int64_t n, int32_t* status, int code) {
  if (i >= 0 && i < n) return i;
  atomicCAS(status, 0, code);
  return 0;
}
#define CASCADE_CHECKED(i, n, status, code) cascade_checked_index((i), (n), (status), (code))
#else
#define CASCADE_CHECKED(i, n, status, code) (i)
#endif

struct MergeParams {
  const void* o_part;
  const float* m_part;
  const float* l_part;
  const int32_t* row_scatter;
  int64_t row_scatter_batch_stride;
  void* o_out;
  Strides os;
  float* lse_out;
  int32_t batch, n_parts, n_rows, H, d;
};

// Post-pass that reads every part from the buffer of the party that computed it (cascade_merge_peers).
constexpr int kMaxMergeSources = 16;
struct MergePeersParams {
  const void* o_src[kMaxMergeSources];   // source s: [batch][parts[s]][n_src_rows][H][d]
  const float* m_src[kMaxMergeSources];  //           [batch][parts[s]][n_src_rows][H]
  const float* l_src[kMaxMergeSources];
  int32_t parts[kMaxMergeSources];
  int32_t n_src, n_src_rows;
  const int32_t* row_gather;  // [n_rows]: row of the source buffers that output row r combines; null = r
  void* o_out;
  Strides os;
  float* lse_out;
  int32_t batch, n_rows, H, d;
};

}  // namespace cascade

struct cascade_plan {
  cascade::PlanDev dev;
  std::vector<int32_t> q_off, q_idx, q_inv, kv_off, kv_idx, kv_inv, kv_slot_shard, vis;
  std::vector<int32_t> kv_pos;  // position of every K/V row; empty = the row's own index
  std::vector<uint8_t> pair_class;
  std::vector<int4> qtiles[cascade::kNumTileSizes];
  void* dev_blob = nullptr;
  size_t dev_blob_bytes = 0;
  // cascade_plan_advance moves the device arrays with a kernel; the host copies of vis and pair_class are then brought
  // up to date only when something reads them (cascade_plan_get, cascade_plan_dense_mask)
  mutable bool host_vis_stale = false;
};

namespace cascade {

void set_error(const char* fmt, ...);
void count_launch(int n = 1);
// Kernel timing (cascade_kernel_timing_begin / _end): brackets a launch with events when recording is on.
void timing_mark(cudaStream_t stream, bool start);
bool timing_recording();  // true between cascade_kernel_timing_begin and _end
struct TimedLaunch {  // RAII: events around the launches issued while it lives
  cudaStream_t st;
  explicit TimedLaunch(cudaStream_t s) : st(s) { timing_mark(st, true); }
  ~TimedLaunch() { timing_mark(st, false); }
};

// Launchers; each returns a cudaError_t from the launch.
cudaError_t launch_attn_simt(const AttnParams& p, cascade_dtype_t dtype, cudaStream_t stream);
// k_sorted / v_sorted: the shard-major copies written by launch_gather_kv, [batch][kv_head][n_kv][128] bf16
cudaError_t launch_attn_tc(const AttnParams& p, const void* k_sorted, const void* v_sorted, cudaStream_t stream);
cudaError_t launch_gather_kv(const AttnParams& p, void* k_out, void* v_out, cudaStream_t stream);
cudaError_t launch_rope_table(int32_t n_positions, int32_t head_dim, double base, float2* table, cudaStream_t stream);
cudaError_t launch_rope_apply(cascade_dtype_t dtype, int32_t batch, int32_t n_rows, int32_t n_heads, int32_t head_dim,
                              const void* x, Strides xs, int32_t first_position, const float2* table, void* y, Strides ys,
                              cudaStream_t stream);
cudaError_t launch_append_rope(int32_t batch, int32_t H, int32_t Hkv, const void* q_new, Strides qs, const void* k_new,
                               Strides kns, const void* v_new, Strides vns, void* q_rot, void* k_cache, Strides kcs,
                               void* v_cache, Strides vcs, int32_t position, const float2* table, cudaStream_t stream);
cudaError_t launch_decode(const AttnParams& p, cudaStream_t stream);
// vis and pair_class of a device plan recomputed for a new q_pos_offset (plans without kv_pos)
cudaError_t launch_plan_advance(const PlanDev& d, int32_t q_pos_offset, cudaStream_t stream);
cudaError_t launch_merge(const MergeParams& p, cascade_dtype_t dtype, cudaStream_t stream);
cudaError_t launch_merge_peers(const MergePeersParams& p, cascade_dtype_t dtype, cudaStream_t stream);

}  // namespace cascade
