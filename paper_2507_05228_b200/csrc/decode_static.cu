// Decode attention for callers that cannot provide or allocate scratch memory.
//
// cascade_attn_sharded needs a caller-provided workspace for the decode step (the per-shard partials that the
// merge kernel then combines).  Some callers have none to give: an inference server whose cache manager has
// already claimed all free HBM, so a cudaMalloc at request time fails or fragments its pool; a latency-critical
// decode loop in which cudaMalloc / cudaFree would synchronise the whole device; a plug-in that is handed raw
// pointers and has no access to the host framework's allocator.  For them this file keeps the scratch in a
// file-scope device array that is part of the library image: it costs kScratchBytes of HBM on every GPU that
// loads the library, for the life of the process, and in exchange this entry point never allocates.
#include <mutex>

#include "cascade_internal.cuh"

namespace cascade {
namespace {

constexpr size_t kScratchBytes = 16u << 20;  // 16 MiB: the 64 x 16-shard x 32-head decode step needs 8.3 MiB
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_decode_scratch[kScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};  // device address of g_decode_scratch, per device ordinal

// Resolves the array's address on the current device (once per device).  Returns nullptr and sets the error
// text on failure.
void* scratch_for_current_device() {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    set_error("cascade_attn_decode_static: cudaGetDevice: %s (device %d)", cudaGetErrorString(e), dev);
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_decode_scratch);
    if (e != cudaSuccess || !ptr) {
      set_error("cascade_attn_decode_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
      return nullptr;
    }
    g_scratch_addr[dev] = ptr;
  }
  return g_scratch_addr[dev];
}

size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace
}  // namespace cascade

using namespace cascade;

extern "C" cascade_status_t cascade_attn_decode_static(const cascade_plan_t* plan, int32_t batch, int32_t n_heads,
                                                       int32_t n_kv_heads, float scale, const void* q,
                                                       cascade_strides_t q_strides, const void* k,
                                                       cascade_strides_t k_strides, const void* v,
                                                       cascade_strides_t v_strides, void* o_out,
                                                       cascade_strides_t o_strides, float* lse_out, void* stream) {
  constexpr int kHeadDim = 128;
  if (!plan || !q || !k || !v || !o_out) {
    set_error("cascade_attn_decode_static: null pointer");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!plan->dev_blob) {
    set_error("cascade_attn_decode_static: host-only plan");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (batch < 1 || n_heads < 1 || n_kv_heads < 1 || (plan->dev.n_maps != 1 && plan->dev.n_maps != batch)) {
    set_error("cascade_attn_decode_static: bad batch or head counts");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!(scale > 0.f) || scale > 3.0e38f) {
    set_error("cascade_attn_decode_static: scale must be positive and finite");
    return CASCADE_ERR_INVALID_ARG;
  }
  const int G = n_kv_heads > 0 && n_heads % n_kv_heads == 0 ? n_heads / n_kv_heads : 0;
  if (plan->dev.n_q != 1 || !(G == 1 || G == 2 || G == 4 || G == 8)) {
    set_error("cascade_attn_decode_static: needs a plan with n_q == 1 and n_heads / n_kv_heads in {1,2,4,8} "
              "(bf16, head_dim 128)");
    return CASCADE_ERR_UNSUPPORTED;
  }
  auto misaligned = [](const void* p) { return ((uintptr_t)p & 15) != 0; };
  auto bad_strides = [](const cascade_strides_t& s) { return (s.batch % 8) || (s.token % 8) || (s.head % 8); };
  if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(o_out) || bad_strides(q_strides) ||
      bad_strides(k_strides) || bad_strides(v_strides) || bad_strides(o_strides)) {
    set_error("cascade_attn_decode_static: pointers and row strides must be 16-byte aligned");
    return CASCADE_ERR_INVALID_ARG;
  }
  if ((int64_t)batch > 65535) {
    set_error("cascade_attn_decode_static: batch exceeds 65535");
    return CASCADE_ERR_UNSUPPORTED;
  }
  const size_t rows = (size_t)batch * plan->dev.n_kv_shards * n_heads;  // one query row per sequence
  const size_t o_bytes = round256(rows * kHeadDim * sizeof(__nv_bfloat16));
  const size_t stat_bytes = round256(rows * sizeof(float));
  const size_t need = o_bytes + 2 * stat_bytes;
  if (need > kScratchBytes) {
    set_error("cascade_attn_decode_static: batch %d x %d KV shards x %d heads needs %zu bytes of scratch, the "
              "built-in array holds %zu; use cascade_attn_sharded with a workspace instead",
              batch, plan->dev.n_kv_shards, n_heads, need, kScratchBytes);
    return CASCADE_ERR_WORKSPACE;
  }
  char* scratch = static_cast<char*>(scratch_for_current_device());
  if (!scratch) return CASCADE_ERR_CUDA;

  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.plan = plan->dev;
  p.q = q;
  p.k = k;
  p.v = v;
  p.qs = {q_strides.batch, q_strides.token, q_strides.head};
  p.ks = {k_strides.batch, k_strides.token, k_strides.head};
  p.vs = {v_strides.batch, v_strides.token, v_strides.head};
  p.batch = batch;
  p.H = n_heads;
  p.Hkv = n_kv_heads;
  p.G = G;
  p.d = kHeadDim;
  p.scale = scale;
  p.fused = 0;
  // Every element of the three regions below is written by the decode kernel before the merge kernel reads it,
  // so nothing left over from an earlier call can leak into this one and nothing has to be cleared.
  p.o_part = scratch;
  p.m_part = reinterpret_cast<float*>(scratch + o_bytes);
  p.l_part = reinterpret_cast<float*>(scratch + o_bytes + stat_bytes);
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = launch_decode(p, st);
  if (e != cudaSuccess) {
    set_error("cascade_attn_decode_static: decode launch: %s", cudaGetErrorString(e));
    return CASCADE_ERR_CUDA;
  }
  MergeParams mp;
  mp.o_part = p.o_part;
  mp.m_part = p.m_part;
  mp.l_part = p.l_part;
  mp.row_scatter = nullptr;
  mp.row_scatter_batch_stride = 0;
  mp.o_out = o_out;
  mp.os = {o_strides.batch, o_strides.token, o_strides.head};
  mp.lse_out = lse_out;
  mp.batch = batch;
  mp.n_parts = plan->dev.n_kv_shards;
  mp.n_rows = 1;
  mp.H = n_heads;
  mp.d = kHeadDim;
  e = launch_merge(mp, CASCADE_BF16, st);
  if (e != cudaSuccess) {
    set_error("cascade_attn_decode_static: merge launch: %s", cudaGetErrorString(e));
    return CASCADE_ERR_CUDA;
  }
  return CASCADE_OK;
}
