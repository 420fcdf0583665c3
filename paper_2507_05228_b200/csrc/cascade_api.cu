// C ABI entry points: argument checks, plan construction (host) and kernel dispatch.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <cmath>
#include <atomic>
#include <new>

#include "cascade_internal.cuh"

namespace cascade {

static thread_local char g_err[512] = "";
static std::atomic<int64_t> g_launches{0};

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- kernel timing
static bool g_timing_on = false;
constexpr int kMaxHostGroups = 128;  // head groups cascade_attn_sharded_host pipelines over
static std::vector<cudaEvent_t> g_ev_start, g_ev_stop;
static size_t g_timed = 0;  // launches bracketed since begin
constexpr size_t kMaxTimedLaunches = 8192;

bool timing_recording() { return g_timing_on; }

void timing_mark(cudaStream_t stream, bool start) {
  if (!g_timing_on) return;
  if (start) {
    if (g_timed >= kMaxTimedLaunches) return;
    if (g_ev_start.size() <= g_timed) {
      cudaEvent_t a = nullptr, b = nullptr;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
      g_ev_start.push_back(a);
      g_ev_stop.push_back(b);
    }
    cudaEventRecord(g_ev_start[g_timed], stream);
  } else {
    if (g_timed >= kMaxTimedLaunches || g_ev_start.size() <= g_timed) return;
    cudaEventRecord(g_ev_stop[g_timed], stream);
    ++g_timed;
  }
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static cascade_status_t cuda_fail(cudaError_t e, const char* what) {
  set_error("%s: %s", what, cudaGetErrorString(e));
  return CASCADE_ERR_CUDA;
}

// Query tiles of `rows_per_tile` slots that stay inside one shard, heaviest first.
static void build_qtiles(const cascade_plan& pl, int map, int rows_per_tile, std::vector<int4>& out) {
  struct Tile {
    int4 t;
    int64_t work;
  };
  std::vector<Tile> tiles;
  const int nq = pl.dev.n_q, P = pl.dev.n_kv_shards, J = pl.dev.n_q_shards;
  const int32_t* off = pl.q_off.data() + (size_t)map * (J + 1);
  const int32_t* vis = pl.vis.data() + (size_t)map * nq * P;
  for (int j = 0; j < J; ++j) {
    for (int r0 = off[j]; r0 < off[j + 1]; r0 += rows_per_tile) {
      const int n = std::min(rows_per_tile, off[j + 1] - r0);
      int64_t work = 0;
      for (int k = 0; k < P; ++k) work += vis[(size_t)(r0 + n - 1) * P + k];
      tiles.push_back({make_int4(r0, n, j, 0), work});
    }
  }
  std::stable_sort(tiles.begin(), tiles.end(), [](const Tile& a, const Tile& b) { return a.work > b.work; });
  out.clear();
  for (auto& t : tiles) out.push_back(t.t);
}

// Visible-prefix lengths vis[r][k] of one map: the number of keys of shard k (a list of K/V rows, ascending) whose
// position is <= the position of query slot r.  A K/V row sits at position kv_pos[row] (its own index if kv_pos is null).
static void fill_vis(const cascade_plan& pl, int mp, int q_pos_offset, int32_t* vis) {
  const PlanDev& d = pl.dev;
  const int n_q = d.n_q, n_kv = d.n_kv, P = d.n_kv_shards;
  const int32_t* qi = pl.q_idx.data() + (size_t)mp * n_q;
  const int32_t* ko = pl.kv_off.data() + (size_t)mp * (P + 1);
  const int32_t* ki = pl.kv_idx.data() + (size_t)mp * n_kv;
  const int32_t* kp = pl.kv_pos.empty() ? nullptr : pl.kv_pos.data() + (size_t)mp * n_kv;
  for (int k = 0; k < P; ++k) {
    const int32_t* tb = ki + ko[k];
    const int32_t* te = ki + ko[k + 1];
    for (int r = 0; r < n_q; ++r) {
      int32_t c = (int32_t)(te - tb);  // every key of the shard, unless the mask is causal and cuts the list
      if (d.causal) {
        const int64_t pos = (int64_t)qi[r] + q_pos_offset;
        if (kp) {
          c = (int32_t)(std::upper_bound(tb, te, pos, [kp](int64_t x, int32_t row) { return x < kp[row]; }) - tb);
        } else if (pos < 0) {
          c = 0;
        } else if (pos < n_kv) {
          c = (int32_t)(std::upper_bound(tb, te, (int32_t)pos) - tb);
        }
      }
      vis[(size_t)r * P + k] = c;
    }
  }
}

// EMPTY / PARTIAL / FULL per (query shard, KV shard) from the prefix lengths of the shard's first and last row
// (rows ascend in position, so the first row has the shortest prefix and the last the longest).
static void fill_pair_class(const cascade_plan& pl, int mp, const int32_t* vis, uint8_t* pc) {
  const int J = pl.dev.n_q_shards, P = pl.dev.n_kv_shards;
  const int32_t* qo = pl.q_off.data() + (size_t)mp * (J + 1);
  const int32_t* ko = pl.kv_off.data() + (size_t)mp * (P + 1);
  for (int j = 0; j < J; ++j)
    for (int k = 0; k < P; ++k) {
      const int len = ko[k + 1] - ko[k];
      uint8_t cls = CASCADE_PAIR_EMPTY;
      if (qo[j + 1] > qo[j] && len > 0) {
        const int lo = vis[(size_t)qo[j] * P + k], hi = vis[(size_t)(qo[j + 1] - 1) * P + k];
        cls = hi == 0 ? CASCADE_PAIR_EMPTY : (lo == len ? CASCADE_PAIR_FULL : CASCADE_PAIR_PARTIAL);
      }
      pc[(size_t)j * P + k] = cls;
    }
}

// Host copies of vis and pair_class for the plan's current q_pos_offset.
static void refresh_host_vis(const cascade_plan& pl, bool force) {
  if (!force && !pl.host_vis_stale) return;
  cascade_plan& w = const_cast<cascade_plan&>(pl);
  const PlanDev& d = pl.dev;
  for (int mp = 0; mp < d.n_maps; ++mp) {
    int32_t* vis = w.vis.data() + (size_t)mp * d.n_q * d.n_kv_shards;
    fill_vis(pl, mp, d.q_pos_offset, vis);
    fill_pair_class(pl, mp, vis, w.pair_class.data() + (size_t)mp * d.n_q_shards * d.n_kv_shards);
  }
  pl.host_vis_stale = false;
}

}  // namespace cascade

using namespace cascade;

extern "C" {

int32_t cascade_version(void) { return 101; }
const char* cascade_last_error(void) { return g_err; }
int64_t cascade_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

cascade_status_t cascade_kernel_timing_begin(void) {
  g_timed = 0;
  g_timing_on = true;
  return CASCADE_OK;
}

cascade_status_t cascade_kernel_timing_end(double* total_ms, int64_t* n_launches) {
  g_timing_on = false;
  cudaError_t e = cudaDeviceSynchronize();
  double sum = 0.0;
  for (size_t i = 0; i < g_timed && e == cudaSuccess; ++i) {
    float ms = 0.f;
    e = cudaEventElapsedTime(&ms, g_ev_start[i], g_ev_stop[i]);
    sum += ms;
  }
  if (total_ms) *total_ms = sum;
  if (n_launches) *n_launches = (int64_t)g_timed;
  g_timed = 0;
  if (e != cudaSuccess) return cuda_fail(e, "cascade_kernel_timing_end");
  return CASCADE_OK;
}

static cascade_status_t plan_host(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                  const int32_t* kv_shard_of, const int32_t* kv_pos, int32_t n_q_shards,
                                  int32_t n_kv_shards, int32_t q_pos_offset, int32_t causal,
                                  cascade_plan_t** out_plan) {
  if (!out_plan || !q_shard_of || !kv_shard_of) {
    set_error("cascade_shard_plan: null pointer");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (n_maps < 1 || n_q < 1 || n_kv < 1 || n_q_shards < 1 || n_kv_shards < 1) {
    set_error("cascade_shard_plan: sizes must be positive (n_maps=%d n_q=%d n_kv=%d shards=%d/%d)", n_maps,
              n_q, n_kv, n_q_shards, n_kv_shards);
    return CASCADE_ERR_INVALID_ARG;
  }
  for (int64_t i = 0; i < (int64_t)n_maps * n_q; ++i)
    if (q_shard_of[i] < 0 || q_shard_of[i] >= n_q_shards) {
      set_error("cascade_shard_plan: q_shard_of[%lld] = %d outside [0,%d)", (long long)i, q_shard_of[i],
                n_q_shards);
      return CASCADE_ERR_BAD_MAP;
    }
  for (int64_t i = 0; i < (int64_t)n_maps * n_kv; ++i)
    if (kv_shard_of[i] < 0 || kv_shard_of[i] >= n_kv_shards) {
      set_error("cascade_shard_plan: kv_shard_of[%lld] = %d outside [0,%d)", (long long)i, kv_shard_of[i],
                n_kv_shards);
      return CASCADE_ERR_BAD_MAP;
    }
  if (kv_pos)
    for (int mp = 0; mp < n_maps; ++mp)
      for (int y = 0; y < n_kv; ++y) {
        const int32_t* kp = kv_pos + (size_t)mp * n_kv;
        if (kp[y] < 0 || (y > 0 && kp[y] <= kp[y - 1])) {
          set_error("cascade_shard_plan: kv_pos must be non-negative and strictly ascending (map %d, row %d)", mp, y);
          return CASCADE_ERR_BAD_MAP;
        }
      }
  cascade_plan* pl = new (std::nothrow) cascade_plan();
  if (!pl) {
    set_error("cascade_shard_plan: host allocation failed");
    return CASCADE_ERR_ALLOC;
  }
  try {
    const int J = n_q_shards, P = n_kv_shards;
    memset(&pl->dev, 0, sizeof(pl->dev));
    pl->dev.n_maps = n_maps;
    pl->dev.n_q = n_q;
    pl->dev.n_kv = n_kv;
    pl->dev.n_q_shards = J;
    pl->dev.n_kv_shards = P;
    pl->dev.q_pos_offset = q_pos_offset;
    pl->dev.causal = causal ? 1 : 0;
    pl->q_off.assign((size_t)n_maps * (J + 1), 0);
    pl->kv_off.assign((size_t)n_maps * (P + 1), 0);
    pl->q_idx.assign((size_t)n_maps * n_q, 0);
    pl->q_inv.assign((size_t)n_maps * n_q, 0);
    pl->kv_idx.assign((size_t)n_maps * n_kv, 0);
    pl->kv_inv.assign((size_t)n_maps * n_kv, 0);
    pl->kv_slot_shard.assign((size_t)n_maps * n_kv, 0);
    pl->vis.assign((size_t)n_maps * n_q * P, 0);
    pl->pair_class.assign((size_t)n_maps * J * P, 0);
    if (kv_pos) pl->kv_pos.assign(kv_pos, kv_pos + (size_t)n_maps * n_kv);
    int max_len = 0;
    // counting sort of token ids by shard id: ascending ids inside every shard
    auto sort_by_shard = [](const int32_t* shard_of, int n, int S, int32_t* off, int32_t* idx, int32_t* inv) {
      std::vector<int32_t> cursor(S + 1, 0);
      for (int t = 0; t < n; ++t) cursor[shard_of[t] + 1]++;
      for (int s = 0; s < S; ++s) cursor[s + 1] += cursor[s];
      for (int s = 0; s <= S; ++s) off[s] = cursor[s];
      for (int t = 0; t < n; ++t) {
        const int slot = cursor[shard_of[t]]++;
        idx[slot] = t;
        inv[t] = slot;
      }
    };
    for (int mp = 0; mp < n_maps; ++mp) {
      int32_t* qo = pl->q_off.data() + (size_t)mp * (J + 1);
      int32_t* ko = pl->kv_off.data() + (size_t)mp * (P + 1);
      int32_t* qi = pl->q_idx.data() + (size_t)mp * n_q;
      int32_t* ki = pl->kv_idx.data() + (size_t)mp * n_kv;
      sort_by_shard(q_shard_of + (size_t)mp * n_q, n_q, J, qo, qi, pl->q_inv.data() + (size_t)mp * n_q);
      sort_by_shard(kv_shard_of + (size_t)mp * n_kv, n_kv, P, ko, ki, pl->kv_inv.data() + (size_t)mp * n_kv);
      int32_t* slot_shard = pl->kv_slot_shard.data() + (size_t)mp * n_kv;
      for (int k = 0; k < P; ++k) {
        max_len = std::max(max_len, (int)(ko[k + 1] - ko[k]));
        std::fill(slot_shard + ko[k], slot_shard + ko[k + 1], k);
      }
      int32_t* vis = pl->vis.data() + (size_t)mp * n_q * P;
      fill_vis(*pl, mp, q_pos_offset, vis);
      fill_pair_class(*pl, mp, vis, pl->pair_class.data() + (size_t)mp * J * P);
    }
    pl->dev.max_kv_shard_len = max_len;
    // tile lists, padded to the same length for every map
    for (int ts = 0; ts < kNumTileSizes; ++ts) {
      std::vector<std::vector<int4>> lists(n_maps);
      size_t n_max = 0;
      for (int mp = 0; mp < n_maps; ++mp) {
        build_qtiles(*pl, mp, 32 << ts, lists[mp]);
        n_max = std::max(n_max, lists[mp].size());
      }
      pl->qtiles[ts].assign(n_max * n_maps, make_int4(0, 0, 0, 0));
      for (int mp = 0; mp < n_maps; ++mp)
        std::copy(lists[mp].begin(), lists[mp].end(), pl->qtiles[ts].begin() + mp * n_max);
      pl->dev.n_qtiles[ts] = (int32_t)n_max;
    }
  } catch (const std::bad_alloc&) {
    delete pl;
    set_error("cascade_shard_plan: host allocation failed");
    return CASCADE_ERR_ALLOC;
  }
  *out_plan = pl;
  return CASCADE_OK;
}

cascade_status_t cascade_shard_plan_host(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                         const int32_t* kv_shard_of, int32_t n_q_shards, int32_t n_kv_shards,
                                         int32_t q_pos_offset, int32_t causal, cascade_plan_t** out_plan) {
  return plan_host(n_maps, n_q, n_kv, q_shard_of, kv_shard_of, nullptr, n_q_shards, n_kv_shards, q_pos_offset, causal,
                   out_plan);
}

cascade_status_t cascade_shard_plan_resident_host(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                                  const int32_t* kv_shard_of, const int32_t* kv_pos,
                                                  int32_t n_q_shards, int32_t n_kv_shards, int32_t q_pos_offset,
                                                  int32_t causal, cascade_plan_t** out_plan) {
  if (!kv_pos) {
    set_error("cascade_shard_plan_resident_host: null kv_pos");
    return CASCADE_ERR_INVALID_ARG;
  }
  return plan_host(n_maps, n_q, n_kv, q_shard_of, kv_shard_of, kv_pos, n_q_shards, n_kv_shards, q_pos_offset, causal,
                   out_plan);
}

static cascade_status_t plan_device(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                    const int32_t* kv_shard_of, const int32_t* kv_pos, int32_t n_q_shards,
                                    int32_t n_kv_shards, int32_t q_pos_offset, int32_t causal, void* stream,
                                    cascade_plan_t** out_plan) {
  cascade_plan* pl = nullptr;
  cascade_status_t hs = plan_host(n_maps, n_q, n_kv, q_shard_of, kv_shard_of, kv_pos, n_q_shards, n_kv_shards,
                                  q_pos_offset, causal, &pl);
  if (hs != CASCADE_OK) return hs;
  *out_plan = nullptr;

  // one device blob, every array 256-byte aligned
  struct Seg {
    const void* src;
    size_t bytes;
    size_t off;
  };
  Seg segs[] = {
      {pl->q_off.data(), pl->q_off.size() * 4, 0},       {pl->q_idx.data(), pl->q_idx.size() * 4, 0},
      {pl->q_inv.data(), pl->q_inv.size() * 4, 0},       {pl->kv_off.data(), pl->kv_off.size() * 4, 0},
      {pl->kv_idx.data(), pl->kv_idx.size() * 4, 0},     {pl->kv_inv.data(), pl->kv_inv.size() * 4, 0},
      {pl->vis.data(), pl->vis.size() * 4, 0},           {pl->pair_class.data(), pl->pair_class.size(), 0},
      {pl->qtiles[0].data(), pl->qtiles[0].size() * 16, 0}, {pl->qtiles[1].data(), pl->qtiles[1].size() * 16, 0},
      {pl->qtiles[2].data(), pl->qtiles[2].size() * 16, 0}, {pl->qtiles[3].data(), pl->qtiles[3].size() * 16, 0},
      {pl->kv_slot_shard.data(), pl->kv_slot_shard.size() * 4, 0},
  };
  static_assert(kNumTileSizes == 4, "one upload segment per tile list");
  size_t total = 256;  // status word first
  for (auto& s : segs) {
    s.off = total;
    total += align_up(s.bytes, 256);
  }
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMalloc(&pl->dev_blob, total);
  if (e != cudaSuccess) {
    delete pl;
    set_error("cascade_shard_plan: cudaMalloc(%zu): %s", total, cudaGetErrorString(e));
    return CASCADE_ERR_ALLOC;
  }
  pl->dev_blob_bytes = total;
  char* base = (char*)pl->dev_blob;
  e = cudaMemsetAsync(base, 0, 256, st);
  for (auto& s : segs)
    if (e == cudaSuccess && s.bytes) e = cudaMemcpyAsync(base + s.off, s.src, s.bytes, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaFree(pl->dev_blob);
    delete pl;
    return cuda_fail(e, "cascade_shard_plan: upload");
  }
  pl->dev.status = (int32_t*)base;
  pl->dev.q_off = (const int32_t*)(base + segs[0].off);
  pl->dev.q_idx = (const int32_t*)(base + segs[1].off);
  pl->dev.q_inv = (const int32_t*)(base + segs[2].off);
  pl->dev.kv_off = (const int32_t*)(base + segs[3].off);
  pl->dev.kv_idx = (const int32_t*)(base + segs[4].off);
  pl->dev.kv_inv = (const int32_t*)(base + segs[5].off);
  pl->dev.vis = (const int32_t*)(base + segs[6].off);
  pl->dev.pair_class = (const uint8_t*)(base + segs[7].off);
  for (int ts = 0; ts < kNumTileSizes; ++ts) pl->dev.qtiles[ts] = (const int4*)(base + segs[8 + ts].off);
  pl->dev.kv_slot_shard = (const int32_t*)(base + segs[12].off);
  *out_plan = pl;
  return CASCADE_OK;
}

cascade_status_t cascade_shard_plan(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                    const int32_t* kv_shard_of, int32_t n_q_shards, int32_t n_kv_shards,
                                    int32_t q_pos_offset, int32_t causal, void* stream,
                                    cascade_plan_t** out_plan) {
  return plan_device(n_maps, n_q, n_kv, q_shard_of, kv_shard_of, nullptr, n_q_shards, n_kv_shards, q_pos_offset,
                     causal, stream, out_plan);
}

cascade_status_t cascade_shard_plan_resident(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                             const int32_t* kv_shard_of, const int32_t* kv_pos, int32_t n_q_shards,
                                             int32_t n_kv_shards, int32_t q_pos_offset, int32_t causal, void* stream,
                                             cascade_plan_t** out_plan) {
  if (!kv_pos) {
    set_error("cascade_shard_plan_resident: null kv_pos");
    return CASCADE_ERR_INVALID_ARG;
  }
  return plan_device(n_maps, n_q, n_kv, q_shard_of, kv_shard_of, kv_pos, n_q_shards, n_kv_shards, q_pos_offset, causal,
                     stream, out_plan);
}

cascade_status_t cascade_plan_destroy(cascade_plan_t* plan) {
  if (!plan) return CASCADE_OK;
  if (!plan->dev_blob) {  // host-only plan: nothing on the device
    delete plan;
    return CASCADE_OK;
  }
  cudaError_t e = cudaDeviceSynchronize();
  cudaFree(plan->dev_blob);
  delete plan;
  if (e != cudaSuccess) return cuda_fail(e, "cascade_plan_destroy: device synchronize");
  return CASCADE_OK;
}

cascade_status_t cascade_plan_get(const cascade_plan_t* plan, int32_t field, const void** host_ptr,
                                  const void** dev_ptr, int64_t* n_elems) {
  if (!plan) {
    set_error("cascade_plan_get: null plan");
    return CASCADE_ERR_INVALID_ARG;
  }
  const void* h = nullptr;
  const void* d = nullptr;
  int64_t n = 0;
  switch (field) {
    case CASCADE_PLAN_Q_OFF: h = plan->q_off.data(); d = plan->dev.q_off; n = plan->q_off.size(); break;
    case CASCADE_PLAN_Q_IDX: h = plan->q_idx.data(); d = plan->dev.q_idx; n = plan->q_idx.size(); break;
    case CASCADE_PLAN_Q_INV: h = plan->q_inv.data(); d = plan->dev.q_inv; n = plan->q_inv.size(); break;
    case CASCADE_PLAN_KV_OFF: h = plan->kv_off.data(); d = plan->dev.kv_off; n = plan->kv_off.size(); break;
    case CASCADE_PLAN_KV_IDX: h = plan->kv_idx.data(); d = plan->dev.kv_idx; n = plan->kv_idx.size(); break;
    case CASCADE_PLAN_KV_INV: h = plan->kv_inv.data(); d = plan->dev.kv_inv; n = plan->kv_inv.size(); break;
    case CASCADE_PLAN_VIS:
      refresh_host_vis(*plan, false);
      h = plan->vis.data(); d = plan->dev.vis; n = plan->vis.size(); break;
    case CASCADE_PLAN_PAIR_CLASS:
      refresh_host_vis(*plan, false);
      h = plan->pair_class.data(); d = plan->dev.pair_class; n = plan->pair_class.size(); break;
    default:
      set_error("cascade_plan_get: unknown field %d", field);
      return CASCADE_ERR_INVALID_ARG;
  }
  if (host_ptr) *host_ptr = h;
  if (dev_ptr) *dev_ptr = d;
  if (n_elems) *n_elems = n;
  return CASCADE_OK;
}

cascade_status_t cascade_plan_dense_mask(const cascade_plan_t* plan, int32_t map, int32_t j, int32_t k,
                                         uint8_t* host_out, int64_t capacity) {
  if (!plan || !host_out) {
    set_error("cascade_plan_dense_mask: null pointer");
    return CASCADE_ERR_INVALID_ARG;
  }
  refresh_host_vis(*plan, false);
  const PlanDev& d = plan->dev;
  if (map < 0 || map >= d.n_maps || j < 0 || j >= d.n_q_shards || k < 0 || k >= d.n_kv_shards) {
    set_error("cascade_plan_dense_mask: index out of range");
    return CASCADE_ERR_INVALID_ARG;
  }
  const int32_t* qo = plan->q_off.data() + (size_t)map * (d.n_q_shards + 1);
  const int32_t* ko = plan->kv_off.data() + (size_t)map * (d.n_kv_shards + 1);
  const int rows = qo[j + 1] - qo[j], cols = ko[k + 1] - ko[k];
  if ((int64_t)rows * cols > capacity) {
    set_error("cascade_plan_dense_mask: need %lld bytes, have %lld", (long long)rows * cols, (long long)capacity);
    return CASCADE_ERR_WORKSPACE;
  }
  const int32_t* vis = plan->vis.data() + (size_t)map * d.n_q * d.n_kv_shards;
  for (int r = 0; r < rows; ++r) {
    const int c_vis = vis[(size_t)(qo[j] + r) * d.n_kv_shards + k];
    for (int c = 0; c < cols; ++c) host_out[(size_t)r * cols + c] = c < c_vis ? 1 : 0;
  }
  return CASCADE_OK;
}

cascade_status_t cascade_plan_advance(cascade_plan_t* plan, int32_t q_pos_offset, void* stream) {
  if (!plan) {
    set_error("cascade_plan_advance: null plan");
    return CASCADE_ERR_INVALID_ARG;
  }
  const PlanDev& d = plan->dev;
  // A decode step (one query row, a few KV shards) is a handful of binary searches and a 64-byte upload: 3 us on the
  // host against 12 us for a dependent-load kernel.  Anything larger goes to the device.
  const int64_t n_vis = (int64_t)d.n_maps * d.n_q * d.n_kv_shards;
  if (plan->dev_blob && plan->kv_pos.empty() && n_vis > 256) {
    // Two small kernels rewrite vis and pair_class in stream order from the plan's own index arrays; nothing is
    // computed on the host and nothing is uploaded.  The host copies follow when they are next read.
    plan->dev.q_pos_offset = q_pos_offset;
    plan->host_vis_stale = true;
    cudaError_t e = launch_plan_advance(plan->dev, q_pos_offset, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "cascade_plan_advance: launch");
    return CASCADE_OK;
  }
  plan->dev.q_pos_offset = q_pos_offset;
  refresh_host_vis(*plan, true);
  if (plan->dev_blob) {
    // pageable source: the runtime stages it before the call returns, the device copy lands in stream order
    cudaError_t e = cudaMemcpyAsync(const_cast<int32_t*>(d.vis), plan->vis.data(), plan->vis.size() * 4,
                                    cudaMemcpyHostToDevice, (cudaStream_t)stream);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(const_cast<uint8_t*>(d.pair_class), plan->pair_class.data(), plan->pair_class.size(),
                          cudaMemcpyHostToDevice, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "cascade_plan_advance: upload");
  }
  return CASCADE_OK;
}

cascade_status_t cascade_plan_device_status(const cascade_plan_t* plan, int32_t* out_code) {
  if (!plan || !out_code || !plan->dev_blob) {
    set_error("cascade_plan_device_status: null pointer or host-only plan");
    return CASCADE_ERR_INVALID_ARG;
  }
  int32_t words[20] = {0};
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(words, plan->dev.status, sizeof(words), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_plan_device_status");
  *out_code = words[0];
  if (*out_code != 0) {
    set_error("device status word = %d: a bounded wait inside a kernel gave up (block %d,%d,%d tile %d; warp progress "
              "%d %d %d %d | %d %d %d %d | %d | %d %d %d)",
              words[0], words[1], words[2], words[3], words[4], words[8], words[9], words[10], words[11], words[12],
              words[13], words[14], words[15], words[16], words[17], words[18], words[19]);
    return CASCADE_ERR_TIMEOUT;
  }
  return CASCADE_OK;
}

}  // extern "C"

namespace cascade {

static size_t elt_size(cascade_dtype_t t) { return t == CASCADE_BF16 ? 2 : 4; }

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

static bool strides_ok(const cascade_strides_t& s, size_t es) {
  return (s.batch * (int64_t)es) % 16 == 0 && (s.token * (int64_t)es) % 16 == 0 && (s.head * (int64_t)es) % 16 == 0;
}

static cascade_status_t check_attn_args(const char* fn, const cascade_plan_t* plan, cascade_dtype_t dtype,
                                        int32_t batch, int32_t H, int32_t Hkv, int32_t d, float scale, const void* q,
                                        const cascade_strides_t& qs, const void* k, const cascade_strides_t& ks,
                                        const void* v, const cascade_strides_t& vs) {
  if (!plan || !q || !k || !v) {
    set_error("%s: null pointer", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!plan->dev_blob) {
    set_error("%s: the plan was built by cascade_shard_plan_host and has no device arrays", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (dtype != CASCADE_F32 && dtype != CASCADE_BF16) {
    set_error("%s: unknown dtype %d", fn, (int)dtype);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (batch < 1 || H < 1 || Hkv < 1) {
    set_error("%s: batch and head counts must be positive", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!(scale > 0.f) || !std::isfinite(scale)) {
    // the kernels take row maxima of the raw logits and scale afterwards, which needs a positive factor
    set_error("%s: scale must be positive and finite", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (H % Hkv != 0) {
    set_error("%s: n_heads %d is not a multiple of n_kv_heads %d", fn, H, Hkv);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (d != 64 && d != 128) {
    set_error("%s: head_dim %d unsupported (64 or 128)", fn, d);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (plan->dev.n_maps != 1 && plan->dev.n_maps != batch) {
    set_error("%s: plan has %d maps but batch is %d", fn, plan->dev.n_maps, batch);
    return CASCADE_ERR_INVALID_ARG;
  }
  const size_t es = elt_size(dtype);
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !strides_ok(qs, es) || !strides_ok(ks, es) ||
      !strides_ok(vs, es)) {
    set_error("%s: q/k/v pointers and row strides must be 16-byte aligned", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (batch > 65535 || H > 65535) {  // grid dimensions of the gather, decode and ALU kernels
    set_error("%s: batch and n_heads may not exceed 65535", fn);
    return CASCADE_ERR_UNSUPPORTED;
  }
  return CASCADE_OK;
}

static AttnParams make_params(const cascade_plan_t* plan, int32_t batch, int32_t H, int32_t Hkv, int32_t d,
                              float scale, const void* q, const cascade_strides_t& qs, const void* k,
                              const cascade_strides_t& ks, const void* v, const cascade_strides_t& vs) {
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.plan = plan->dev;
  p.q = q;
  p.k = k;
  p.v = v;
  p.qs = {qs.batch, qs.token, qs.head};
  p.ks = {ks.batch, ks.token, ks.head};
  p.vs = {vs.batch, vs.token, vs.head};
  p.batch = batch;
  p.H = H;
  p.Hkv = Hkv;
  p.G = H / Hkv;
  p.d = d;
  p.scale = scale;
  return p;
}

static bool use_decode(const cascade_plan_t* plan, cascade_dtype_t dtype, int H, int Hkv, int d) {
  const int G = H / Hkv;
  return plan->dev.n_q == 1 && dtype == CASCADE_BF16 && d == 128 && (G == 1 || G == 2 || G == 4 || G == 8);
}
static bool use_tc(const cascade_plan_t* plan, cascade_dtype_t dtype, int d) {
  // the tensor-core kernel keeps per-shard bookkeeping in shared memory: at most 256 KV shards
  return dtype == CASCADE_BF16 && d == 128 && plan->dev.n_q > 1 && plan->dev.n_kv_shards <= 256;
}

// Shard-major K and V copies for the tensor-core path: two regions of batch * kv_heads * n_kv rows of 256 bytes.
static size_t sorted_kv_bytes(const cascade_plan_t* plan, int batch, int Hkv) {
  return align_up((size_t)batch * Hkv * plan->dev.n_kv * 128 * 2, 256);
}

static size_t decode_ws_bytes(const cascade_plan_t* plan, cascade_dtype_t dtype, int batch, int H, int d) {
  const size_t rows = (size_t)batch * plan->dev.n_kv_shards * plan->dev.n_q * H;
  return align_up(rows * d * elt_size(dtype), 256) + 2 * align_up(rows * 4, 256);
}

// Tensor-core route: shard gather of K and V into the workspace, then the attention kernel (two launches).
static cascade_status_t run_tc(const AttnParams& p, const char* fn, const cascade_plan_t* plan, void* workspace,
                               size_t workspace_bytes, cudaStream_t st, cudaError_t* launch_error) {
  const size_t each = sorted_kv_bytes(plan, p.batch, p.Hkv);
  if (!workspace || workspace_bytes < 2 * each || ((uintptr_t)workspace & 255)) {
    set_error("%s: workspace of %zu bytes (256-byte aligned) required for the shard-major K/V copies, got %zu", fn,
              2 * each, workspace_bytes);
    return CASCADE_ERR_WORKSPACE;
  }
  char* ws = (char*)workspace;
  *launch_error = launch_gather_kv(p, ws, ws + each, st);
  if (*launch_error == cudaSuccess) *launch_error = launch_attn_tc(p, ws, ws + each, st);
  return CASCADE_OK;
}

// How many KV heads cascade_attn_sharded_host moves and computes at a time: enough that a strided row of the group's
// query heads is at least 1 KiB (256-byte rows made the 2-D copies slower than the pipelining gained; 2 KiB rows, i.e.
// half as many stages, were slower again: 0.80 / 0.66 / 0.72 ms on the headline shape), at most all of them.
static int host_call_group(int H, int Hkv, int d, size_t es) {
  const size_t row = (size_t)(H / Hkv) * d * es;
  int gs = 1;
  while (gs < Hkv && row * gs < 1024) ++gs;
  while (Hkv % gs != 0) ++gs;
  return gs;
}

// Device-side staging of cascade_attn_sharded_host: dense copies of q, k, v, o and the scratch of one head group's
// fused call, each region 256-byte aligned.
struct HostCallLayout {
  size_t q, k, v, o, inner, inner_bytes, total;
};
static HostCallLayout host_call_layout(const cascade_plan_t* plan, cascade_dtype_t dtype, int batch, int H, int Hkv,
                                       int d) {
  const size_t es = elt_size(dtype);
  const size_t q_bytes = (size_t)batch * plan->dev.n_q * H * d * es;
  const size_t kv_bytes = (size_t)batch * plan->dev.n_kv * Hkv * d * es;
  const int G = H / Hkv, gs = host_call_group(H, Hkv, d, es);
  HostCallLayout L;
  L.q = 0;
  L.k = L.q + align_up(q_bytes, 256);
  L.v = L.k + align_up(kv_bytes, 256);
  L.o = L.v + align_up(kv_bytes, 256);
  L.inner = L.o + align_up(q_bytes, 256);
  // gs KV heads and their query heads per inner call
  const bool decode = use_decode(plan, dtype, G * gs, gs, d);
  L.inner_bytes = decode ? decode_ws_bytes(plan, dtype, batch, G * gs, d)
                         : (use_tc(plan, dtype, d) ? 2 * sorted_kv_bytes(plan, batch, gs) : 0);
  L.total = L.inner + align_up(L.inner_bytes, 256);
  return L;
}

// Copy streams and events of cascade_attn_sharded_host, made on first use per device.
struct HostCallStreams {
  bool ready = false;
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t start = nullptr, done = nullptr;
  std::vector<cudaEvent_t> uploaded, computed;  // one pair per head group, created when a call first needs it
};
static HostCallStreams g_host_streams[64];

}  // namespace cascade

extern "C" {

cascade_status_t cascade_workspace_bytes(const cascade_plan_t* plan, int32_t which_call, cascade_dtype_t dtype,
                                         int32_t batch, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                         size_t* out_bytes) {
  if (!plan || !out_bytes) {
    set_error("cascade_workspace_bytes: null pointer");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (batch < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0) {
    set_error("cascade_workspace_bytes: bad batch or head counts");
    return CASCADE_ERR_INVALID_ARG;
  }
  const bool decode = use_decode(plan, dtype, n_heads, n_kv_heads, head_dim);
  const size_t tc_bytes = !decode && use_tc(plan, dtype, head_dim) ? 2 * sorted_kv_bytes(plan, batch, n_kv_heads) : 0;
  if (which_call == CASCADE_CALL_PARTIALS) {
    *out_bytes = tc_bytes;
  } else if (which_call == CASCADE_CALL_SHARDED) {
    *out_bytes = decode ? decode_ws_bytes(plan, dtype, batch, n_heads, head_dim) : tc_bytes;
  } else if (which_call == CASCADE_CALL_SHARDED_HOST) {
    *out_bytes = host_call_layout(plan, dtype, batch, n_heads, n_kv_heads, head_dim).total;
  } else if (which_call == CASCADE_CALL_DECODE_STEP_ROPE) {
    if (!decode) {
      set_error("cascade_workspace_bytes: the decode step needs a plan with one query row, bf16, head_dim 128");
      return CASCADE_ERR_UNSUPPORTED;
    }
    // the partials of the decode kernel, then the rotated query rows
    *out_bytes = align_up(decode_ws_bytes(plan, dtype, batch, n_heads, head_dim), 256) +
                 align_up((size_t)batch * n_heads * head_dim * elt_size(dtype), 256);
  } else {
    set_error("cascade_workspace_bytes: unknown call %d", which_call);
    return CASCADE_ERR_INVALID_ARG;
  }
  return CASCADE_OK;
}

cascade_status_t cascade_attn_partials(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                       int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                       const void* q, cascade_strides_t q_strides, const void* k,
                                       cascade_strides_t k_strides, const void* v, cascade_strides_t v_strides,
                                       void* o_part, float* m_part, float* l_part, void* workspace,
                                       size_t workspace_bytes, void* stream) {
  cascade_status_t s = check_attn_args("cascade_attn_partials", plan, dtype, batch, n_heads, n_kv_heads,
                                       head_dim, scale, q, q_strides, k, k_strides, v, v_strides);
  if (s != CASCADE_OK) return s;
  if (!o_part || !m_part || !l_part) {
    set_error("cascade_attn_partials: null output pointer");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!aligned16(o_part) || !aligned16(m_part) || !aligned16(l_part)) {
    set_error("cascade_attn_partials: outputs must be 16-byte aligned");
    return CASCADE_ERR_INVALID_ARG;
  }
  AttnParams p = make_params(plan, batch, n_heads, n_kv_heads, head_dim, scale, q, q_strides, k, k_strides, v,
                             v_strides);
  p.fused = 0;
  p.o_part = o_part;
  p.m_part = m_part;
  p.l_part = l_part;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (use_decode(plan, dtype, n_heads, n_kv_heads, head_dim)) {
    e = launch_decode(p, st);
  } else if (use_tc(plan, dtype, head_dim)) {
    cascade_status_t ws = run_tc(p, "cascade_attn_partials", plan, workspace, workspace_bytes, st, &e);
    if (ws != CASCADE_OK) return ws;
  } else {
    if ((int64_t)batch * plan->dev.n_kv_shards > 65535) {  // grid z of the ALU kernel on this route
      set_error("cascade_attn_partials: batch * n_kv_shards exceeds 65535 on the route without tensor cores");
      return CASCADE_ERR_UNSUPPORTED;
    }
    e = launch_attn_simt(p, dtype, st);
  }
  if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_partials: launch");
  return CASCADE_OK;
}

cascade_status_t cascade_merge(cascade_dtype_t dtype, int32_t batch, int32_t n_parts, int32_t n_rows,
                               int32_t n_heads, int32_t head_dim, const void* o_part, const float* m_part,
                               const float* l_part, const int32_t* row_scatter, int64_t row_scatter_batch_stride,
                               void* o_out, cascade_strides_t o_strides, float* lse_out, void* stream) {
  if (!o_part || !m_part || !l_part || !o_out) {
    set_error("cascade_merge: null pointer");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (dtype != CASCADE_F32 && dtype != CASCADE_BF16) {
    set_error("cascade_merge: unknown dtype %d", (int)dtype);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (batch < 1 || n_parts < 1 || n_rows < 1 || n_heads < 1) {
    set_error("cascade_merge: sizes must be positive");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (head_dim != 64 && head_dim != 128) {
    set_error("cascade_merge: head_dim %d unsupported (64 or 128)", head_dim);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (!aligned16(o_part) || !aligned16(o_out) || !strides_ok(o_strides, elt_size(dtype))) {
    set_error("cascade_merge: partial/output pointers and row strides must be 16-byte aligned");
    return CASCADE_ERR_INVALID_ARG;
  }
  MergeParams p;
  p.o_part = o_part;
  p.m_part = m_part;
  p.l_part = l_part;
  p.row_scatter = row_scatter;
  p.row_scatter_batch_stride = row_scatter_batch_stride;
  p.o_out = o_out;
  p.os = {o_strides.batch, o_strides.token, o_strides.head};
  p.lse_out = lse_out;
  p.batch = batch;
  p.n_parts = n_parts;
  p.n_rows = n_rows;
  p.H = n_heads;
  p.d = head_dim;
  cudaError_t e = launch_merge(p, dtype, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_merge: launch");
  return CASCADE_OK;
}

cascade_status_t cascade_merge_peers(cascade_dtype_t dtype, int32_t batch, int32_t n_sources,
                                     const void* const* o_parts, const float* const* m_parts,
                                     const float* const* l_parts, const int32_t* parts_per_source,
                                     int32_t n_source_rows, const int32_t* row_gather, int32_t n_rows,
                                     int32_t n_heads, int32_t head_dim, void* o_out, cascade_strides_t o_strides,
                                     float* lse_out, void* stream) {
  const char* fn = "cascade_merge_peers";
  if (!o_parts || !m_parts || !l_parts || !parts_per_source || !o_out) {
    set_error("%s: null pointer", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (dtype != CASCADE_F32 && dtype != CASCADE_BF16) {
    set_error("%s: unknown dtype %d", fn, (int)dtype);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (n_sources < 1 || n_sources > kMaxMergeSources) {
    set_error("%s: between 1 and %d sources", fn, kMaxMergeSources);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (batch < 1 || n_source_rows < 1 || n_rows < 1 || n_heads < 1) {
    set_error("%s: sizes must be positive", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (head_dim != 64 && head_dim != 128) {
    set_error("%s: head_dim %d unsupported (64 or 128)", fn, head_dim);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (!aligned16(o_out) || !strides_ok(o_strides, elt_size(dtype))) {
    set_error("%s: output pointer and row strides must be 16-byte aligned", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  MergePeersParams p;
  memset(&p, 0, sizeof(p));
  int total_parts = 0;
  for (int s = 0; s < n_sources; ++s) {
    if (parts_per_source[s] < 0 || (parts_per_source[s] > 0 && (!o_parts[s] || !m_parts[s] || !l_parts[s])) ||
        !aligned16(o_parts[s])) {
      set_error("%s: source %d: null or misaligned buffer, or a negative part count", fn, s);
      return CASCADE_ERR_INVALID_ARG;
    }
    p.o_src[s] = o_parts[s];
    p.m_src[s] = m_parts[s];
    p.l_src[s] = l_parts[s];
    p.parts[s] = parts_per_source[s];
    total_parts += parts_per_source[s];
  }
  if (total_parts < 1) {
    set_error("%s: no parts", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  p.n_src = n_sources;
  p.n_src_rows = n_source_rows;
  p.row_gather = row_gather;
  p.o_out = o_out;
  p.os = {o_strides.batch, o_strides.token, o_strides.head};
  p.lse_out = lse_out;
  p.batch = batch;
  p.n_rows = n_rows;
  p.H = n_heads;
  p.d = head_dim;
  cudaError_t e = launch_merge_peers(p, dtype, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_merge_peers: launch");
  return CASCADE_OK;
}

}  // extern "C"

// The fused route; rope_table != null adds the rotary step (cascade_attn_sharded_rope).
static cascade_status_t attn_sharded_impl(const char* fn, const cascade_plan_t* plan, cascade_dtype_t dtype,
                                          int32_t batch, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                                          float scale, const void* q, cascade_strides_t q_strides, const void* k,
                                          cascade_strides_t k_strides, const void* v, cascade_strides_t v_strides,
                                          const float* rope_table, int32_t n_positions, void* o_out,
                                          cascade_strides_t o_strides, float* lse_out, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  cascade_status_t s = check_attn_args(fn, plan, dtype, batch, n_heads, n_kv_heads, head_dim, scale, q, q_strides, k,
                                       k_strides, v, v_strides);
  if (s != CASCADE_OK) return s;
  if (!o_out) {
    set_error("%s: null output pointer", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!aligned16(o_out) || !strides_ok(o_strides, elt_size(dtype))) {
    set_error("%s: output pointer and row strides must be 16-byte aligned", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  AttnParams p = make_params(plan, batch, n_heads, n_kv_heads, head_dim, scale, q, q_strides, k, k_strides, v,
                             v_strides);
  if (rope_table) {
    if (!aligned16(rope_table)) {
      set_error("%s: the positional table must be 16-byte aligned", fn);
      return CASCADE_ERR_INVALID_ARG;
    }
    const int64_t need = std::max<int64_t>((int64_t)plan->dev.q_pos_offset + plan->dev.n_q, plan->dev.n_kv);
    if (n_positions < need) {
      set_error("%s: the positional table has %d rows, the plan needs %lld", fn, n_positions, (long long)need);
      return CASCADE_ERR_INVALID_ARG;
    }
    if (!plan->kv_pos.empty()) {
      set_error("%s: the rotary step takes a key row's position from its index, which a plan over resident K/V rows "
                "(cascade_shard_plan_resident) does not have", fn);
      return CASCADE_ERR_UNSUPPORTED;
    }
    if (use_decode(plan, dtype, n_heads, n_kv_heads, head_dim) || !use_tc(plan, dtype, head_dim)) {
      set_error("%s: the rotary step is fused on the tensor-core route only (bf16, head_dim 128, more than one query "
                "row, at most %d KV shards)", fn, 256);
      return CASCADE_ERR_UNSUPPORTED;
    }
    p.rope = reinterpret_cast<const float2*>(rope_table);
  }
  cudaStream_t st = (cudaStream_t)stream;
  if (use_decode(plan, dtype, n_heads, n_kv_heads, head_dim)) {
    // one query row per sequence: every KV shard is an independent partial, combined by the merge kernel
    const size_t need = decode_ws_bytes(plan, dtype, batch, n_heads, head_dim);
    if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) {
      set_error("%s: workspace of %zu bytes (256-byte aligned) required, got %zu", fn, need, workspace_bytes);
      return CASCADE_ERR_WORKSPACE;
    }
    const size_t rows = (size_t)batch * plan->dev.n_kv_shards * plan->dev.n_q * n_heads;
    char* ws = (char*)workspace;
    p.fused = 0;
    p.o_part = ws;
    p.m_part = (float*)(ws + align_up(rows * head_dim * elt_size(dtype), 256));
    p.l_part = (float*)((char*)p.m_part + align_up(rows * 4, 256));
    cudaError_t e = launch_decode(p, st);
    if (e != cudaSuccess) return cuda_fail(e, "attention (fused route): decode launch");
    MergeParams mp;
    mp.o_part = p.o_part;
    mp.m_part = p.m_part;
    mp.l_part = p.l_part;
    mp.row_scatter = nullptr;  // a single query row: slot 0 is token 0
    mp.row_scatter_batch_stride = 0;
    mp.o_out = o_out;
    mp.os = {o_strides.batch, o_strides.token, o_strides.head};
    mp.lse_out = lse_out;
    mp.batch = batch;
    mp.n_parts = plan->dev.n_kv_shards;
    mp.n_rows = plan->dev.n_q;
    mp.H = n_heads;
    mp.d = head_dim;
    e = launch_merge(mp, dtype, st);
    if (e != cudaSuccess) return cuda_fail(e, "attention (fused route): merge launch");
    return CASCADE_OK;
  }
  p.fused = 1;
  p.o_out = o_out;
  p.os = {o_strides.batch, o_strides.token, o_strides.head};
  p.lse_out = lse_out;
  cudaError_t e;
  if (use_tc(plan, dtype, head_dim)) {
    cascade_status_t ws = run_tc(p, fn, plan, workspace, workspace_bytes, st, &e);
    if (ws != CASCADE_OK) return ws;
  } else {
    e = launch_attn_simt(p, dtype, st);
  }
  if (e != cudaSuccess) return cuda_fail(e, "attention (fused route): launch");
  return CASCADE_OK;
}

extern "C" {

cascade_status_t cascade_attn_sharded(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                      int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                      const void* q, cascade_strides_t q_strides, const void* k,
                                      cascade_strides_t k_strides, const void* v, cascade_strides_t v_strides,
                                      void* o_out, cascade_strides_t o_strides, float* lse_out, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  return attn_sharded_impl("cascade_attn_sharded", plan, dtype, batch, n_heads, n_kv_heads, head_dim, scale, q,
                           q_strides, k, k_strides, v, v_strides, nullptr, 0, o_out, o_strides, lse_out, workspace,
                           workspace_bytes, stream);
}

cascade_status_t cascade_attn_sharded_rope(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                           int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                           const void* q, cascade_strides_t q_strides, const void* k,
                                           cascade_strides_t k_strides, const void* v, cascade_strides_t v_strides,
                                           const float* rope_table, int32_t n_positions, void* o_out,
                                           cascade_strides_t o_strides, float* lse_out, void* workspace,
                                           size_t workspace_bytes, void* stream) {
  if (!rope_table) {
    set_error("cascade_attn_sharded_rope: null positional table");
    return CASCADE_ERR_INVALID_ARG;
  }
  return attn_sharded_impl("cascade_attn_sharded_rope", plan, dtype, batch, n_heads, n_kv_heads, head_dim, scale, q,
                           q_strides, k, k_strides, v, v_strides, rope_table, n_positions, o_out, o_strides, lse_out,
                           workspace, workspace_bytes, stream);
}

cascade_status_t cascade_rope_table(int32_t n_positions, int32_t head_dim, double base, float* table, void* stream) {
  if (!table || n_positions < 1 || head_dim < 2 || head_dim % 2 != 0 || !(base > 1.0)) {
    set_error("cascade_rope_table: need a table pointer, n_positions >= 1, an even head_dim >= 2 and base > 1");
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!aligned16(table)) {
    set_error("cascade_rope_table: the table must be 16-byte aligned");
    return CASCADE_ERR_INVALID_ARG;
  }
  cudaError_t e = launch_rope_table(n_positions, head_dim, base, reinterpret_cast<float2*>(table),
                                    (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_rope_table: launch");
  return CASCADE_OK;
}

cascade_status_t cascade_rope_apply(cascade_dtype_t dtype, int32_t batch, int32_t n_rows, int32_t n_heads,
                                    int32_t head_dim, const void* x, cascade_strides_t x_strides,
                                    int32_t first_position, const float* rope_table, int32_t n_positions, void* y,
                                    cascade_strides_t y_strides, void* stream) {
  const char* fn = "cascade_rope_apply";
  if (!x || !y || !rope_table) {
    set_error("%s: null pointer", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (dtype != CASCADE_F32 && dtype != CASCADE_BF16) {
    set_error("%s: unknown dtype %d", fn, (int)dtype);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (head_dim != 64 && head_dim != 128) {
    set_error("%s: head_dim %d unsupported (64 or 128)", fn, head_dim);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (batch < 1 || n_rows < 1 || n_heads < 1 || first_position < 0 ||
      (int64_t)first_position + n_rows > (int64_t)n_positions) {
    set_error("%s: sizes must be positive and positions %d .. %lld must lie inside the table of %d rows", fn,
              first_position, (long long)first_position + n_rows - 1, n_positions);
    return CASCADE_ERR_INVALID_ARG;
  }
  const size_t es = elt_size(dtype);
  if (!aligned16(x) || !aligned16(y) || !aligned16(rope_table) || !strides_ok(x_strides, es) ||
      !strides_ok(y_strides, es)) {
    set_error("%s: pointers and row strides must be 16-byte aligned", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  cudaError_t e = launch_rope_apply(dtype, batch, n_rows, n_heads, head_dim, x,
                                    {x_strides.batch, x_strides.token, x_strides.head}, first_position,
                                    reinterpret_cast<const float2*>(rope_table), y,
                                    {y_strides.batch, y_strides.token, y_strides.head}, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_rope_apply: launch");
  return CASCADE_OK;
}

cascade_status_t cascade_decode_step_rope(cascade_plan_t* plan, int32_t batch, int32_t n_heads, int32_t n_kv_heads,
                                          float scale, const void* q_new, cascade_strides_t q_strides,
                                          const void* k_new, cascade_strides_t k_new_strides, const void* v_new,
                                          cascade_strides_t v_new_strides, void* k_cache,
                                          cascade_strides_t k_cache_strides, void* v_cache,
                                          cascade_strides_t v_cache_strides, int32_t position, const float* rope_table,
                                          int32_t n_positions, void* o_out, cascade_strides_t o_strides, float* lse_out,
                                          void* workspace, size_t workspace_bytes, void* stream) {
  const char* fn = "cascade_decode_step_rope";
  constexpr int kHeadDim = 128;
  if (!plan || !q_new || !k_new || !v_new || !k_cache || !v_cache || !rope_table || !o_out) {
    set_error("%s: null pointer", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  cascade_status_t s = check_attn_args(fn, plan, CASCADE_BF16, batch, n_heads, n_kv_heads, kHeadDim, scale, q_new,
                                       q_strides, k_cache, k_cache_strides, v_cache, v_cache_strides);
  if (s != CASCADE_OK) return s;
  if (!use_decode(plan, CASCADE_BF16, n_heads, n_kv_heads, kHeadDim) || !plan->kv_pos.empty()) {
    set_error("%s: needs a plan with one query row over the whole cache (cascade_shard_plan with n_q = 1) and "
              "n_heads / n_kv_heads in {1,2,4,8}", fn);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (position < 0 || position >= plan->dev.n_kv || position >= n_positions) {
    set_error("%s: position %d outside the cache of %d rows or the table of %d rows", fn, position, plan->dev.n_kv,
              n_positions);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(rope_table) || !aligned16(o_out) ||
      !strides_ok(k_new_strides, 2) || !strides_ok(v_new_strides, 2) || !strides_ok(o_strides, 2)) {
    set_error("%s: pointers and row strides must be 16-byte aligned", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  const size_t part_bytes = align_up(decode_ws_bytes(plan, CASCADE_BF16, batch, n_heads, kHeadDim), 256);
  const size_t need = part_bytes + align_up((size_t)batch * n_heads * kHeadDim * 2, 256);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) {
    set_error("%s: workspace of %zu bytes (256-byte aligned) required, got %zu", fn, need, workspace_bytes);
    return CASCADE_ERR_WORKSPACE;
  }
  // the new token sits at `position`: it is the query position, and the mask admits the cache rows up to it
  s = cascade_plan_advance(plan, position - plan->q_idx[0], stream);
  if (s != CASCADE_OK) return s;
  char* ws = (char*)workspace;
  void* q_rot = ws + part_bytes;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = launch_append_rope(batch, n_heads, n_kv_heads, q_new, {q_strides.batch, q_strides.token, q_strides.head},
                                     k_new, {k_new_strides.batch, k_new_strides.token, k_new_strides.head}, v_new,
                                     {v_new_strides.batch, v_new_strides.token, v_new_strides.head}, q_rot, k_cache,
                                     {k_cache_strides.batch, k_cache_strides.token, k_cache_strides.head}, v_cache,
                                     {v_cache_strides.batch, v_cache_strides.token, v_cache_strides.head}, position,
                                     reinterpret_cast<const float2*>(rope_table), st);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_decode_step_rope: append launch");
  const cascade_strides_t qr = {(int64_t)n_heads * kHeadDim, (int64_t)n_heads * kHeadDim, kHeadDim};
  return attn_sharded_impl(fn, plan, CASCADE_BF16, batch, n_heads, n_kv_heads, kHeadDim, scale, q_rot, qr, k_cache,
                           k_cache_strides, v_cache, v_cache_strides, nullptr, 0, o_out, o_strides, lse_out, ws, part_bytes,
                           st);
}

cascade_status_t cascade_attn_sharded_host(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                           int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                           const void* q_host, const void* k_host, const void* v_host, void* o_host,
                                           void* workspace, size_t workspace_bytes, void* stream) {
  const char* fn = "cascade_attn_sharded_host";
  if (!plan || !q_host || !k_host || !v_host || !o_host) {
    set_error("%s: null pointer", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (!plan->dev_blob) {
    set_error("%s: the plan was built by cascade_shard_plan_host and has no device arrays", fn);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (dtype != CASCADE_F32 && dtype != CASCADE_BF16) {
    set_error("%s: unknown dtype %d", fn, (int)dtype);
    return CASCADE_ERR_UNSUPPORTED;
  }
  if (batch < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads != 0 || n_kv_heads > kMaxHostGroups) {
    set_error("%s: bad batch or head counts (at most %d KV heads)", fn, kMaxHostGroups);
    return CASCADE_ERR_INVALID_ARG;
  }
  if (head_dim != 64 && head_dim != 128) {
    set_error("%s: head_dim %d unsupported (64 or 128)", fn, head_dim);
    return CASCADE_ERR_UNSUPPORTED;
  }
  const HostCallLayout L = host_call_layout(plan, dtype, batch, n_heads, n_kv_heads, head_dim);
  if (!workspace || workspace_bytes < L.total || ((uintptr_t)workspace & 255)) {
    set_error("%s: workspace of %zu bytes (256-byte aligned) required, got %zu", fn, L.total, workspace_bytes);
    return CASCADE_ERR_WORKSPACE;
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: cudaGetDevice");
  if (dev < 0 || dev >= 64) {
    set_error("%s: device ordinal %d not supported", fn, dev);
    return CASCADE_ERR_UNSUPPORTED;
  }
  HostCallStreams& hs = g_host_streams[dev];
  if (!hs.ready) {
    e = cudaStreamCreateWithFlags(&hs.h2d, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&hs.d2h, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&hs.start, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&hs.done, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: creating streams and events");
    hs.ready = true;
  }
  const int n_groups = n_kv_heads / host_call_group(n_heads, n_kv_heads, head_dim, elt_size(dtype));
  while ((int)hs.uploaded.size() < n_groups) {
    cudaEvent_t a = nullptr, b = nullptr;
    e = cudaEventCreateWithFlags(&a, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&b, cudaEventDisableTiming);
    if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: creating events");
    hs.uploaded.push_back(a);
    hs.computed.push_back(b);
  }
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  const size_t es = elt_size(dtype);
  const int G = n_heads / n_kv_heads;
  const int gs = host_call_group(n_heads, n_kv_heads, head_dim, es);  // KV heads per group
  const size_t q_rows = (size_t)batch * plan->dev.n_q, kv_rows = (size_t)batch * plan->dev.n_kv;
  const size_t q_pitch = (size_t)n_heads * head_dim * es, kv_pitch = (size_t)n_kv_heads * head_dim * es;
  const size_t q_width = (size_t)gs * G * head_dim * es;  // the query heads of one group, contiguous in a token row
  const cascade_strides_t qs = {(int64_t)plan->dev.n_q * n_heads * head_dim, (int64_t)n_heads * head_dim, head_dim};
  const cascade_strides_t ks = {(int64_t)plan->dev.n_kv * n_kv_heads * head_dim, (int64_t)n_kv_heads * head_dim,
                                head_dim};
  // the copy streams start after whatever the caller's stream has queued (it may still use the workspace)
  e = cudaEventRecord(hs.start, st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hs.h2d, hs.start, 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(hs.d2h, hs.start, 0);
  // K and V are small next to Q and O and contiguous: one copy each, up front (per-head copies of 256-byte rows were
  // measured slower than the pipelining gains)
  if (e == cudaSuccess) e = cudaMemcpyAsync(ws + L.k, k_host, kv_rows * kv_pitch, cudaMemcpyHostToDevice, hs.h2d);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ws + L.v, v_host, kv_rows * kv_pitch, cudaMemcpyHostToDevice, hs.h2d);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: queuing the K/V copies");
  for (int g = 0; g < n_kv_heads / gs; ++g) {
    const size_t q_off = (size_t)g * q_width, kv_off = (size_t)g * gs * head_dim * es;
    e = cudaMemcpy2DAsync(ws + L.q + q_off, q_pitch, (const char*)q_host + q_off, q_pitch, q_width, q_rows,
                          cudaMemcpyHostToDevice, hs.h2d);
    if (e == cudaSuccess) e = cudaEventRecord(hs.uploaded[g], hs.h2d);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, hs.uploaded[g], 0);
    if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: queuing a query copy");
    cascade_status_t rc = attn_sharded_impl(fn, plan, dtype, batch, G * gs, gs, head_dim, scale, ws + L.q + q_off, qs,
                                            ws + L.k + kv_off, ks, ws + L.v + kv_off, ks, nullptr, 0,
                                            ws + L.o + q_off, qs, nullptr, L.inner_bytes ? ws + L.inner : nullptr,
                                            L.inner_bytes, st);
    if (rc != CASCADE_OK) return rc;
    e = cudaEventRecord(hs.computed[g], st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(hs.d2h, hs.computed[g], 0);
    if (e == cudaSuccess)
      e = cudaMemcpy2DAsync((char*)o_host + q_off, q_pitch, ws + L.o + q_off, q_pitch, q_width, q_rows,
                            cudaMemcpyDeviceToHost, hs.d2h);
    if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: queuing an output copy");
  }
  // the caller's stream is done when the last output copy is
  e = cudaEventRecord(hs.done, hs.d2h);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, hs.done, 0);
  if (e != cudaSuccess) return cuda_fail(e, "cascade_attn_sharded_host: joining the copy stream");
  return CASCADE_OK;
}

}  // extern "C"
