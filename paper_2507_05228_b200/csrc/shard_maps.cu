// Host-side shard-map generators and shard-safety measures (integer only, no device work): the (c, delta)-sharding
// of Section 6, the m-split of AttnNodes of Section 6.4, and the cluster/gap measures that Sections 6.2-6.3 and the
// collusion appendix tie to the vocab-matching threshold rho.  Their outputs are the token -> shard maps that
// cascade_shard_plan takes.
#include <stdint.h>

#include <vector>

#include "cascade_internal.cuh"

using cascade::set_error;

extern "C" {

cascade_status_t cascade_cdelta_shard_map(int32_t n_tokens, int32_t c, int32_t delta, int32_t* shard_of,
                                          int32_t* n_shards_out) {
  if (n_tokens < 0 || c < 1 || delta < c || (!shard_of && n_tokens > 0)) {
    set_error("cascade_cdelta_shard_map: need n_tokens >= 0, 1 <= c <= delta and an output array");
    return CASCADE_ERR_INVALID_ARG;
  }
  // token t sits at offset t mod delta of its period; offsets [i c, i c + c) belong to sequence i
  int32_t offset = 0, shard = 0, in_cluster = 0;
  for (int32_t t = 0; t < n_tokens; ++t) {
    shard_of[t] = shard;
    ++offset;
    if (++in_cluster == c) {
      in_cluster = 0;
      ++shard;
    }
    if (offset == delta) offset = 0, shard = 0, in_cluster = 0;
  }
  if (n_shards_out) *n_shards_out = (delta + c - 1) / c;  // alpha = ceil(delta / c)
  return CASCADE_OK;
}

cascade_status_t cascade_msplit_shard_map(int32_t n_tokens, const int32_t* r_shard_of, int32_t n_r_shards, int32_t m,
                                          int32_t* s_shard_of) {
  if (n_tokens < 0 || n_r_shards < 1 || m < 1 || (n_tokens > 0 && (!r_shard_of || !s_shard_of))) {
    set_error("cascade_msplit_shard_map: need n_tokens >= 0, n_r_shards >= 1, m >= 1 and both arrays");
    return CASCADE_ERR_INVALID_ARG;
  }
  if ((int64_t)n_r_shards * m > INT32_MAX) {
    set_error("cascade_msplit_shard_map: %d x %d shards overflow", n_r_shards, m);
    return CASCADE_ERR_INVALID_ARG;
  }
  // walking the tokens in ascending order visits each R_i in sorted order: the x-th, (x+m)-th, ... member goes to R_{i,x}
  std::vector<int32_t> next_piece((size_t)n_r_shards, 0);
  for (int32_t t = 0; t < n_tokens; ++t) {
    const int32_t i = r_shard_of[t];
    if (i < 0 || i >= n_r_shards) {
      set_error("cascade_msplit_shard_map: r_shard_of[%d] = %d outside [0, %d)", t, i, n_r_shards);
      return CASCADE_ERR_BAD_MAP;
    }
    s_shard_of[t] = m * i + next_piece[i];
    if (++next_piece[i] == m) next_piece[i] = 0;
  }
  return CASCADE_OK;
}

cascade_status_t cascade_index_set_gaps(int32_t n_tokens, const uint8_t* held, int32_t* n_indices, int32_t* n_clusters,
                                        int32_t* min_gap, int32_t* max_gap) {
  if (n_tokens < 0 || (n_tokens > 0 && !held)) {
    set_error("cascade_index_set_gaps: need n_tokens >= 0 and the membership flags");
    return CASCADE_ERR_INVALID_ARG;
  }
  int32_t count = 0, clusters = 0, lo = -1, hi = -1;
  int32_t run_missing = 0;  // unheld tokens since the last held one
  bool seen = false;
  for (int32_t t = 0; t < n_tokens; ++t) {
    if (!held[t]) {
      ++run_missing;
      continue;
    }
    ++count;
    if (!seen) {
      clusters = 1;
    } else if (run_missing > 0) {
      ++clusters;
      if (lo < 0 || run_missing < lo) lo = run_missing;
      if (run_missing > hi) hi = run_missing;
    }
    seen = true;
    run_missing = 0;
  }
  if (n_indices) *n_indices = count;
  if (n_clusters) *n_clusters = clusters;
  if (min_gap) *min_gap = lo;
  if (max_gap) *max_gap = hi;
  return CASCADE_OK;
}

cascade_status_t cascade_kl_gaps(int32_t n_tokens, const uint8_t* r_held, const int32_t* s_shard_of, int32_t n_s_shards,
                                 int32_t* min_gap_per_shard) {
  if (n_tokens < 0 || n_s_shards < 1 || !min_gap_per_shard || (n_tokens > 0 && (!r_held || !s_shard_of))) {
    set_error("cascade_kl_gaps: need n_tokens >= 0, n_s_shards >= 1 and all three arrays");
    return CASCADE_ERR_INVALID_ARG;
  }
  for (int32_t k = 0; k < n_s_shards; ++k) min_gap_per_shard[k] = -1;
  // between two neighbouring indices of the node, count the foreign tokens per KV shard; close the counts at the next
  // index of the node (tokens before its first and after its last index bound no gap)
  std::vector<int32_t> count((size_t)n_s_shards, 0);
  std::vector<int32_t> touched;
  bool open = false;
  for (int32_t t = 0; t < n_tokens; ++t) {
    if (r_held[t]) {
      for (int32_t k : touched) {
        if (open && (min_gap_per_shard[k] < 0 || count[k] < min_gap_per_shard[k])) min_gap_per_shard[k] = count[k];
        count[k] = 0;
      }
      touched.clear();
      open = true;
      continue;
    }
    const int32_t k = s_shard_of[t];
    if (k < 0 || k >= n_s_shards) {
      set_error("cascade_kl_gaps: s_shard_of[%d] = %d outside [0, %d)", t, k, n_s_shards);
      return CASCADE_ERR_BAD_MAP;
    }
    if (count[k]++ == 0) touched.push_back(k);
  }
  return CASCADE_OK;
}

}  // extern "C"
