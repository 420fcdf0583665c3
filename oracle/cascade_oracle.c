/*
 * Cascade sequence-sharded attention -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, fp64 restatement of what the paper's attention path computes, written from the
 * paper's definitions.  It exists to judge the CUDA library and to be timed as the CPU baseline;
 * it shares no source, header, table or helper with the CUDA path, and the CUDA path never calls it.
 * Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may load it.
 *
 * Tensors are token-major and contiguous:  q[B][n_q][H][d],  k,v[B][n_kv][H_KV][d]  (float32 holding
 * values already rounded to the I/O type; every product and sum below is in double).
 * Token positions are 0-based: query row i sits at position i + q_pos_offset, KV row y at position y.
 *
 * What pins each function (see tests/test_oracle_*.py):
 *   oracle_attention_unsharded  the textbook definition; checked against torch's fp64 causal SDPA,
 *                               brute force without max-subtraction on 8-token inputs, weights sum to 1
 *   oracle_attn_pass            Section 5.1 identities (un-normalised forms), the one-shard special case
 *   oracle_post_pass            the post-pass identity: merged result == unsharded attention for any
 *                               partition, any shard count, any token permutation
 *   oracle_shard_plan           Section 6.4 worked example (N=18), brute force on all maps of 8 tokens
 *   The paper prints no numeric m/e/u values for any input, so element values are pinned only through
 *   those identities and special cases ("parity unpinned by printed values").
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_EMPTY 0
#define ORACLE_PARTIAL 1
#define ORACLE_FULL 2

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* KV head serving query head h: the paper broadcasts H_KV heads to H ("repeat_kv" in the Attention-Pass
 * algorithm); contiguous groups of G = H / H_KV query heads share one KV head. */
static inline int kv_head_of(int h, int H, int Hkv) { return h / (H / Hkv); }

/* scale * <q_row, k_row> in double */
static inline double logit(const float* qr, const float* kr, int d, double scale) {
  double acc = 0.0;
  for (int c = 0; c < d; ++c) acc += (double)qr[c] * (double)kr[c];
  return acc * scale;
}

/*
 * Unsharded attention: the definition the sharded method must reproduce exactly
 * (Section 5.2.3: the post-pass sum equals softmax(a)[:, R_i, :] v).
 * For each selected query row i (rows_sel == NULL -> all rows), head h:
 *   a_y = scale * q_i . k_y   for every KV row y with y <= i + q_pos_offset (all y if !causal)
 *   o   = sum_y softmax(a)_y v_y,   lse = log sum_y exp(a_y)
 * Outputs: o[B][n_sel][H][d], lse[B][n_sel][H] (double).  A row with no visible key gives o = 0,
 * lse = -inf.
 */
void oracle_attention_unsharded(int B, int n_q, int n_kv, int H, int Hkv, int d, double scale,
                                int q_pos_offset, int causal, const float* q, const float* k,
                                const float* v, const int32_t* rows_sel, int n_sel, double* o,
                                double* lse) {
  const int n_rows = rows_sel ? n_sel : n_q;
  const long total = (long)B * n_rows * H;
#pragma omp parallel
  {
    double* a = (double*)malloc(sizeof(double) * (size_t)(n_kv > 0 ? n_kv : 1));
#pragma omp for schedule(dynamic, 8)
    for (long job = 0; job < total; ++job) {
      const int h = (int)(job % H);
      const int r = (int)((job / H) % n_rows);
      const int b = (int)(job / ((long)H * n_rows));
      const int i = rows_sel ? rows_sel[r] : r;
      const int g = kv_head_of(h, H, Hkv);
      const float* qr = q + (((size_t)b * n_q + i) * H + h) * d;
      long last = causal ? (long)i + q_pos_offset : (long)n_kv - 1;
      if (last > n_kv - 1) last = n_kv - 1;
      double* orow = o + (((size_t)b * n_rows + r) * H + h) * d;
      for (int c = 0; c < d; ++c) orow[c] = 0.0;
      if (last < 0) {
        lse[((size_t)b * n_rows + r) * H + h] = -INFINITY;
        continue;
      }
      double mx = -INFINITY;
      for (long y = 0; y <= last; ++y) {
        a[y] = logit(qr, k + (((size_t)b * n_kv + y) * Hkv + g) * d, d, scale);
        if (a[y] > mx) mx = a[y];
      }
      double sum = 0.0;
      for (long y = 0; y <= last; ++y) {
        a[y] = exp(a[y] - mx);
        sum += a[y];
      }
      for (long y = 0; y <= last; ++y) {
        const double w = a[y] / sum;
        const float* vr = v + (((size_t)b * n_kv + y) * Hkv + g) * d;
        for (int c = 0; c < d; ++c) orow[c] += w * (double)vr[c];
      }
      lse[((size_t)b * n_rows + r) * H + h] = mx + log(sum);
    }
    free(a);
  }
}

/*
 * Shard plan (Section 5.1: disjoint index sets S_j, T_k; Section 5.2.2: a shard's rows are kept in
 * ascending token order).  shard_of maps are per token; one map serves every sequence of the batch.
 *   off[s] .. off[s+1]  : slots of shard s in idx       (off has n_shards+1 entries)
 *   idx[slot]           : token id, ascending inside each shard
 *   inv[token]          : slot of that token            (idx[inv[t]] == t)
 *   vis[r][kk]          : for query slot r (shard-major order) and KV shard kk, the number of tokens
 *                         y of T_kk with y <= q_idx[r] + q_pos_offset (|T_kk| if !causal).  Because a
 *                         shard is sorted, the visible keys of a row are a prefix of the shard: the
 *                         sharded mask s^{S_j S_k} has each row = zeros followed by -inf (Appendix E).
 *   pair_class[j][kk]   : EMPTY if no row of S_j sees any key of T_kk, FULL if every row sees all of
 *                         them, else PARTIAL (an empty S_j or T_kk gives EMPTY).
 * Returns 0, or -1 if a shard id is out of range.
 */
int oracle_shard_plan(int n_q, int n_kv, const int32_t* q_shard_of, const int32_t* kv_shard_of,
                      int n_q_shards, int n_kv_shards, int q_pos_offset, int causal, int32_t* q_off,
                      int32_t* q_idx, int32_t* q_inv, int32_t* kv_off, int32_t* kv_idx,
                      int32_t* kv_inv, int32_t* vis, uint8_t* pair_class) {
  for (int t = 0; t < n_q; ++t)
    if (q_shard_of[t] < 0 || q_shard_of[t] >= n_q_shards) return -1;
  for (int t = 0; t < n_kv; ++t)
    if (kv_shard_of[t] < 0 || kv_shard_of[t] >= n_kv_shards) return -1;
  /* slot lists: walk shards in order, tokens in ascending order */
  int slot = 0;
  for (int s = 0; s < n_q_shards; ++s) {
    q_off[s] = slot;
    for (int t = 0; t < n_q; ++t)
      if (q_shard_of[t] == s) {
        q_idx[slot] = t;
        q_inv[t] = slot;
        ++slot;
      }
  }
  q_off[n_q_shards] = slot;
  slot = 0;
  for (int s = 0; s < n_kv_shards; ++s) {
    kv_off[s] = slot;
    for (int t = 0; t < n_kv; ++t)
      if (kv_shard_of[t] == s) {
        kv_idx[slot] = t;
        kv_inv[t] = slot;
        ++slot;
      }
  }
  kv_off[n_kv_shards] = slot;
  /* visible counts straight from the mask definition */
  for (int r = 0; r < n_q; ++r) {
    const long pos = (long)q_idx[r] + q_pos_offset;
    for (int kk = 0; kk < n_kv_shards; ++kk) {
      int cnt = 0;
      for (int s2 = kv_off[kk]; s2 < kv_off[kk + 1]; ++s2)
        if (!causal || (long)kv_idx[s2] <= pos) ++cnt;
      vis[(size_t)r * n_kv_shards + kk] = cnt;
    }
  }
  for (int j = 0; j < n_q_shards; ++j)
    for (int kk = 0; kk < n_kv_shards; ++kk) {
      const int len = kv_off[kk + 1] - kv_off[kk];
      int all_zero = 1, all_full = 1;
      for (int r = q_off[j]; r < q_off[j + 1]; ++r) {
        const int c = vis[(size_t)r * n_kv_shards + kk];
        if (c != 0) all_zero = 0;
        if (c != len) all_full = 0;
      }
      uint8_t cls = ORACLE_PARTIAL;
      if (all_zero) cls = ORACLE_EMPTY; /* also when S_j or T_kk is empty */
      else if (all_full) cls = ORACLE_FULL;
      pair_class[(size_t)j * n_kv_shards + kk] = cls;
    }
  return 0;
}

/*
 * Attention-pass of every AttnNode_{jk} (the AttnNode Single Layer Attention-Pass algorithm; the derived tensors m,
 * e, u of Section 5.1), from their definitions, one (query row, head, KV shard) at a time:
 *   a_y = scale * q . k_y  for the keys y of T_kk that the row may see (KV position <= query position; all of T_kk
 *         if !causal) -- the sharded mask s^{S_j T_kk} removes the others;
 *   m   = max_y a_y,   e = sum_y exp(a_y - m),   u = (sum_y exp(a_y - m) v_y) / e.
 * Rows evaluated: the n_rows query tokens listed in row_tok (normally q_idx, i.e. every slot in shard-major
 * order; a subset is allowed so that large cases can be sampled).  Outputs:
 *   u[B][n_kv_shards][n_rows][H][d],  m,e[B][n_kv_shards][n_rows][H]   (double).
 * A row that sees no key of the shard has m = -inf, e = 0, u = 0 (the definitions would divide by zero there; the
 * post-pass gives such a term weight zero).
 */
void oracle_attn_pass(int B, int n_q, int n_kv, int H, int Hkv, int d, double scale,
                      int q_pos_offset, int causal, const float* q, const float* k, const float* v,
                      const int32_t* row_tok, int n_rows, int n_kv_shards, const int32_t* kv_off,
                      const int32_t* kv_idx, double* u, double* m, double* e) {
  const long total = (long)B * n_kv_shards * n_rows * H;
#pragma omp parallel
  {
    double* a = (double*)malloc(sizeof(double) * (size_t)(n_kv > 0 ? n_kv : 1));
    int32_t* seen = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n_kv > 0 ? n_kv : 1));
#pragma omp for schedule(dynamic, 16)
    for (long job = 0; job < total; ++job) {
      const int h = (int)(job % H);
      const int r = (int)((job / H) % n_rows);
      const int kk = (int)((job / ((long)H * n_rows)) % n_kv_shards);
      const int b = (int)(job / ((long)H * n_rows * n_kv_shards));
      const int g = kv_head_of(h, H, Hkv);
      const int tok = row_tok[r];
      const long pos = (long)tok + q_pos_offset;
      const float* qr = q + (((size_t)b * n_q + tok) * H + h) * d;
      const size_t stat = (((size_t)b * n_kv_shards + kk) * n_rows + r) * H + h;
      double* urow = u + stat * d;
      for (int c = 0; c < d; ++c) urow[c] = 0.0;
      /* the keys of T_kk this row may see, and their scaled logits */
      int n_seen = 0;
      double mx = -INFINITY;
      for (int s2 = kv_off[kk]; s2 < kv_off[kk + 1]; ++s2) {
        const int y = kv_idx[s2];
        if (causal && (long)y > pos) continue;
        seen[n_seen] = y;
        a[n_seen] = logit(qr, k + (((size_t)b * n_kv + y) * Hkv + g) * d, d, scale);
        if (a[n_seen] > mx) mx = a[n_seen];
        ++n_seen;
      }
      if (n_seen == 0) {
        m[stat] = -INFINITY;
        e[stat] = 0.0;
        continue;
      }
      double sum = 0.0;
      for (int t = 0; t < n_seen; ++t) {
        const double w = exp(a[t] - mx);
        sum += w;
        const float* vr = v + (((size_t)b * n_kv + seen[t]) * Hkv + g) * d;
        for (int c = 0; c < d; ++c) urow[c] += w * (double)vr[c];
      }
      for (int c = 0; c < d; ++c) urow[c] /= sum;
      m[stat] = mx;
      e[stat] = sum;
    }
    free(a);
    free(seen);
  }
}

/*
 * Post-pass combine (the CompNode Single Layer Post-Pass algorithm up to the attention output; identity of
 * Section 5.2.3), for every row and head over the parts p:
 *   n = max_p m_p ;  w = sum_p exp(m_p - n) e_p ;  o = (sum_p exp(m_p - n) e_p u_p) / w.
 * Inputs in the layout oracle_attn_pass writes (parts = KV shards).  Output rows go back to token
 * order when row_scatter (= q_idx) is given: o[B][n_rows][H][d], lse[B][n_rows][H] = n + log w.
 * Parts with e_p = 0 (m_p = -inf) contribute nothing; if all parts are empty o = 0, lse = -inf.
 */
void oracle_post_pass(int B, int n_parts, int n_rows, int H, int d, const double* u, const double* m,
                      const double* e, const int32_t* row_scatter, double* o, double* lse) {
  const long total = (long)B * n_rows * H;
#pragma omp parallel for schedule(static)
  for (long job = 0; job < total; ++job) {
    const int h = (int)(job % H);
    const int r = (int)((job / H) % n_rows);
    const int b = (int)(job / ((long)H * n_rows));
    const int out_row = row_scatter ? row_scatter[r] : r;
    double* orow = o + (((size_t)b * n_rows + out_row) * H + h) * d;
    for (int c = 0; c < d; ++c) orow[c] = 0.0;
    double nmax = -INFINITY;
    for (int p = 0; p < n_parts; ++p) {
      const double mp = m[(((size_t)b * n_parts + p) * n_rows + r) * H + h];
      if (mp > nmax) nmax = mp;
    }
    if (nmax == -INFINITY) {
      lse[((size_t)b * n_rows + out_row) * H + h] = -INFINITY;
      continue;
    }
    double w = 0.0;
    for (int p = 0; p < n_parts; ++p) {
      const size_t stat = (((size_t)b * n_parts + p) * n_rows + r) * H + h;
      if (e[stat] == 0.0) continue;
      const double wt = exp(m[stat] - nmax) * e[stat];
      w += wt;
      const double* urow = u + stat * d;
      for (int c = 0; c < d; ++c) orow[c] += wt * urow[c];
    }
    for (int c = 0; c < d; ++c) orow[c] /= w;
    lse[((size_t)b * n_rows + out_row) * H + h] = nmax + log(w);
  }
}

/*
 * Softmax weights of one query row against all visible keys (used by the "rows sum to 1" pin and
 * by the brute-force comparison): w[y] for y in [0, n_kv), zero where masked.
 */
void oracle_softmax_row(int n_kv, int d, double scale, int pos, int causal, const float* q_row,
                        const float* k_rows /* [n_kv][d] */, double* w) {
  double mx = -INFINITY;
  for (int y = 0; y < n_kv; ++y) {
    if (causal && y > pos) {
      w[y] = -INFINITY;
      continue;
    }
    w[y] = logit(q_row, k_rows + (size_t)y * d, d, scale);
    if (w[y] > mx) mx = w[y];
  }
  double sum = 0.0;
  for (int y = 0; y < n_kv; ++y) {
    w[y] = (w[y] == -INFINITY) ? 0.0 : exp(w[y] - mx);
    sum += w[y];
  }
  for (int y = 0; y < n_kv; ++y) w[y] = sum > 0.0 ? w[y] / sum : 0.0;
}
