/*
 * cascade.h -- C ABI of the B200 (sm_100a) library for Cascade's sequence-sharded attention.
 *
 * The paper (Cascade: Token-Sharded Private LLM Inference) splits the tokens of a layer into disjoint
 * index sets -- query shards S_j and key/value shards T_k (Section 5.1) -- lets one "AttnNode" per pair
 * (j, k) compute a partial attention output u with per-row statistics m (row max) and e (sum of
 * exponentials) (the Attention-Pass algorithm), and combines the partials over k with a log-sum-exp weighted average
 * (Section 5.2.3, the Post-Pass algorithm), which reproduces unsharded softmax attention exactly.
 * This library runs all parties on one GPU.
 *
 * Conventions
 *  - Every function returns a cascade_status_t; CASCADE_OK is 0.  Nothing throws or aborts across the ABI.
 *    cascade_last_error() returns a thread-local, NUL-terminated description of the last failure.
 *  - Pointers named *_dev / q / k / v / o_* / m_* / l_* / workspace are DEVICE pointers owned by the
 *    caller.  Token-to-shard maps and read-back buffers are HOST pointers.
 *  - All GPU work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL = default
 *    stream) without synchronising, except where a function says it synchronises.  On the tensor-core route
 *    the attention grid is launched as a programmatic dependent of the K/V gather grid of the same call, so
 *    the two overlap; both are ordered after earlier work on the stream and before later work, as usual.
 *  - The library allocates device memory only inside cascade_shard_plan (released by
 *    cascade_plan_destroy).  Scratch memory is caller-provided after cascade_workspace_bytes.
 *  - Token ids, shard ids, rows and positions are 0-based.  Query row i of a sequence sits at position
 *    i + q_pos_offset; KV row y at position y.  With causal != 0 row i sees KV rows y <= i + q_pos_offset.
 *  - Tensors are token-major: element (b, token, head, c) lives at
 *    base + b*strides.batch + token*strides.token + head*strides.head + c   (units: elements, c contiguous).
 *    Row starts must be 16-byte aligned.
 *  - Query head h reads KV head h / (n_heads / n_kv_heads)  ("repeat_kv", the Attention-Pass algorithm).
 *  - "Shard-major row order": query rows listed shard 0 first, then shard 1, ..., ascending token id
 *    inside a shard (Section 5.2.2: rows are concatenated in sorted order).  Slot r of that order holds
 *    token Q_IDX[r].
 *  - Statistics: m is the true row maximum of the scaled, masked logits in natural-log units, l is
 *    sum exp(a - m) (the paper's e), both fp32.  A row that sees no key of a shard has m = -inf, l = 0 and
 *    an all-zero partial output.  The stored partial output is the paper's u: normalised inside its shard.
 */
#ifndef CASCADE_H_
#define CASCADE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t cascade_status_t;
enum {
  CASCADE_OK = 0,
  CASCADE_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, misaligned pointer or stride */
  CASCADE_ERR_BAD_MAP = 2,      /* shard id outside [0, n_shards) */
  CASCADE_ERR_UNSUPPORTED = 3,  /* head_dim not in {64,128}, n_heads % n_kv_heads != 0, unknown dtype */
  CASCADE_ERR_WORKSPACE = 4,    /* workspace missing or smaller than cascade_workspace_bytes reports */
  CASCADE_ERR_ALLOC = 5,        /* host or device allocation failed */
  CASCADE_ERR_CUDA = 6,         /* a CUDA runtime call or launch failed */
  CASCADE_ERR_TIMEOUT = 7       /* a bounded device-side wait gave up (see cascade_plan_device_status) */
};

typedef enum { CASCADE_F32 = 0, CASCADE_BF16 = 1 } cascade_dtype_t;

/* Strides in elements; the head_dim axis is contiguous. */
typedef struct {
  int64_t batch, token, head;
} cascade_strides_t;

typedef struct cascade_plan cascade_plan_t; /* opaque, library-owned */

/* Plan arrays readable with cascade_plan_get.  All int32 except PAIR_CLASS (uint8).
 * Leading dimension n_maps (1 when one map serves the whole batch). */
enum {
  CASCADE_PLAN_Q_OFF = 0,      /* [n_maps][n_q_shards+1]   first slot of each query shard            */
  CASCADE_PLAN_Q_IDX = 1,      /* [n_maps][n_q]            token id held by each shard-major slot     */
  CASCADE_PLAN_Q_INV = 2,      /* [n_maps][n_q]            slot of each token                         */
  CASCADE_PLAN_KV_OFF = 3,     /* [n_maps][n_kv_shards+1]                                             */
  CASCADE_PLAN_KV_IDX = 4,     /* [n_maps][n_kv]                                                      */
  CASCADE_PLAN_KV_INV = 5,     /* [n_maps][n_kv]                                                      */
  CASCADE_PLAN_VIS = 6,        /* [n_maps][n_q][n_kv_shards] visible-prefix length of slot r in T_k   */
  CASCADE_PLAN_PAIR_CLASS = 7  /* [n_maps][n_q_shards][n_kv_shards]  0 EMPTY, 1 PARTIAL, 2 FULL       */
};
enum { CASCADE_PAIR_EMPTY = 0, CASCADE_PAIR_PARTIAL = 1, CASCADE_PAIR_FULL = 2 };

int32_t cascade_version(void);
const char* cascade_last_error(void);

/* Number of kernels this library has launched in this process (monotone; for benchmark accounting). */
int64_t cascade_launch_count(void);

/*
 * Device-side timing of the attention kernel (for roofline accounting; not a step of the method).  Between
 * cascade_kernel_timing_begin() and cascade_kernel_timing_end() every launch of the tensor-core attention kernel or of
 * the decode kernel is bracketed by a pair of CUDA events recorded on the launch stream (at most 8192 launches; later
 * ones are not timed).  cascade_kernel_timing_end SYNCHRONISES the device, stops the recording and returns the summed
 * duration in milliseconds and the number of timed launches (either pointer may be NULL).  The shard-gather and merge
 * launches are not included.  Not thread-safe against concurrent attention calls.  Errors: CUDA.
 */
cascade_status_t cascade_kernel_timing_begin(void);
cascade_status_t cascade_kernel_timing_end(double* total_ms, int64_t* n_launches);

/*
 * cascade_shard_plan -- index maps and causal pair mask (Section 5.1 index sets; Section 5.2.2 sorted
 * concatenation; the sharded mask s^{S_j T_k} = s[:, S_j, T_k]).
 * Because each shard is kept in ascending token order and the mask is unidirectional, row r of pair
 * (j, k) sees exactly the first VIS[r][k] keys of T_k (each mask row is visible entries followed by
 * -inf, Appendix E), so the mask is stored as that prefix length.
 *   n_maps        1 (one map for every sequence) or the batch size (maps laid out [n_maps][n])
 *   q_shard_of    HOST int32 [n_maps][n_q],  values in [0, n_q_shards)
 *   kv_shard_of   HOST int32 [n_maps][n_kv], values in [0, n_kv_shards)
 *   q_pos_offset  position of query row 0 (0 for prefill, n_kv - n_q for decode with the new tokens
 *                 already in the cache)
 *   causal        1 unidirectional mask, 0 no mask
 * Copies the maps, builds the arrays on the host, uploads them on `stream` and SYNCHRONISES that stream.
 * Empty shards are allowed.  Errors: INVALID_ARG, BAD_MAP, ALLOC, CUDA.  *out_plan is set only on success.
 */
cascade_status_t cascade_shard_plan(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                    const int32_t* kv_shard_of, int32_t n_q_shards, int32_t n_kv_shards,
                                    int32_t q_pos_offset, int32_t causal, void* stream,
                                    cascade_plan_t** out_plan);

/*
 * cascade_shard_plan_resident -- a plan for a party that holds only SOME of the K/V rows: an AttnNode keeps the k, v
 * rows of its own KV shards and nothing else (Section 5.2: every AttnNode_{jk} receives k^{T_k}, v^{T_k}; "Caching" in
 * the appendix on cost optimizations: each node stores the rows of its shard).  The k/v tensors of the attention calls
 * then have n_kv = (number of resident rows) rows, and row y is the token at ORIGINAL position kv_pos[y]; the causal
 * mask compares that position with the query position, so VIS[r][k] = #{y in T_k : kv_pos[y] <= q_idx[r] + q_pos_offset}.
 *   kv_pos   HOST int32 [n_maps][n_kv], non-negative and strictly ascending inside a map (rows kept in token order)
 * Everything else as cascade_shard_plan (which is this call with kv_pos[y] = y).  The partials of such a plan are the
 * columns of the full problem's partials that belong to the resident shards; cascade_merge over the union of all
 * parties' columns gives the exact result (Section 5.2.3).  cascade_attn_sharded_rope refuses these plans (it takes a
 * key row's position from its index).  Errors as cascade_shard_plan; BAD_MAP also for a kv_pos that is not ascending.
 */
cascade_status_t cascade_shard_plan_resident(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                             const int32_t* kv_shard_of, const int32_t* kv_pos, int32_t n_q_shards,
                                             int32_t n_kv_shards, int32_t q_pos_offset, int32_t causal, void* stream,
                                             cascade_plan_t** out_plan);
/* The same, built on the host only (see cascade_shard_plan_host). */
cascade_status_t cascade_shard_plan_resident_host(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                                  const int32_t* kv_shard_of, const int32_t* kv_pos,
                                                  int32_t n_q_shards, int32_t n_kv_shards, int32_t q_pos_offset,
                                                  int32_t causal, cascade_plan_t** out_plan);

/* Same arrays as cascade_shard_plan, built on the host only: no CUDA call is made, so it works on a machine
 * without a GPU.  The plan can be read with cascade_plan_get / cascade_plan_dense_mask (device pointers are
 * NULL) and must be destroyed as usual; the attention calls reject it with INVALID_ARG. */
cascade_status_t cascade_shard_plan_host(int32_t n_maps, int32_t n_q, int32_t n_kv, const int32_t* q_shard_of,
                                         const int32_t* kv_shard_of, int32_t n_q_shards, int32_t n_kv_shards,
                                         int32_t q_pos_offset, int32_t causal, cascade_plan_t** out_plan);

/* Frees host and device memory of a plan (NULL is accepted).  Synchronises the device first. */
cascade_status_t cascade_plan_destroy(cascade_plan_t* plan);

/* Read-back of a plan array: host copy (library-owned, valid until destroy), device copy and element
 * count.  Any of the three outputs may be NULL. */
cascade_status_t cascade_plan_get(const cascade_plan_t* plan, int32_t field, const void** host_ptr,
                                  const void** dev_ptr, int64_t* n_elems);

/* Dense mask of pair (j, k) of map `map`: host_out[r * |T_k| + c] = 1 if row r of S_j sees key c of T_k.
 * capacity = bytes available at host_out; WORKSPACE error if smaller than |S_j| * |T_k|. */
cascade_status_t cascade_plan_dense_mask(const cascade_plan_t* plan, int32_t map, int32_t j, int32_t k,
                                         uint8_t* host_out, int64_t capacity);

/* Reads the plan's device status word (SYNCHRONISES the device): 0 = no kernel that used this plan hit a
 * bounded-wait limit; otherwise a code identifying the wait.  Returns TIMEOUT if non-zero.
 * The word is sticky: once a wait inside the tensor-core kernel has given up (2 s without progress), every later
 * attention call on this plan returns CASCADE_OK from the host but its blocks exit at once and write nothing.  A
 * non-zero status therefore invalidates the outputs of every call made on the plan since the last check that read 0;
 * destroy the plan and build a new one.  A caller that cannot afford stale outputs polls this after the calls whose
 * results it is about to use. */
cascade_status_t cascade_plan_device_status(const cascade_plan_t* plan, int32_t* out_code);

/*
 * cascade_attn_partials -- the attention-pass of every AttnNode_{jk} (the Attention-Pass algorithm) in one launch:
 * for each query shard j and KV shard k, a = scale * q^{S_j} (k^{T_k})^T + s^{S_j T_k}; m = row max;
 * l = row sum exp(a - m); u = softmax(a) v^{T_k}.  Rows of Q/K/V are gathered through the plan's maps.
 *   q  [batch][n_q][n_heads][head_dim], k, v [batch][n_kv][n_kv_heads][head_dim]  (strides given)
 *   o_part  [batch][n_kv_shards][n_q shard-major][n_heads][head_dim], same dtype as q, contiguous
 *   m_part, l_part  fp32 [batch][n_kv_shards][n_q shard-major][n_heads], contiguous
 * (Together these are the paper's stage-B payload: n_kv_shards * (head_dim + 2) * n_heads * n_q values
 * per sequence, Appendix D.)  batch must equal n_maps when the plan has per-sequence maps.
 * head_dim in {64,128}; bf16 with head_dim 128 runs on the tensor cores (tcgen05), everything else on
 * the fp32 ALU kernel; n_q == 1 with bf16 runs the KV-streaming decode kernel.
 * scale must be positive and finite (INVALID_ARG otherwise: the kernels take row maxima before scaling).
 * Only the k/v rows that some query row of the plan sees have to hold finite values: positions later than the last
 * query position (the unwritten tail of a preallocated cache) may hold anything, NaN bit patterns included; no route
 * lets them reach a result.  batch and n_heads may not exceed 65535 (and batch * n_kv_shards on the ALU route).
 * workspace: as reported by cascade_workspace_bytes(CASCADE_CALL_PARTIALS) (may be 0 -> NULL allowed).  The
 * tensor-core route first copies K and V into shard-major order there (the stage-A hand-over of each KV shard to
 * its AttnNodes, Appendix D): 2 * batch * n_kv_heads * n_kv * head_dim * 2 bytes, overwritten by every call.
 */
cascade_status_t cascade_attn_partials(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                       int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                       const void* q, cascade_strides_t q_strides, const void* k,
                                       cascade_strides_t k_strides, const void* v,
                                       cascade_strides_t v_strides, void* o_part, float* m_part,
                                       float* l_part, void* workspace, size_t workspace_bytes,
                                       void* stream);

/*
 * cascade_merge -- the post-pass combine (the Post-Pass algorithm; derivation in Section 5.2.3):
 * n = max_p m_p;  w = sum_p exp(m_p - n) l_p;  o = sum_p exp(m_p - n) l_p u_p / w.
 * Needs no plan.  Inputs in the layout cascade_attn_partials writes, with n_parts = n_kv_shards.
 *   row_scatter  DEVICE int32 [n_rows] or NULL: output token row of partial row r (the plan's Q_IDX
 *                device array); NULL = identity.  With per-sequence maps pass row_scatter_batch_stride
 *                = n_rows, else 0.
 *   o_out        [batch][n_rows][n_heads][head_dim] with strides, dtype as the partials
 *   lse_out      optional fp32 [batch][n_rows][n_heads] (token order): n + ln w; -inf if all parts empty
 * Rows whose parts are all empty produce zeros.
 */
cascade_status_t cascade_merge(cascade_dtype_t dtype, int32_t batch, int32_t n_parts, int32_t n_rows,
                               int32_t n_heads, int32_t head_dim, const void* o_part, const float* m_part,
                               const float* l_part, const int32_t* row_scatter,
                               int64_t row_scatter_batch_stride, void* o_out, cascade_strides_t o_strides,
                               float* lse_out, void* stream);

/*
 * cascade_merge_peers -- stage B of the layer and the post-pass combine in one kernel (Single Layer Forward Pass
 * algorithm: "CompNode_i gets m, e, u" from the AttnNodes, then the Post-Pass algorithm; Section 5.2.3): the parts are
 * read where they were computed instead of being copied to the combining party first.  Source s is the set of
 * partial buffers one party wrote with cascade_attn_partials for ITS KV shards (cascade_shard_plan_resident):
 *   o_parts[s]  DEVICE [batch][parts_per_source[s]][n_source_rows][n_heads][head_dim] in `dtype`
 *   m_parts[s], l_parts[s]  DEVICE fp32 [batch][parts_per_source[s]][n_source_rows][n_heads]
 * The three pointer tables and parts_per_source are HOST arrays of n_sources entries (at most 16).  A source pointer
 * may address another GPU's memory that is mapped into this process (CUDA IPC, peer access): the kernel reads it
 * with plain loads, each 16-byte piece once; it uses no multicast and no TMA.  The caller orders this call after the
 * writers of every source (their streams, or a barrier between processes).
 *   row_gather  DEVICE int32 [n_rows] or NULL: the row of the source buffers (shard-major slot of the whole sequence)
 *               that output row r combines -- the rows of the query shards this party owns; NULL = row r
 *   o_out       [batch][n_rows][n_heads][head_dim] with strides;  lse_out optional fp32 [batch][n_rows][n_heads]
 * The result equals cascade_merge over the union of all sources' parts restricted to the gathered rows.
 * Errors: INVALID_ARG, UNSUPPORTED (dtype, head_dim, more than 16 sources), CUDA.
 */
cascade_status_t cascade_merge_peers(cascade_dtype_t dtype, int32_t batch, int32_t n_sources,
                                     const void* const* o_parts, const float* const* m_parts,
                                     const float* const* l_parts, const int32_t* parts_per_source,
                                     int32_t n_source_rows, const int32_t* row_gather, int32_t n_rows,
                                     int32_t n_heads, int32_t head_dim, void* o_out, cascade_strides_t o_strides,
                                     float* lse_out, void* stream);

/*
 * cascade_attn_sharded -- attention-pass and post-pass fused (the Attention-Pass algorithm followed by the Post-Pass algorithm): walks the KV shards of the plan one after another for each query-shard tile and carries
 * (n, w, o) across shards, so no partial is written to memory; by the identity of Section 5.2.3 the
 * result equals cascade_merge(cascade_attn_partials(...)).  Output in token order:
 *   o_out [batch][n_q][n_heads][head_dim] with strides; lse_out optional fp32 [batch][n_q][n_heads].
 * For n_q == 1 (decode, Appendix F "Caching") the KV shards are processed as independent partials in
 * `workspace` and merged by a second launch.  The tensor-core route (bf16, head_dim 128) uses `workspace` for
 * the shard-major K/V copies as cascade_attn_partials does.  Size: cascade_workspace_bytes(CASCADE_CALL_SHARDED).
 */
cascade_status_t cascade_attn_sharded(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                      int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                      const void* q, cascade_strides_t q_strides, const void* k,
                                      cascade_strides_t k_strides, const void* v,
                                      cascade_strides_t v_strides, void* o_out,
                                      cascade_strides_t o_strides, float* lse_out, void* workspace,
                                      size_t workspace_bytes, void* stream);

/*
 * cascade_rope_table -- the positional table p of the rotary embedding (Section 5.1 lists p among the tensors set up
 * before inference and sharded with the tokens; the Pre-Pass algorithm consumes its rows p^{R_i}).  The paper does not print
 * the rotary formula; this library takes the rotate-half form with theta_i = base^(-2 i / head_dim):
 *   table[t][i] = (cos(t theta_i), sin(t theta_i)),  t = 0 .. n_positions-1,  i = 0 .. head_dim/2 - 1,
 * angles formed and evaluated in fp64, stored as fp32 pairs.
 *   table  DEVICE fp32 [n_positions][head_dim/2][2], 16-byte aligned, caller-owned; written on `stream`.
 * Errors: CASCADE_ERR_INVALID_ARG (null / misaligned table, n_positions < 1, odd head_dim, base <= 1),
 * CASCADE_ERR_CUDA (launch failure).
 */
cascade_status_t cascade_rope_table(int32_t n_positions, int32_t head_dim, double base, float* table,
                                    void* stream);

/*
 * cascade_attn_sharded_rope -- cascade_attn_sharded with the tail of the pre-pass fused in (the Pre-Pass algorithm:
 * q <- rotary_pos_emb(q, p^{R_i}), k <- rotary_pos_emb(k, p^{R_i})): q and k are given UNROTATED; every query row is
 * turned by the table row of its position (q_pos_offset + token index) and every key row by the row of its token
 * index while they are staged for the attention kernel, so no separate pass over q and k runs:
 *   y[i] = x[i] cos - x[i + d/2] sin,   y[i + d/2] = x[i + d/2] cos + x[i] sin,   (cos, sin) = table[pos][i],
 * computed in fp32 and rounded once to bf16, the type the pre-pass would hand q and k on in.  Because a row's angle
 * depends on its original index only, the result equals rotating the whole sequence first and calling
 * cascade_attn_sharded.
 *   rope_table   DEVICE table written by cascade_rope_table for head_dim 128, 16-byte aligned, read-only
 *   n_positions  its row count; must cover max(q_pos_offset + n_q, n_kv)
 * All other arguments, the workspace and the outputs are those of cascade_attn_sharded.
 * Supported on the tensor-core route only (bf16, head_dim 128, n_q > 1, at most 256 KV shards); other shapes return
 * CASCADE_ERR_UNSUPPORTED and the caller rotates q and k beforehand.
 */
cascade_status_t cascade_attn_sharded_rope(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                           int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                           const void* q, cascade_strides_t q_strides, const void* k,
                                           cascade_strides_t k_strides, const void* v,
                                           cascade_strides_t v_strides, const float* rope_table,
                                           int32_t n_positions, void* o_out, cascade_strides_t o_strides,
                                           float* lse_out, void* workspace, size_t workspace_bytes,
                                           void* stream);

/*
 * Shard-map generators and shard-safety measures.  HOST arrays only, integer only, no device work; the maps they
 * write are what cascade_shard_plan takes.  Token indices are 0-based (the paper prints 1-based ones).
 *
 * cascade_cdelta_shard_map -- (c, delta)-sharding (Section 6, definition of a (c, delta)-sequence): sequence i holds
 * the tokens i c .. i c + c - 1 of every period of delta tokens, shard_of[t] = (t mod delta) / c; the number of
 * sequences that covers [N] is alpha = ceil(delta / c), written to *n_shards_out (optional).  If c does not divide
 * delta the last sequence has clusters of delta mod c tokens.
 *   shard_of  HOST int32 [n_tokens], written.   Errors: INVALID_ARG unless 1 <= c <= delta, n_tokens >= 0.
 */
cascade_status_t cascade_cdelta_shard_map(int32_t n_tokens, int32_t c, int32_t delta, int32_t* shard_of,
                                          int32_t* n_shards_out);

/*
 * cascade_msplit_shard_map -- the m-split of AttnNodes (Section 6.4): every hidden shard R_i is cut into m pieces,
 * R_{i,x} taking the members of sorted R_i at ranks x, x + m, x + 2m, ... (the rule the section's worked example
 * with N = 18, c = 2, delta = 6, m = 2 follows), and the query/KV shards are S_{m i + x} = R_{i,x}; beta = m alpha.
 *   r_shard_of  HOST int32 [n_tokens], values in [0, n_r_shards)     s_shard_of  HOST int32 [n_tokens], written
 * Errors: INVALID_ARG (sizes, null arrays), BAD_MAP (an id outside [0, n_r_shards); the message names the token).
 */
cascade_status_t cascade_msplit_shard_map(int32_t n_tokens, const int32_t* r_shard_of, int32_t n_r_shards, int32_t m,
                                          int32_t* s_shard_of);

/*
 * cascade_index_set_gaps -- clusters and gaps of the index set a node holds, or of the union a colluding set of nodes
 * pools (CompNode_i: R_i; AttnNode_jk: S_j u T_k; appendix on collusion).  A cluster is a maximal run of consecutive
 * held indices; the gap between neighbouring clusters is the number of indices strictly between them, i.e. the
 * unknown tokens a generalized vocab-matching attack must enumerate (V^gap candidates).  For a (c, delta)-sequence
 * every gap is delta - c (Section 6.2 states it as the cluster-to-cluster distance delta - c + 1).  Criteria:
 *   Section 6.2 (leakage from the node's own hidden states):  min_gap + 1 >= rho
 *   Theorem of Section 6.3 and the collusion appendix:         min_gap     >= rho
 *   held  HOST uint8 [n_tokens], non-zero = the index is held.
 *   n_indices, n_clusters, min_gap, max_gap: optional outputs; min_gap = max_gap = -1 with fewer than two clusters.
 */
cascade_status_t cascade_index_set_gaps(int32_t n_tokens, const uint8_t* held, int32_t* n_indices,
                                        int32_t* n_clusters, int32_t* min_gap, int32_t* max_gap);

/*
 * cascade_kl_gaps -- the (k, l)-gaps from the proof of the Section 6.3 theorem: for the node's sorted indices
 * r_1 < r_2 < ... and KV shard S_k, gap (k, l) = { s in S_k : r_l < s < r_{l+1} } without the node's own indices.
 * The attack of the proof needs a NON-EMPTY gap with fewer than rho members, so the call reports, per KV shard, the
 * size of the smallest non-empty gap over l (-1 if every gap of that shard is empty).
 *   r_held  HOST uint8 [n_tokens]      s_shard_of  HOST int32 [n_tokens], values in [0, n_s_shards)
 *   min_gap_per_shard  HOST int32 [n_s_shards], written.   Errors: INVALID_ARG, BAD_MAP.
 */
cascade_status_t cascade_kl_gaps(int32_t n_tokens, const uint8_t* r_held, const int32_t* s_shard_of,
                                 int32_t n_s_shards, int32_t* min_gap_per_shard);

/*
 * cascade_attn_sharded_host -- cascade_attn_sharded for callers whose tensors live in HOST memory (the paper's nodes
 * exchange q, k, v and the outputs over a network; here the host side of the PCIe link stands in for it).  The call
 * copies k and v to the device, then works through the KV heads one at a time: the G = n_heads / n_kv_heads query
 * heads of KV head g are uploaded on one copy stream while the fused attention of head g - 1 runs on the caller's
 * stream and the output of head g - 2 travels back on a second copy stream, so the transfers in both directions
 * overlap each other and the compute.  Results are those of cascade_attn_sharded.
 *   q_host, o_host  HOST, dense [batch][n_q][n_heads][head_dim]; k_host, v_host  HOST, dense
 *                   [batch][n_kv][n_kv_heads][head_dim].  Pinned memory is needed for the copies to be asynchronous.
 *   workspace       DEVICE, 256-byte aligned, cascade_workspace_bytes(CASCADE_CALL_SHARDED_HOST) bytes: staging for
 *                   q, k, v, o and the scratch of one head group.  Overwritten by every call.
 * All work is ordered after what `stream` holds at the time of the call, and `stream` waits for the last output
 * copy: synchronising `stream` makes o_host valid.  The first call on a device creates two internal copy streams and
 * their events (no device memory); all calls on a device share them, so calls from several host threads for the same
 * device must be serialised by the caller.  Errors as cascade_attn_sharded, plus CASCADE_ERR_INVALID_ARG for more than 128 KV
 * heads.
 */
cascade_status_t cascade_attn_sharded_host(const cascade_plan_t* plan, cascade_dtype_t dtype, int32_t batch,
                                           int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                           const void* q_host, const void* k_host, const void* v_host,
                                           void* o_host, void* workspace, size_t workspace_bytes, void* stream);

/*
 * cascade_plan_advance -- moves the query block of a plan to a new position: token-sharded KV caching (Appendix F,
 * "Caching").  Under a (c, delta)-style scheme the shard of every future token is known in advance, so a decode loop
 * builds ONE plan over the whole cache capacity (n_kv = capacity, every slot already mapped to its KV shard, n_q = 1)
 * and, for each generated token, writes that token's k and v rows at its index of the caller's cache tensors and
 * calls this function with the token's position: the causal mask (key token <= query position) then admits exactly
 * the cache rows written so far, and the new row belongs to its shard's list without any list being rebuilt.
 * Recomputes VIS and PAIR_CLASS for query position q_pos_offset + token index; the index lists do not change.  On a
 * device plan with more than 256 (query row, KV shard) entries two small kernels rewrite the device arrays in stream
 * order from the plan's own index lists (no host computation, no upload; the host copies that cascade_plan_get and
 * cascade_plan_dense_mask return are brought up to date when they are next asked for).  Smaller plans (a decode
 * step), host-only plans and plans over resident K/V rows (kv_pos) recompute on the host and upload in stream order.  Works for any n_q (a prefill chunk that slides along the sequence);
 * the work-sorted order of the plan's query tiles is left as it was built, which affects speed only.
 * Calls that use the plan before and after must be on `stream` or ordered with it.
 * Cache rows beyond the new position need not be initialised (see cascade_attn_partials); rows at or before it must be
 * written, and finite, before the attention call that follows.
 * Errors: CASCADE_ERR_INVALID_ARG (null plan), CASCADE_ERR_CUDA.
 */
cascade_status_t cascade_plan_advance(cascade_plan_t* plan, int32_t q_pos_offset, void* stream);

/*
 * cascade_attn_decode_static -- the decode case of cascade_attn_sharded (one query row per sequence, bf16,
 * head_dim 128, n_heads / n_kv_heads in {1,2,4,8}) without a workspace argument and without any allocation.
 * (The paper has no counterpart: this is a convenience of this library, not a step of the method.)
 *
 * Who it is for: callers that cannot hand over scratch memory and cannot allocate it either -- a server whose
 * cache manager already owns all free HBM, a decode loop that must not hit the device-wide synchronisation of
 * cudaMalloc / cudaFree, a plug-in that only receives raw pointers.  The per-shard partials that the merge
 * kernel combines live in a 16 MiB array compiled into the library (every GPU that loads the library carries
 * it until the process exits).  The call issues no cudaMalloc, cudaFree or other allocating routine.
 *
 *  - Limit: batch * n_kv_shards * n_heads * 264 bytes (rounded up per region to 256) must fit in 16 MiB,
 *    e.g. batch 64 x 16 shards x 32 heads = 8.3 MiB.  Larger problems return CASCADE_ERR_WORKSPACE with a
 *    message naming the sizes; use cascade_attn_sharded with a workspace for those.
 *  - The first call on each device looks up the array's device address (the device current at that moment).
 *    Make that first call during start-up, before any stream capture.
 *  - All calls share the one array.  Its contents are overwritten completely by each call before they are read,
 *    so results never depend on an earlier call; but two calls whose kernels overlap on the GPU (different
 *    streams, no ordering between them) race on it.  Keep calls on one stream or order them with events.
 *  - Inputs, outputs, strides, stream and results are exactly those of cascade_attn_sharded.
 */
cascade_status_t cascade_attn_decode_static(const cascade_plan_t* plan, int32_t batch, int32_t n_heads,
                                            int32_t n_kv_heads, float scale, const void* q,
                                            cascade_strides_t q_strides, const void* k,
                                            cascade_strides_t k_strides, const void* v,
                                            cascade_strides_t v_strides, void* o_out, cascade_strides_t o_strides,
                                            float* lse_out, void* stream);

/*
 * cascade_rope_apply -- the rotary steps of the Pre-Pass algorithm (q <- rotary_pos_emb(q, p^{R_i}), the same for k) as
 * a pass of its own, for rows that no fused call covers (fp32, head_dim 64, rows rotated once and then cached):
 *   y[b][r][h][i]       = x[..][i] cos - x[..][i + d/2] sin
 *   y[b][r][h][i + d/2] = x[..][i + d/2] cos + x[..][i] sin,      (cos, sin) = table[first_position + r][i]
 * in fp32, rounded once to `dtype`.  Row r of every sequence sits at position first_position + r.
 *   x, y         DEVICE [batch][n_rows][n_heads][head_dim] with strides (y may be x: in place); head_dim 64 or 128
 *   rope_table   DEVICE table of cascade_rope_table for this head_dim; n_positions its row count
 * Errors: INVALID_ARG (null, misaligned, positions outside the table), UNSUPPORTED (dtype, head_dim), CUDA.
 */
cascade_status_t cascade_rope_apply(cascade_dtype_t dtype, int32_t batch, int32_t n_rows, int32_t n_heads,
                                    int32_t head_dim, const void* x, cascade_strides_t x_strides,
                                    int32_t first_position, const float* rope_table, int32_t n_positions, void* y,
                                    cascade_strides_t y_strides, void* stream);

/*
 * cascade_decode_step_rope -- one generated token against a token-sharded KV cache ("Caching" in the appendix on cost
 * optimizations), with the tail of the Pre-Pass algorithm folded in: given the new token's UNROTATED q, k, v rows
 *   1. moves the plan's query block to `position` (cascade_plan_advance: the mask admits cache rows <= position),
 *   2. rotates the k row by the table row of `position` and writes it, and the v row as it is, at row `position` of the
 *      caches -- the node that holds the token's KV shard appends it; rows already cached are not touched again,
 *   3. rotates the q row and runs the decode route of cascade_attn_sharded on the caches (one partial per KV shard,
 *      then the post-pass combine).
 *   plan            built by cascade_shard_plan over the cache CAPACITY with n_q = 1 (see cascade_plan_advance)
 *   q_new           DEVICE bf16 [batch][1][n_heads][128];  k_new, v_new  DEVICE bf16 [batch][1][n_kv_heads][128]
 *   k_cache, v_cache  DEVICE bf16 [batch][capacity][n_kv_heads][128] with strides; row `position` is WRITTEN
 *   rope_table      DEVICE table of cascade_rope_table for head_dim 128 with more than `position` rows
 *   o_out, lse_out  as cascade_attn_sharded (one row per sequence)
 *   workspace       cascade_workspace_bytes(CASCADE_CALL_DECODE_STEP_ROPE) bytes
 * bf16, head_dim 128, n_heads / n_kv_heads in {1, 2, 4, 8}.  Errors as cascade_attn_sharded and cascade_plan_advance.
 */
cascade_status_t cascade_decode_step_rope(cascade_plan_t* plan, int32_t batch, int32_t n_heads, int32_t n_kv_heads,
                                          float scale, const void* q_new, cascade_strides_t q_strides,
                                          const void* k_new, cascade_strides_t k_new_strides, const void* v_new,
                                          cascade_strides_t v_new_strides, void* k_cache,
                                          cascade_strides_t k_cache_strides, void* v_cache,
                                          cascade_strides_t v_cache_strides, int32_t position, const float* rope_table,
                                          int32_t n_positions, void* o_out, cascade_strides_t o_strides, float* lse_out,
                                          void* workspace, size_t workspace_bytes, void* stream);

enum {
  CASCADE_CALL_PARTIALS = 0,
  CASCADE_CALL_SHARDED = 1,
  CASCADE_CALL_SHARDED_HOST = 2,
  CASCADE_CALL_DECODE_STEP_ROPE = 3
};

/* Scratch bytes the given call needs for this plan and shape (0 if none).  The workspace must be
 * 256-byte aligned. */
cascade_status_t cascade_workspace_bytes(const cascade_plan_t* plan, int32_t which_call,
                                         cascade_dtype_t dtype, int32_t batch, int32_t n_heads,
                                         int32_t n_kv_heads, int32_t head_dim, size_t* out_bytes);

#ifdef __cplusplus
}
#endif
#endif /* CASCADE_H_ */
