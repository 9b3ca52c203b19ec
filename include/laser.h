/*
 * laser.h - C ABI of the B200-native Draft-Then-Verify decoding loop of LASER
 * (arXiv 2408.05676): retrieval-based drafting from per-group token pools, one
 * target-model verify forward over [pending token + drafts], strict / relaxed
 * acceptance, KV-cache commit, and the generation loop that chains them.
 *
 * Conventions
 *  - Every function returns a laser_status; 0 is success, negatives are errors.
 *    laser_last_error() gives a thread-local message for the last failure.  There are
 *    no exceptions, no abort(), no device traps; arguments are validated on the host
 *    before any launch.
 *  - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are
 *    ordinary host memory.  The library neither frees nor keeps caller arrays past the
 *    call, except the weight pointers given to laser_model_create(), which are borrowed
 *    for the model's lifetime.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *    enqueued on it and is asynchronous unless stated otherwise; outputs are valid once
 *    the stream has been synchronised.
 *  - Opaque handles (laser_pool, laser_model, laser_kv) are owned by the library and
 *    released by the matching *_free call.
 *  - Per-sequence step arrays use a fixed row stride of K+1: slot 0 is the pending
 *    (not yet cached) token x_t, slots 1..m the drafts.  Unused slots hold -1.
 *  - The library keeps lazily grown scratch buffers per device; calls that overlap
 *    on the GPU from different streams must not share a device.
 */
#ifndef LASER_H_
#define LASER_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t laser_status;
enum {
  LASER_OK = 0,
  LASER_ERR_INVALID_ARG = -1,
  LASER_ERR_OOM = -2,
  LASER_ERR_CUDA = -3,
  LASER_ERR_CAPACITY = -4,   /* KV pages exhausted, K above the compiled maximum, ...   */
  LASER_ERR_TIMEOUT = -5,    /* a bounded device-side wait ran out                        */
  LASER_ERR_UNSUPPORTED = -6
};

/* Acceptance rules (Section 3.4 and the ablation of Section 4.3.2). */
enum {
  LASER_MODE_STRICT = 0,   /* Eq. 4: draft == arg max q_i                                  */
  LASER_MODE_RELAXED = 1,  /* Eq. 8: draft in TopK(q_i, k) and q_i(draft) > p              */
  LASER_MODE_TOPK = 2,     /* Eq. 7 alone                                                  */
  LASER_MODE_TOPP = 3,     /* draft == arg max q_i, or q_i(draft) > p                      */
  LASER_MODE_RELAXED_ARGMAX = 4  /* draft == arg max q_i, or Eq. 8: Eq. 8 with the arg-max always
                              accepted ("highest probability or", Section 4.3.2); accepts whatever
                              STRICT or RELAXED accepts                                    */
};

typedef struct laser_pool laser_pool;
typedef struct laser_model laser_model;
typedef struct laser_kv laser_kv;

/* Llama-style decoder shape.  max_batch * (max_draft + 1) bounds the rows of one step. */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int32_t page_size;   /* tokens per KV page; must be 16                                   */
  int32_t max_draft;   /* K: row stride of a step is max_draft + 1                         */
  int32_t max_batch;   /* most sequences in one laser_verify_step call                     */
  int32_t precise;     /* non-zero: every activation that enters a matrix product (the attention's
                          queries and probabilities included) is carried as a pair of bf16 values,
                          hi + lo, about 16 significant bits; weights and cache stay bf16, sums fp32.
                          Logits then lie within 2e-2 of an exact forward at the 7B depth (0.006
                          measured); about 1.5 x the step time (each weight block is multiplied twice) */
} laser_model_cfg;

/* bf16 device pointers, matrices row-major [out_features, in_features] and 16-byte aligned,
 * norm gains 8-byte aligned (laser_model_create returns INVALID_ARG otherwise).  The per-layer
 * members are host arrays of n_layers device pointers. */
typedef struct {
  const void* tok_emb;     /* [vocab, d_model]                                             */
  const void* lm_head;     /* [vocab, d_model]                                             */
  const void* final_norm;  /* [d_model]                                                    */
  const void* const* wq;   /* [n_heads*head_dim, d_model]                                  */
  const void* const* wk;   /* [n_kv_heads*head_dim, d_model]                               */
  const void* const* wv;   /* [n_kv_heads*head_dim, d_model]                               */
  const void* const* wo;   /* [d_model, n_heads*head_dim]                                  */
  const void* const* w_gate; /* [d_ffn, d_model]                                           */
  const void* const* w_up;   /* [d_ffn, d_model]                                           */
  const void* const* w_down; /* [d_model, d_ffn]                                           */
  const void* const* attn_norm; /* [d_model]                                               */
  const void* const* ffn_norm;  /* [d_model]                                               */
} laser_weights;

typedef struct {
  /* drafting (Section 3.3) */
  int32_t K;          /* maximum draft length                                              */
  int32_t n_min;      /* shortest suffix tried                                             */
  int32_t n_max;      /* longest suffix tried first                                        */
  int32_t min_draft;  /* keep shrinking n while the draft is shorter than this (>= 1)      */
  int32_t max_occ;    /* use only the first max_occ occurrences by position; 0 = all       */
  /* acceptance (Section 3.4; the paper's defaults are topk = 2, p = 0.1) */
  int32_t mode;       /* LASER_MODE_*                                                      */
  int32_t topk;
  float p;            /* widened to fp64 for the comparison q > p                          */
  /* generation loop */
  int32_t max_new;    /* tokens to generate per sequence                                   */
  int32_t eos_id;     /* stop after emitting this token; -1 = none                         */
  int32_t temp_branches; /* laser_generate: non-zero = also draft from the sequence's own prompt and
                            generated tokens (temporary branch, Section 3.2; needs max_occ in 1..64) */
  int32_t tree;          /* laser_generate: non-zero = draft a token tree and verify it with tree
                            attention (Section 3.3; needs K <= 32 and max_occ in 1..64)            */
  int32_t fused_accept;  /* laser_generate: non-zero = chain steps run laser_verify_accept (no logits
                            are stored); ignored for token trees                                  */
} laser_params;

typedef struct {
  int64_t steps;      /* decoding steps summed over sequences                              */
  int64_t drafted;    /* draft tokens proposed                                             */
  int64_t accepted;   /* draft tokens accepted (sum of n_accept)                           */
  int64_t emitted;    /* tokens written to the output                                      */
  int64_t launches;   /* kernels launched                                                  */
  int64_t verify_calls; /* batched verify forwards after the prefill                       */
  float ms_prefill, ms_draft, ms_verify, ms_accept, ms_total;
} laser_stats;

const char* laser_version(void);
const char* laser_last_error(void);
/* Kernels launched by this process through the library so far. */
int64_t laser_launch_count(void);

/* ---- Customized Retrieval Pool (Section 3.2) ------------------------------------------
 * Builds the device index of one pool: for every group and every n in [n_min, n_max], a
 * hash from the n-gram to the ascending list of positions where it ends.  This returns
 * what the per-group trie of Section 3.2 returns for a prefix lookup (all continuations
 * of all occurrences, with multiplicity).
 *   tokens         host or dev int32[n_tokens]; -1 separates documents, other ids >= 0
 *   group_offsets  host int64[n_groups+1], ascending, [0] = 0, [n_groups] = n_tokens
 * The pool keeps its own device copy of the tokens.  Synchronous (returns when built).
 * Errors: INVALID_ARG for bad sizes/offsets, OOM, CUDA. */
laser_status laser_pool_build(const int32_t* tokens, int64_t n_tokens,
                              const int64_t* group_offsets, int32_t n_groups,
                              int32_t n_min, int32_t n_max, void* stream, laser_pool** out);
laser_status laser_pool_free(laser_pool* pool);
/* Host-side facts: tokens, distinct (group, n-gram) keys over all n, device bytes held. */
laser_status laser_pool_info(const laser_pool* pool, int64_t* n_tokens, int64_t* n_keys,
                             int64_t* device_bytes);

/* ---- Draft retrieval: Retrieve(D, tail, K), Eq. 5 (Section 3.3) ------------------------
 * For each sequence b: for n = min(n_max, tail_len[b]) down to n_min, take the positions
 * where the last n tail tokens occur in group group_id[b] (first max_occ of them if
 * max_occ > 0), and follow the most frequent next token (ties: smallest id) for up to K
 * steps without leaving the document.  The first n whose draft has >= min_draft tokens
 * wins, else the longest draft (ties: larger n).
 *   tails      dev int32[B, n_max], right-aligned: column n_max-1 is the newest token
 *   tail_len   dev int32[B], 0..n_max
 *   group_id   dev int32[B]
 *   draft      dev int32[B, K] out, padded with -1
 *   draft_len  dev int32[B] out;  match_n dev int32[B] out (0 when the draft is empty)
 * p->n_min/n_max must lie inside the range the pool was built for.
 * Errors: INVALID_ARG (K < 1, K > 64, n range), UNSUPPORTED (vocabulary too large for the
 * unlimited-occurrence path). */
laser_status laser_draft(const laser_pool* pool, const int32_t* tails, const int32_t* tail_len,
                         const int32_t* group_id, int32_t B, const laser_params* p,
                         int32_t* draft, int32_t* draft_len, int32_t* match_n, void* stream);

/* ---- Draft retrieval with temporary branches (Section 3.2) ---------------------------------
 * While a text is generated, its prompt and the tokens generated so far belong to the trie as
 * a temporary branch and leave it when the generation ends.  Same retrieval as laser_draft,
 * with the sequence's own text searched as one more document: its occurrences of the tail that
 * still have a following token come first (ascending), the group's follow (ascending), and the
 * list is cut to p->max_occ, which must lie in 1..64 here; the frequencies of both add up.
 *   hist      dev int32[B, hist_stride]: row b holds the sequence's text, oldest first, ids >= 0
 *             (normally it ends with the tail)
 *   hist_len  dev int32[B], 0..hist_stride
 * group_id[b] outside the pool's groups searches the history alone.  Nothing is stored in the
 * pool: the branch lasts as long as the caller keeps passing the buffer.
 * Errors: as laser_draft; INVALID_ARG also for max_occ outside 1..64. */
laser_status laser_draft_temp(const laser_pool* pool, const int32_t* tails, const int32_t* tail_len,
                              const int32_t* group_id, const int32_t* hist, const int32_t* hist_len,
                              int64_t hist_stride, int32_t B, const laser_params* p,
                              int32_t* draft, int32_t* draft_len, int32_t* match_n, void* stream);

/* ---- Tree-based drafting: T_t = Retrieve(D, tail, K) as a token tree (Section 3.3) -------------
 * The sub-tree of the group's trie under the matched tail: a node is a sequence of continuation
 * tokens, its frequency the number of occurrences of the tail followed by that sequence inside
 * one document.  When the sub-tree has more than K nodes the K most frequent are kept (ties: the
 * shallower node, then the smaller token path), which keeps every kept node's parent.  The kept
 * nodes are listed depth-first, children by (frequency descending, token id ascending): the
 * pseudo-sequence S_t.  Its first branch is what laser_draft would return, as far as it is kept.
 * The suffix length n shrinks from n_max as in laser_draft (a tree counts by its nodes).
 *   hist, hist_len, hist_stride   temporary branch as in laser_draft_temp, or null / null / 0
 *   draft          dev int32[B, K] out: node tokens in depth-first order, padded with -1
 *   draft_parents  dev int32[B, K] out: row of each node's parent, where row 0 is the root (the
 *                  pending token) and node j is row j + 1; padded with -1
 *   draft_len      dev int32[B] out: nodes;  match_n dev int32[B] out
 * Occurrences: the first p->max_occ (1..64), the history's first.
 * Errors: INVALID_ARG (K outside 1..32, max_occ outside 1..64, n range). */
laser_status laser_draft_tree(const laser_pool* pool, const int32_t* tails, const int32_t* tail_len,
                              const int32_t* group_id, const int32_t* hist, const int32_t* hist_len,
                              int64_t hist_stride, int32_t B, const laser_params* p, int32_t* draft,
                              int32_t* draft_parents, int32_t* draft_len, int32_t* match_n, void* stream);

/* Rows of a tree step: laser_make_rows plus parents[b,0] = -1, parents[b,1+j] = draft_parents[b,j]
 * for j < draft_len[b], rest -1 (the layout laser_verify_step_tree and laser_accept_tree read). */
laser_status laser_make_rows_tree(const int32_t* last_token, const int32_t* draft,
                                  const int32_t* draft_parents, const int32_t* draft_len, int32_t B,
                                  int32_t K, int32_t* tokens, int32_t* parents, int32_t* n_rows,
                                  void* stream);

/* Builds the verify rows from the drafts: tokens[b,0] = last_token[b],
 * tokens[b,1..] = draft[b,:draft_len[b]], rest -1; n_rows[b] = 1 + draft_len[b], or 0
 * where last_token[b] < 0 (inactive slot).  All dev; tokens is [B, K+1]. */
laser_status laser_make_rows(const int32_t* last_token, const int32_t* draft,
                             const int32_t* draft_len, int32_t B, int32_t K,
                             int32_t* tokens, int32_t* n_rows, void* stream);

/* ---- Target model and paged KV cache --------------------------------------------------- */
laser_status laser_model_create(const laser_model_cfg* cfg, const laser_weights* w,
                                laser_model** out);
laser_status laser_model_free(laser_model* m);

/* Cache of n_pages pages of 16 tokens, bf16, for up to max_seqs sequences.  Sequence s
 * initially owns pages_per_seq = n_pages / max_seqs pages, interleaved (logical page j of
 * sequence s is physical page j * max_seqs + s). */
laser_status laser_kv_create(const laser_model* m, int32_t max_seqs, int64_t n_pages,
                             laser_kv** out);
laser_status laser_kv_free(laser_kv* kv);
/* host int32[max_seqs * pages_per_seq]: physical page of each logical page; every entry
 * must be unique and < n_pages.  Synchronous. */
laser_status laser_kv_set_page_table(laser_kv* kv, const int32_t* table);
/* Committed length (tokens whose K/V are valid) of each listed sequence.  Host arrays;
 * both calls synchronise `stream`. */
laser_status laser_kv_set_len(laser_kv* kv, const int32_t* seq_ids, const int32_t* lens,
                              int32_t n, void* stream);
laser_status laser_kv_get_len(const laser_kv* kv, const int32_t* seq_ids, int32_t* lens,
                              int32_t n, void* stream);
/* Forgets every sequence of the cache: all committed lengths become 0 (the pages keep their
 * contents, which are no longer valid).  Asynchronous on `stream`. */
laser_status laser_kv_reset(laser_kv* kv, void* stream);
/* Same as laser_kv_set_len for slots 0..n-1 with a dev int32[n] source; asynchronous. */
laser_status laser_kv_set_len_dev(laser_kv* kv, const int32_t* lens_dev, int32_t n, void* stream);
/* Copy K and V of one layer for token positions [pos0, pos0+n) of one sequence between the
 * pages and contiguous dev bf16 arrays [n, n_kv_heads*head_dim]. */
laser_status laser_kv_import(laser_kv* kv, int32_t seq, int32_t layer, int32_t pos0, int32_t n,
                             const void* k, const void* v, void* stream);
laser_status laser_kv_export(const laser_kv* kv, int32_t seq, int32_t layer, int32_t pos0,
                             int32_t n, void* k, void* v, void* stream);

/* ---- Verify forward: q_i = M(x_<=t, x~_<i), i = 1..K+1, Eq. 3 / Eq. 6 -------------------
 * One forward of the decoder over the rows of B sequences.  Row i of sequence b is
 * tokens[b,i] at position len_b + i; it attends to the len_b cached tokens and to rows
 * 0..i of the same call (the chain form of the mask and position ids of Section 3.3).
 * K and V of every row are written to the cache at positions len_b .. len_b+n_rows-1; the
 * committed length is not changed.  bf16 operands, fp32 accumulation and residual stream.
 *   seq_ids  dev int32[B] distinct cache slots;  tokens dev int32[B, K+1];
 *   n_rows   dev int32[B], 0..K+1 (0 = inactive);  logits dev fp32[B, K+1, vocab] out
 * with K = cfg.max_draft.  Rows >= n_rows[b] are left unspecified.  logits must be 16-byte aligned.
 * Errors: INVALID_ARG (B > max_batch, misaligned logits), CAPACITY (a sequence would outgrow its pages: found
 * on the device, the rows are then not cached, and laser_check() reports it). */
laser_status laser_verify_step(laser_model* m, laser_kv* kv, const int32_t* seq_ids,
                               const int32_t* tokens, const int32_t* n_rows, int32_t B,
                               float* logits, void* stream);

/* ---- Verify forward of a token tree (Section 3.3, tree attention) ------------------------------
 * As laser_verify_step, for a pseudo-sequence that lists a token tree in depth-first order.
 *   parents  dev int32[B, K+1]: parents[b,i] = row of row i's parent, 0 <= parents[b,i] < i for
 *            i >= 1; entry [b,0] is not read (row 0, the pending token, is the root)
 * Row i takes the position ctx + depth(i) (P_t), attends to the cache and to its ancestors and
 * itself (M_t), and its K and V are written to cache slot ctx + i: after acceptance the
 * accepted path is moved to consecutive slots (laser_accept_tree, laser_kv_compact_path).
 * A chain given as parents[b,i] = i - 1 gives laser_verify_step's result.
 * Errors: as laser_verify_step; INVALID_ARG when K + 1 > 64 or (reported by laser_check) when
 * a parent is not an earlier row. */
laser_status laser_verify_step_tree(laser_model* m, laser_kv* kv, const int32_t* seq_ids,
                                    const int32_t* tokens, const int32_t* parents,
                                    const int32_t* n_rows, int32_t B, float* logits, void* stream);
/* Synchronises `stream` and returns the first device-side error recorded since the last
 * check (CAPACITY, TIMEOUT), clearing it. */
laser_status laser_check(laser_model* m, void* stream);

/* Measurement aid for the forward of Eq. 3: while enabled, every dense-contraction launch
 * (class 0) and every attention launch (class 1) of laser_verify_step is bracketed by CUDA
 * events on the call's stream.  laser_profile_read synchronises the device and returns the
 * summed device time and the number of launches of one class since the previous read. */
laser_status laser_profile_enable(laser_model* m, int32_t on);
laser_status laser_profile_read(laser_model* m, int32_t cls, double* ms, int64_t* launches);

/* ---- Acceptance and commit (Section 2.1, Section 3.4, Eq. 4 / Eq. 7 / Eq. 8) ------------
 * Drafts are verified in order against rows 0.. of the logits; n_accept[b] = drafts that
 * pass before the first failure; out_tokens[b] = those drafts followed by arg max of row
 * n_accept[b] (correction or bonus token); n_out[b] = n_accept[b] + 1.  Ties between equal
 * logits rank the smaller id first; probabilities are softmax at temperature 1 evaluated
 * in fp64.  If kv != NULL the committed length of seq_ids[b] grows by n_out[b].
 *   logits dev fp32[B, K+1, V];  tokens dev int32[B, K+1];  n_rows dev int32[B];
 *   n_accept, n_out dev int32[B] out;  out_tokens dev int32[B, K+1] out (padded -1)
 * with K = p->K.  Sequences with n_rows[b] == 0 give n_accept = n_out = 0. */
laser_status laser_accept_commit(laser_kv* kv, const int32_t* seq_ids, const float* logits,
                                 const int32_t* tokens, const int32_t* n_rows, int32_t B,
                                 int32_t V, const laser_params* p, int32_t* n_accept,
                                 int32_t* out_tokens, int32_t* n_out, void* stream);

/* ---- Verification of a token tree (Section 3.4, tree verification: the children of a rejected
 * node are not examined, and of all verified nodes the deepest one fixes the accepted path) ------
 * tokens / parents / n_rows as for laser_verify_step_tree, logits its result.  Node i is verified
 * when its parent is (row 0 always is) and tokens[b,i] passes p->mode on the row of its parent.
 * The verified node of greatest depth wins, the first in depth-first order among equals.
 *   n_accept    dev int32[B]       depth of the winner = accepted drafts a
 *   out_tokens  dev int32[B, K+1]  the a tokens of its path, then arg max of its own row, then -1
 *   n_out       dev int32[B]       a + 1 (0 for an inactive sequence)
 *   path_rows   dev int32[B, K+1]  rows of the accepted path, root excluded, then -1
 * kv non-null: the K and V of the accepted rows move from cache slot len + row to len + 1 .. len + a
 * and the lengths advance by n_out (laser_kv_compact_path, then the update).  kv null: verdict only.
 * Errors: INVALID_ARG (K + 1 > 64, mode, topk), OOM, CUDA. */
laser_status laser_accept_tree(laser_kv* kv, const int32_t* seq_ids, const float* logits,
                               const int32_t* tokens, const int32_t* parents, const int32_t* n_rows,
                               int32_t B, int32_t V, const laser_params* p, int32_t* n_accept,
                               int32_t* out_tokens, int32_t* n_out, int32_t* path_rows, void* stream);

/* Cache compaction after tree verification (Section 3.3: the rows of a tree are not consecutive
 * positions).  For sequence seq_ids[b] with committed length len: slot len + path_rows[b,j] is
 * copied to slot len + j + 1 for j = 0 .. n_accept[b]-1, in every layer, K and V.  path_rows is
 * [B, row_stride], rows ascending (as laser_accept_tree writes them).  Lengths are not changed. */
laser_status laser_kv_compact_path(laser_kv* kv, const int32_t* seq_ids, const int32_t* path_rows,
                                   const int32_t* n_accept, int32_t B, int32_t row_stride, void* stream);

/* Same result as laser_accept_commit, for callers that must not allocate device memory.
 * (The paper has no counterpart; this exists for integration.)  Some hosts of this library
 * cannot call cudaMalloc on the decoding path: a serving engine that reserved all of HBM for
 * its own pools at start-up has nothing left for the driver to hand out, and an allocation
 * in the middle of a step would also stall every stream of the device while the driver
 * serves it.  laser_accept_commit keeps its per-row verdicts in a lazily grown scratch
 * buffer; this variant keeps them in a fixed 132 KB array that is part of the library image
 * on every GPU that loads it, and itself calls no allocating routine.
 *   Limits: B <= 1024 sequences and B * (K+1) <= 16384 rows; larger calls return
 *   LASER_ERR_CAPACITY and launch nothing.
 *   The first call on each device looks up the array's device address (the device must be
 *   current).  With lazy module loading that look-up, or the first launch, is also when the
 *   CUDA runtime loads this part of the library onto the device (the kernel image and the
 *   132 KB array), which needs driver memory: make the first call at start-up, before the
 *   host reserves the rest of HBM and before starting any stream capture.  Later calls touch
 *   no allocator.  The look-up is serialised between host threads.
 *   All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 *   (different streams) race on it and give undefined results.  Serialise them. */
laser_status laser_accept_commit_noalloc(laser_kv* kv, const int32_t* seq_ids, const float* logits,
                                         const int32_t* tokens, const int32_t* n_rows, int32_t B,
                                         int32_t V, const laser_params* p, int32_t* n_accept,
                                         int32_t* out_tokens, int32_t* n_out, void* stream);

/* ---- Verify forward with fused acceptance (Section 3.4; Eq. 4, Eq. 7, Eq. 8) -------------
 * laser_verify_step followed by laser_accept_commit as one call in which the [B, K+1, vocab]
 * logits are never stored: the LM head's epilogue keeps, per row and 128-token vocabulary tile,
 * the tile's largest logits with their ids, the tile's sum of exp(l - tile max) and the logit
 * of the row's draft token, and a small second kernel finishes the rule from those.
 *   Arguments as for the two calls (p->K must equal the model's max_draft); commit != 0 advances
 *   the cache lengths by n_out as laser_accept_commit does with a cache.
 *   logits  dev fp32 [B, K+1, vocab] or NULL.  When given (16-byte aligned), the same launch also
 *           stores the logits it decided on, so that the verdicts can be checked against the rule
 *           applied to stored logits; NULL is the form meant for decoding.
 *   The arg max, the rank test (Eq. 7) and so STRICT and TOPK are exact: identical to
 *   laser_accept_commit on the stored logits.  Probabilities are combined in fp64 from per-tile
 *   fp32 sums and agree with the two-pass rule to a few 1e-6 relative, so a RELAXED / TOPP /
 *   RELAXED_ARGMAX verdict can differ only where the draft's probability lies within that distance
 *   of p.  Rules that rank need topk <= 4 (four logits are kept per tile): UNSUPPORTED otherwise.
 * Asynchronous on `stream`.  Errors: as laser_verify_step, and INVALID_ARG / UNSUPPORTED above. */
laser_status laser_verify_accept(laser_model* m, laser_kv* kv, const int32_t* seq_ids,
                                 const int32_t* tokens, const int32_t* n_rows, int32_t B,
                                 const laser_params* p, int32_t commit, float* logits,
                                 int32_t* n_accept, int32_t* out_tokens, int32_t* n_out, void* stream);

/* Self-test of the library's failure path (the paper has no counterpart).  Every wait inside the
 * TMA-fed kernels is bounded; when one runs out the kernel stops waiting, lets its copies in flight
 * land, records LASER_ERR_TIMEOUT in the model's status word and returns, and the context stays
 * usable.  This call runs that path on purpose without harming anything: one small kernel waits on
 * a barrier nobody arrives on, for at most limit_cycles clock cycles (1e3 .. 2e9), while a second
 * role of the same kernel drains one bulk copy.  Afterwards laser_check() returns
 * LASER_ERR_TIMEOUT once (and clears it), and the model works as before.
 *   report  dev int32[4] out: [0] the starved wait gave up, [1] the abort flag reached the
 *           producer role, [2] the producer saw its copy land, [3] cycles the wait took.
 * Asynchronous on `stream`.  Errors: INVALID_ARG. */
laser_status laser_selftest_wait(laser_model* m, int64_t limit_cycles, int32_t* report, void* stream);

/* ---- Grouping (Section 3.2, Collaborative-based Grouping) ------------------------------
 * K-means over embeddings (Lloyd's iteration): the clustering by which the paper assigns users
 * and items to the groups that each own a retrieval pool.  `iters` times: every point goes to its
 * nearest centroid (squared Euclidean distance in fp32, ties to the smaller index), then every
 * centroid becomes the mean of its points (a cluster without points keeps its centroid).
 *   x dev fp32 [n, dim] row-major (dim <= 256); centroids dev fp32 [k, dim]: in = the starting
 *   centroids, out = the final ones; assign dev int32[n] out: the assignment of the last
 *   iteration (the group id of each point); counts dev int32[k] out: points per cluster in it.
 * Assignments are identical from run to run for given centroids; the means are summed with
 * atomics, so centroids agree between runs to fp32 summation accuracy.  Asynchronous on `stream`.
 * Errors: INVALID_ARG (null pointer, sizes out of range, k * dim beyond shared memory), OOM. */
laser_status laser_group_kmeans(const float* x, int64_t n, int32_t dim, int32_t k, int32_t iters,
                                float* centroids, int32_t* assign, int32_t* counts, void* stream);

/* ---- Generation loop (Section 2.1 / Section 3) ----------------------------------------
 * Prefills each prompt except its last token, then repeats draft -> verify -> accept ->
 * commit until every sequence has max_new tokens (the last step is truncated) or has
 * emitted eos_id.  pool may be NULL: plain greedy autoregressive decoding (Eq. 1).
 *   prompts host int32 (concatenated), prompt_offsets host int64[B+1], group_id host
 *   int32[B];  out host int32[B, max_new] (padded -1), out_len host int32[B];
 *   stats may be NULL.  Uses cache slots 0..B-1 and resets their length.  Synchronous. */
laser_status laser_generate(laser_model* m, laser_kv* kv, const laser_pool* pool,
                            const int32_t* prompts, const int64_t* prompt_offsets,
                            const int32_t* group_id, int32_t B, const laser_params* p,
                            int32_t* out, int32_t* out_len, laser_stats* stats, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LASER_H_ */
