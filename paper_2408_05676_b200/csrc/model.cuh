// Internal definition of the model handle and of the GEMM entry used by the verify forward.
#pragma once
#include <vector>

#include "state.cuh"

struct laser_model {
  laser_model_cfg cfg{};
  int rows_per_seq = 0;  // max_draft + 1
  int R = 0;             // max_batch * rows_per_seq
  int R_pad = 0;         // R rounded up to a multiple of 16
  int dq = 0, dkv = 0, dqkv = 0;
  const __nv_bfloat16 *tok_emb = nullptr, *lm_head = nullptr, *final_norm = nullptr;
  std::vector<const __nv_bfloat16*> wqkv, wo, wgu, wdown, attn_norm, ffn_norm;
  std::vector<void*> owned;  // device allocations released with the model
  // workspace (all device)
  float* resid = nullptr;          // [R_pad, d] residual stream, fp32
  __nv_bfloat16* xn = nullptr;     // [R_pad, d] normalised activations (GEMM operand)
  __nv_bfloat16* q = nullptr;      // [R_pad, dq] rotated queries
  float* qf = nullptr;             // [R_pad, dq] the same in fp32 (precise mode only)
  bool precise = false;            // activations handed to the contractions as hi + lo bf16 pairs: xn, attn, act are
                                   // [R_pad, 2 x width] with the lo parts in the second half of a row
  __nv_bfloat16* attn = nullptr;   // [R_pad, dq] attention output
  __nv_bfloat16* act = nullptr;    // [R_pad, f] SwiGLU output
  float* sumsq = nullptr;          // [ceil(d/128)][R_pad] per-tile sums of squares of the residual
  float* rope = nullptr;           // [R_pad, head_dim/2, 2] cos, sin of each row's position
  int32_t* row_pos = nullptr;      // [R_pad] position of the row, -1 = inactive
  int32_t* row_seq = nullptr;      // [R_pad] cache slot of the row
  int32_t* row_ctx = nullptr;      // [max_batch] committed length of each sequence of the step
  int32_t* row_n = nullptr;        // [max_batch] effective rows of each sequence
  unsigned long long* row_mask = nullptr;  // [R_pad] token tree: rows of its sequence a row attends to (bit j = row j)
  // acceptance fused into the LM head: what its epilogue leaves per (row, 128-token vocabulary tile)
  int32_t* row_draft = nullptr;    // [R_pad] token whose verdict the row gives, -1 = none
  float* draft_logit = nullptr;    // [R_pad] logit of that token
  float4* top_val = nullptr;       // [R_pad][vocab tiles] the tile's four largest logits, in order
  int4* top_idx = nullptr;         // [R_pad][vocab tiles] their token ids
  float* tile_sum = nullptr;       // [R_pad][vocab tiles] sum over the tile of exp(l - tile max)
  int32_t* status = nullptr;       // first device-side error of the stream, 0 = none
  void* gemm_state = nullptr;      // tensor-map cache of the tensor-core GEMM
  void* gen_buf = nullptr;         // work buffers of laser_generate, kept between calls (in `owned`)
  size_t gen_bytes = 0;
  // optional per-class kernel timing (class 0 = GEMM, 1 = attention)
  bool profile = false;
  std::vector<cudaEvent_t> prof_events[2];  // begin/end pairs
  size_t prof_used[2] = {0, 0};
};

namespace laser {

// What the GEMM does with a finished 128-feature x NT-row accumulator tile.
enum { EPI_PLAIN = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_QKV = 3, EPI_VERDICT = 4 };

struct GemmEpilogue {
  int R_rows = 0;                    // rows the activation / output buffers really have
  // Operands as hi + lo bf16 pairs (the precise mode): the A operand's rows are [hi | lo] with lo starting at column
  // a_lo_off (0 = plain bf16 operand); out_split = the bf16 activations this epilogue writes (xb, act) are pairs too
  int a_lo_off = 0, out_split = 0;
  // RMSNorm of the A operand, applied as a per-row scale of the result: the producer left
  // x * gain in bf16 and one sum of squares per (128-feature tile, row); null = no scale
  const float* sumsq_in = nullptr;
  int sumsq_in_tiles = 0, sumsq_ld = 0;
  float inv_d = 0.f, eps = 0.f;
  // EPI_PLAIN: out[r][n] = scale * acc (fp32), rows < R_store
  float* out = nullptr;
  int ldo = 0, R_store = 0;
  // EPI_VERDICT: the scaled row is a row of logits; per (row, weight tile) the tile's top_n largest of them with
  // their ids (ties: smaller id first), the sum of exp(l - tile max) when tile_sum is given, and the logit of the
  // row's draft token from the tile that holds it; `out` may be null (logits never stored)
  const int32_t* row_draft = nullptr;
  float* draft_logit = nullptr;
  float4* top_val = nullptr;
  int4* top_idx = nullptr;
  float* tile_sum = nullptr;
  int top_n = 0, n_vtiles = 0;
  // EPI_RESID: resid[r][n] += acc; xb = bf16(resid * gain_next); sumsq_out[tile][r]
  float* resid = nullptr;
  __nv_bfloat16* xb = nullptr;
  const __nv_bfloat16* gain_next = nullptr;
  float* sumsq_out = nullptr;
  // EPI_SWIGLU: W is [gate rows | up rows] (f each); act[r][j] = silu(gate_j) * up_j
  __nv_bfloat16* act = nullptr;
  int f = 0;
  // EPI_QKV: rotary embedding, Q store (bf16, or fp32 into qf when given), K/V page write
  __nv_bfloat16* q = nullptr;
  float* qf = nullptr;
  __nv_bfloat16* pages_layer = nullptr;
  size_t page_elems = 0;
  const int32_t* page_table = nullptr;
  int pages_per_seq = 0;
  const int32_t* row_pos = nullptr;
  const int32_t* row_seq = nullptr;
  const float* rope = nullptr;
  int H = 0, Hkv = 0, dh = 0;
};

// acc[r][n] = sum_k A[r][k] * W[n][k] (A bf16 [R_pad, K], W bf16 [N, K], both row-major),
// finished by the epilogue `epi`.  N and K must be multiples of 8.
laser_status gemm_fused(laser_model* m, const __nv_bfloat16* A, const __nv_bfloat16* W, int R_pad, int N, int K, int epi,
                        const GemmEpilogue& e, cudaStream_t stream);
void gemm_state_free(laser_model* m);

// Brackets one launch with events when profiling is on.
struct ProfScope {
  laser_model* m; int cls; cudaStream_t st; bool on;
  ProfScope(laser_model* m_, int cls_, cudaStream_t st_) : m(m_), cls(cls_), st(st_), on(m_->profile) { mark(); }
  ~ProfScope() { mark(); }
  void mark() {
    if (!on) return;
    auto& ev = m->prof_events[cls];
    size_t& used = m->prof_used[cls];
    if (used == ev.size()) { cudaEvent_t e; if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; } ev.push_back(e); }
    cudaEventRecord(ev[used++], st);
  }
};


// TMA-fed paged attention (head_dim 64 or 128 and a cache small enough for 32-bit row
// coordinates); the verify forward falls back to a plain kernel otherwise.
bool attention_tma_supported(const laser_model* m, const laser_kv* kv);
laser_status attention_tma_launch(laser_model* m, laser_kv* kv, int layer, const int32_t* seq_ids, int B, int Rs, bool tree,
                                  cudaStream_t stream);

// Prompt processing: the verify forward without the LM head over B sequences of Rs rows each (any Rs with
// B * Rs inside the model's row workspace); K and V of the rows go to the cache, lengths are not changed.
laser_status prefill_rows(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                          const int32_t* n_rows, int32_t B, int32_t Rs, cudaStream_t stream);


// The verify forward with acceptance fused into the LM head: per (row, 128-token vocabulary tile) the tile's
// top_n (1..4) largest logits and ids, with `sums` the tile's sum of exp(l - tile max), and per row the logit of
// its draft token, all in the model's buffers; logits (may be null) are stored only when given.
laser_status verify_fused(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                          const int32_t* n_rows, int32_t B, float* logits, int top_n, bool sums, cudaStream_t stream);

}  // namespace laser
