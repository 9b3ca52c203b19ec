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
  __nv_bfloat16* attn = nullptr;   // [R_pad, dq] attention output
  __nv_bfloat16* act = nullptr;    // [R_pad, f] SwiGLU output
  float* part = nullptr;           // split-K partial sums
  size_t part_floats = 0;
  float* rope = nullptr;           // [R_pad, head_dim/2, 2] cos, sin of each row's position
  int32_t* row_pos = nullptr;      // [R_pad] position of the row, -1 = inactive
  int32_t* row_seq = nullptr;      // [R_pad] cache slot of the row
  int32_t* row_ctx = nullptr;      // [max_batch] committed length of each sequence of the step
  int32_t* row_n = nullptr;        // [max_batch] effective rows of each sequence
  int32_t* status = nullptr;       // first device-side error of the stream, 0 = none
  void* gemm_state = nullptr;      // tensor-map cache of the tensor-core GEMM
  // optional per-class kernel timing (class 0 = GEMM, 1 = attention)
  bool profile = false;
  std::vector<cudaEvent_t> prof_events[2];  // begin/end pairs
  size_t prof_used[2] = {0, 0};
};

namespace laser {

// out[s][r][n] = sum over the s-th K-range of A[r][k] * W[n][k]; A bf16 [R_pad, K] row-major,
// W bf16 [N, K] row-major, out fp32 with row stride ldo and split stride split_stride
// (floats).  Rows >= R_store are not written.  Returns the number of splits used through
// *splits_out; the caller sums the partial results.
struct GemmPlan { int splits; };
GemmPlan gemm_plan(int R_pad, int N, int K);
laser_status gemm_launch(laser_model* m, const __nv_bfloat16* A, const __nv_bfloat16* W, float* out,
                         int R_pad, int R_store, int N, int K, int splits, size_t split_stride, int ldo,
                         cudaStream_t stream);
void gemm_state_free(laser_model* m);

// TMA-fed paged attention (head_dim 64 or 128 and a cache small enough for 32-bit row
// coordinates); the verify forward falls back to a plain kernel otherwise.
bool attention_tma_supported(const laser_model* m, const laser_kv* kv);
laser_status attention_tma_launch(laser_model* m, laser_kv* kv, int layer, const int32_t* seq_ids, int B,
                                  cudaStream_t stream);

}  // namespace laser
