// Verify forward with acceptance fused into the LM head (Section 3.4: Eq. 4, Eq. 7, Eq. 8 and the variants of
// Section 4.3.2), so that the [rows, vocabulary] logits are never stored.
//
// The LM-head epilogue leaves, per (row, 128-token vocabulary tile): the tile's largest logits with their ids
// (equal logits: smaller id first), the tile's sum of exp(l - tile max), and - once per row - the logit of the
// row's draft token.  The kernel below finishes the rule from these few numbers per tile:
//   arg max      the best first entry over the tiles (exact);
//   rank < k     entries of all tiles' lists ranked ahead of the draft token; a tile's list holds `top_n >= k`
//                entries, so the capped count is below k exactly when the true count is (exact);
//   probability  exp(l_draft - max) / sum over tiles of tile_sum * exp(tile max - max), combined in fp64.  The
//                tile sums are fp32, so the probability agrees with the two-pass rule on stored logits (fp64 sum
//                of exponentials of fp32 differences) to about 1e-6 relative: the verdicts are the same except
//                for a probability within that distance of the threshold p.
// One CTA per sequence, one warp per row; thread 0 then walks the verdicts in order and commits.
#include "model.cuh"
#include "verdict.cuh"

namespace laser {
namespace {

constexpr int kFusedThreads = 256;

__global__ void __launch_bounds__(kFusedThreads)
accept_fused_kernel(const float4* __restrict__ top_val, const int4* __restrict__ top_idx, const float* __restrict__ tile_sum,
                    const float* __restrict__ draft_logit, const int32_t* __restrict__ tokens, const int32_t* __restrict__ n_rows,
                    const int32_t* __restrict__ seq_ids, int32_t R, int32_t V, int32_t n_vtiles, int32_t top_n, int32_t mode,
                    int32_t topk, double p, int32_t* __restrict__ n_accept, int32_t* __restrict__ out_tokens,
                    int32_t* __restrict__ n_out, int32_t* __restrict__ kv_len) {
  extern __shared__ int32_t s_row[];   // [R] arg max, [R] verdict
  int32_t* s_arg = s_row;
  int32_t* s_pass = s_row + R;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nr = min(n_rows[b], R);
  if (nr <= 0) {
    if (tid == 0) { n_accept[b] = 0; n_out[b] = 0; }
    for (int j = tid; j < R; j += kFusedThreads) out_tokens[b * R + j] = -1;
    return;
  }
  const bool need_p = mode == LASER_MODE_RELAXED || mode == LASER_MODE_TOPP || mode == LASER_MODE_RELAXED_ARGMAX;
  const bool need_rank = mode == LASER_MODE_RELAXED || mode == LASER_MODE_TOPK || mode == LASER_MODE_RELAXED_ARGMAX;
  for (int i = warp; i < nr; i += kFusedThreads / 32) {
    const size_t base = (size_t(b) * R + i) * n_vtiles;
    // max and arg max of the row
    float mx = -INFINITY;
    int arg = 0x7fffffff;
    for (int t = lane; t < n_vtiles; t += 32) better(mx, arg, top_val[base + t].x, top_idx[base + t].x);
    for (int o = 16; o; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, mx, o);
      const int oi = __shfl_xor_sync(0xffffffffu, arg, o);
      better(mx, arg, ov, oi);
    }
    int pass = 0;
    const int d = i + 1 < nr ? tokens[b * R + i + 1] : -1;
    if (d >= 0 && d < V) {
      if (mode == LASER_MODE_STRICT) {
        pass = d == arg;
      } else {
        const float ld = draft_logit[size_t(b) * R + i];
        int ahead = 0;
        double sum = 0.0;
        for (int t = lane; t < n_vtiles; t += 32) {
          const float4 v = top_val[base + t];
          if (need_rank) {
            const int4 id = top_idx[base + t];
            ahead += (v.x > ld) || (v.x == ld && id.x < d);
            if (top_n > 1) ahead += (v.y > ld) || (v.y == ld && id.y < d);
            if (top_n > 2) ahead += (v.z > ld) || (v.z == ld && id.z < d);
            if (top_n > 3) ahead += (v.w > ld) || (v.w == ld && id.w < d);
          }
          if (need_p) sum += double(tile_sum[base + t]) * exp(double(v.x) - double(mx));
        }
        for (int o = 16; o; o >>= 1) {
          ahead += __shfl_xor_sync(0xffffffffu, ahead, o);
          sum += __shfl_xor_sync(0xffffffffu, sum, o);
        }
        const bool in_topk = ahead < topk;
        const bool above_p = need_p && (exp(double(ld) - double(mx)) / sum > p);
        if (mode == LASER_MODE_RELAXED) pass = in_topk && above_p;
        else if (mode == LASER_MODE_TOPK) pass = in_topk;
        else if (mode == LASER_MODE_RELAXED_ARGMAX) pass = (d == arg) || (in_topk && above_p);
        else pass = (d == arg) || above_p;
      }
    }
    if (lane == 0) { s_arg[i] = arg; s_pass[i] = pass; }
  }
  __syncthreads();
  __shared__ int s_a;
  if (tid == 0) {
    int a = 0;
    while (a < nr - 1 && s_pass[a]) ++a;
    s_a = a;
    n_accept[b] = a;
    n_out[b] = a + 1;
    if (kv_len) kv_len[seq_ids[b]] += a + 1;
  }
  __syncthreads();
  const int a = s_a;
  for (int j = tid; j < R; j += kFusedThreads)
    out_tokens[b * R + j] = j < a ? tokens[b * R + j + 1] : (j == a ? s_arg[a] : -1);
}

}  // namespace
}  // namespace laser

LASER_API laser_status laser_verify_accept(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                                           const int32_t* n_rows, int32_t B, const laser_params* p, int32_t commit,
                                           float* logits, int32_t* n_accept, int32_t* out_tokens, int32_t* n_out,
                                           void* stream_) {
  using namespace laser;
  LASER_REQUIRE(m && kv && seq_ids && tokens && n_rows && p && n_accept && out_tokens && n_out, "null argument");
  LASER_REQUIRE(p->K + 1 == m->rows_per_seq, "K = %d but the model steps %d rows per sequence", p->K, m->rows_per_seq);
  LASER_REQUIRE(p->mode >= LASER_MODE_STRICT && p->mode <= LASER_MODE_RELAXED_ARGMAX, "mode = %d", p->mode);
  const bool need_rank = p->mode == LASER_MODE_RELAXED || p->mode == LASER_MODE_TOPK || p->mode == LASER_MODE_RELAXED_ARGMAX;
  const bool need_p = p->mode == LASER_MODE_RELAXED || p->mode == LASER_MODE_TOPP || p->mode == LASER_MODE_RELAXED_ARGMAX;
  LASER_REQUIRE(!need_rank || p->topk >= 1, "topk = %d", p->topk);
  if (need_rank && p->topk > 4) {
    set_error("the fused rule keeps four logits per vocabulary tile: topk = %d needs laser_verify_step + laser_accept_commit", p->topk);
    return LASER_ERR_UNSUPPORTED;
  }
  cudaStream_t stream = as_stream(stream_);
  const int top_n = need_rank ? p->topk : 1;
  LASER_TRY(verify_fused(m, kv, seq_ids, tokens, n_rows, B, logits, top_n, need_p, stream));
  const int R = m->rows_per_seq;
  accept_fused_kernel<<<B, kFusedThreads, size_t(2) * R * sizeof(int32_t), stream>>>(
      m->top_val, m->top_idx, m->tile_sum, m->draft_logit, tokens, n_rows, seq_ids, R, m->cfg.vocab,
      ceil_div(m->cfg.vocab, 128), top_n, p->mode, p->topk, double(p->p), n_accept, out_tokens, n_out,
      commit ? kv->seq_len : nullptr);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}
