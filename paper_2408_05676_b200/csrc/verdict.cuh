// Row passes shared by the acceptance kernels (Eq. 4, Eq. 7, Eq. 8 and the variants of Section
// 4.3.2): max and arg max of a row of logits, and the verdict on one token given its row - its rank
// (tokens ahead of it; equal logits rank the smaller id first) and, where the rule needs it, its
// probability with the denominator summed in fp64 from fp32 differences.  One CTA of kVerdictThreads
// threads works on one row; reductions have a fixed shape, so results are identical from run to run.
#pragma once
#include "common.cuh"

namespace laser {

constexpr int kVerdictThreads = 256;

__device__ __forceinline__ void better(float& v, int& i, float ov, int oi) {
  if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

// max and arg max (smallest id on ties) of a row, by the whole CTA
static __device__ void cta_argmax(const float* __restrict__ row, int V, float* mx_out, int* arg_out) {
  __shared__ float s_val[kVerdictThreads / 32];
  __shared__ int s_idx[kVerdictThreads / 32];
  __shared__ float s_max;
  __shared__ int s_arg;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(row) & 15) == 0);
  float best = -INFINITY;
  int besti = 0x7fffffff;
  if (vec) {
    const float4* r4 = reinterpret_cast<const float4*>(row);
    for (int j = tid; j < V / 4; j += kVerdictThreads) {
      const float4 x = r4[j];
      better(best, besti, x.x, 4 * j); better(best, besti, x.y, 4 * j + 1);
      better(best, besti, x.z, 4 * j + 2); better(best, besti, x.w, 4 * j + 3);
    }
  } else {
    for (int j = tid; j < V; j += kVerdictThreads) better(best, besti, row[j], j);
  }
  for (int o = 16; o; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
    better(best, besti, ov, oi);
  }
  __syncthreads();   // the shared slots may still be read from an earlier call
  if (lane == 0) { s_val[warp] = best; s_idx[warp] = besti; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kVerdictThreads / 32; ++w) better(best, besti, s_val[w], s_idx[w]);
    s_max = best; s_arg = besti;
  }
  __syncthreads();
  *mx_out = s_max;
  *arg_out = s_arg;
}

// whether token t passes on `row` (whose max and arg max are given); the result is valid in thread 0
static __device__ int cta_verdict(const float* __restrict__ row, int V, int t, float mx, int arg, int mode, int topk, double p) {
  if (t < 0 || t >= V) return 0;
  if (mode == LASER_MODE_STRICT) return t == arg;
  __shared__ int s_cnt[kVerdictThreads / 32];
  __shared__ double s_sum[kVerdictThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(row) & 15) == 0);
  const float lt = row[t];
  const bool need_p = (mode == LASER_MODE_RELAXED || mode == LASER_MODE_TOPP || mode == LASER_MODE_RELAXED_ARGMAX);
  int ahead = 0;
  double sum = 0.0;
  auto visit = [&](float x, int j) {
    ahead += (x > lt) || (x == lt && j < t);
    if (need_p) sum += exp(double(x - mx));
  };
  if (vec) {
    const float4* r4 = reinterpret_cast<const float4*>(row);
    for (int j = tid; j < V / 4; j += kVerdictThreads) {
      const float4 x = r4[j];
      visit(x.x, 4 * j); visit(x.y, 4 * j + 1); visit(x.z, 4 * j + 2); visit(x.w, 4 * j + 3);
    }
  } else {
    for (int j = tid; j < V; j += kVerdictThreads) visit(row[j], j);
  }
  for (int o = 16; o; o >>= 1) {
    ahead += __shfl_xor_sync(0xffffffffu, ahead, o);
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
  }
  if (lane == 0) { s_cnt[warp] = ahead; s_sum[warp] = sum; }
  __syncthreads();
  int pass = 0;
  if (tid == 0) {
    for (int w = 1; w < kVerdictThreads / 32; ++w) { ahead += s_cnt[w]; sum += s_sum[w]; }
    const bool in_topk = ahead < topk;
    const bool above_p = need_p && (exp(double(lt - mx)) / sum > p);
    if (mode == LASER_MODE_RELAXED) pass = in_topk && above_p;
    else if (mode == LASER_MODE_TOPK) pass = in_topk;
    else if (mode == LASER_MODE_RELAXED_ARGMAX) pass = (t == arg) || (in_topk && above_p);
    else pass = (t == arg) || above_p;
  }
  return pass;
}

}  // namespace laser
