// Acceptance and commit: greedy verification (Eq. 4), Relaxed Verification (Eq. 8) and the
// ablation variants (Eq. 7; "top-p" of Section 4.3.2), longest accepted prefix, correction
// or bonus token, and the KV-cache length update.
//
// One CTA per (sequence, row): pass 1 finds max / arg max (smallest id on ties), pass 2
// (the row is now in L1/L2) counts the tokens ranked ahead of the draft token and, where the
// rule needs a probability, sums exp(l - max) in fp64.  The last CTA of a sequence to finish
// walks the per-row verdicts in order and writes the outputs.  Reductions have a fixed
// shape, so results are identical from run to run.
#include <mutex>

#include "state.cuh"

namespace laser {
namespace {

constexpr int kAcceptThreads = 256;
constexpr int kMaxAcceptSeqs = 1 << 16;  // counters live at the start of the scratch

struct RowVerdict { int32_t argmax; int32_t pass; };

__device__ __forceinline__ void better(float& v, int& i, float ov, int oi) {
  if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

__global__ void __launch_bounds__(kAcceptThreads)
accept_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens,
                   const int32_t* __restrict__ n_rows, const int32_t* __restrict__ seq_ids,
                   int32_t R, int32_t V, int32_t mode, int32_t topk, double p,
                   int32_t* __restrict__ counters, RowVerdict* __restrict__ verdicts,
                   int32_t* __restrict__ n_accept, int32_t* __restrict__ out_tokens,
                   int32_t* __restrict__ n_out, int32_t* __restrict__ kv_len) {
  const int b = blockIdx.x / R, i = blockIdx.x % R;
  const int nr = min(n_rows[b], R);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (nr <= 0) {
    if (i == 0) {
      if (tid == 0) { n_accept[b] = 0; n_out[b] = 0; }
      for (int j = tid; j < R; j += kAcceptThreads) out_tokens[b * R + j] = -1;
    }
    return;
  }
  if (i >= nr) return;

  const float* row = logits + (size_t(b) * R + i) * V;
  const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(row) & 15) == 0);
  __shared__ float s_val[kAcceptThreads / 32];
  __shared__ int s_idx[kAcceptThreads / 32];
  __shared__ int s_cnt[kAcceptThreads / 32];
  __shared__ double s_sum[kAcceptThreads / 32];
  __shared__ float s_max;
  __shared__ int s_arg;

  // pass 1: max and arg max
  float best = -INFINITY;
  int besti = 0x7fffffff;
  if (vec) {
    const float4* r4 = reinterpret_cast<const float4*>(row);
    for (int j = tid; j < V / 4; j += kAcceptThreads) {
      float4 x = r4[j];
      better(best, besti, x.x, 4 * j); better(best, besti, x.y, 4 * j + 1);
      better(best, besti, x.z, 4 * j + 2); better(best, besti, x.w, 4 * j + 3);
    }
  } else {
    for (int j = tid; j < V; j += kAcceptThreads) better(best, besti, row[j], j);
  }
  for (int o = 16; o; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, best, o);
    int oi = __shfl_xor_sync(0xffffffffu, besti, o);
    better(best, besti, ov, oi);
  }
  if (lane == 0) { s_val[warp] = best; s_idx[warp] = besti; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kAcceptThreads / 32; ++w) better(best, besti, s_val[w], s_idx[w]);
    s_max = best; s_arg = besti;
  }
  __syncthreads();
  const float mx = s_max;
  const int arg = s_arg;

  // pass 2: verdict on the draft token verified by this row (if any); all branch
  // conditions below are uniform across the CTA
  int pass = 0;
  if (i + 1 < nr) {
    const int t = tokens[b * R + i + 1];
    if (t >= 0 && t < V) {
      if (mode == LASER_MODE_STRICT) {
        pass = (t == arg);
      } else {
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
          for (int j = tid; j < V / 4; j += kAcceptThreads) {
            float4 x = r4[j];
            visit(x.x, 4 * j); visit(x.y, 4 * j + 1); visit(x.z, 4 * j + 2); visit(x.w, 4 * j + 3);
          }
        } else {
          for (int j = tid; j < V; j += kAcceptThreads) visit(row[j], j);
        }
        for (int o = 16; o; o >>= 1) {
          ahead += __shfl_xor_sync(0xffffffffu, ahead, o);
          sum += __shfl_xor_sync(0xffffffffu, sum, o);
        }
        if (lane == 0) { s_cnt[warp] = ahead; s_sum[warp] = sum; }
        __syncthreads();
        if (tid == 0) {
          for (int w = 1; w < kAcceptThreads / 32; ++w) { ahead += s_cnt[w]; sum += s_sum[w]; }
          const bool in_topk = ahead < topk;
          const bool above_p = need_p && (exp(double(lt - mx)) / sum > p);
          if (mode == LASER_MODE_RELAXED) pass = in_topk && above_p;
          else if (mode == LASER_MODE_TOPK) pass = in_topk;
          else if (mode == LASER_MODE_RELAXED_ARGMAX) pass = (t == arg) || (in_topk && above_p);
          else pass = (t == arg) || above_p;
        }
      }
    }
  }

  // publish, then let the last CTA of this sequence scan the verdicts in order
  __shared__ int s_last;
  if (tid == 0) {
    verdicts[b * R + i] = RowVerdict{arg, pass};
    __threadfence();
    const int done = atomicAdd(&counters[b], 1);
    s_last = (done == nr - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  __shared__ int s_a;
  const volatile RowVerdict* v = verdicts + b * R;
  if (tid == 0) {
    int a = 0;
    while (a < nr - 1 && v[a].pass) ++a;
    s_a = a;
    n_accept[b] = a;
    n_out[b] = a + 1;
    if (kv_len) kv_len[seq_ids[b]] += a + 1;
    counters[b] = 0;  // ready for the next call
  }
  __syncthreads();
  const int a = s_a;
  for (int j = tid; j < R; j += kAcceptThreads)
    out_tokens[b * R + j] = j < a ? tokens[b * R + j + 1] : (j == a ? v[a].argmax : -1);
}

// Fixed scratch of the allocation-free entry point: per-sequence counters, then row verdicts.
constexpr int kNoAllocMaxSeqs = 1024;
constexpr int kNoAllocMaxRows = 16384;
constexpr size_t kNoAllocCounterBytes = sizeof(int32_t) * kNoAllocMaxSeqs;
constexpr size_t kNoAllocBytes = kNoAllocCounterBytes + sizeof(RowVerdict) * kNoAllocMaxRows;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// Device address of g_noalloc_scratch on the current device, resolved once per device.  Host threads
// may make their first calls at the same time: the table is guarded by a mutex.
laser_status noalloc_scratch(void** out) {
  constexpr int kMaxDevices = 64;
  static void* addr[kMaxDevices] = {};
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  LASER_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) { set_error("device index %d out of range", dev); return LASER_ERR_UNSUPPORTED; }
  if (!addr[dev]) {
    void* p = nullptr;
    // the symbol's name is only a host-side handle; the kernel needs the address the runtime maps it to
    LASER_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    addr[dev] = p;
  }
  *out = addr[dev];
  return LASER_OK;
}

}  // namespace
}  // namespace laser

LASER_API laser_status laser_accept_commit_noalloc(laser_kv* kv, const int32_t* seq_ids, const float* logits,
                                                   const int32_t* tokens, const int32_t* n_rows, int32_t B,
                                                   int32_t V, const laser_params* p, int32_t* n_accept,
                                                   int32_t* out_tokens, int32_t* n_out, void* stream) {
  using namespace laser;
  LASER_REQUIRE(p && logits && tokens && n_rows && n_accept && out_tokens && n_out, "null argument");
  LASER_REQUIRE(B >= 0 && V >= 1 && p->K >= 0, "B = %d, V = %d, K = %d", B, V, p->K);
  LASER_REQUIRE(p->mode >= LASER_MODE_STRICT && p->mode <= LASER_MODE_RELAXED_ARGMAX, "mode = %d", p->mode);
  LASER_REQUIRE(p->mode == LASER_MODE_STRICT || p->mode == LASER_MODE_TOPP || p->topk >= 1, "topk = %d", p->topk);
  LASER_REQUIRE(kv == nullptr || seq_ids != nullptr, "seq_ids is required when committing");
  const int64_t rows = int64_t(B) * (int64_t(p->K) + 1);
  if (B > kNoAllocMaxSeqs || rows > kNoAllocMaxRows) {
    set_error("laser_accept_commit_noalloc handles at most %d sequences and %d rows (B * (K+1)); got B = %d, rows = %lld",
              kNoAllocMaxSeqs, kNoAllocMaxRows, B, (long long)rows);
    return LASER_ERR_CAPACITY;
  }
  if (B == 0) return LASER_OK;
  void* scratch = nullptr;
  LASER_TRY(noalloc_scratch(&scratch));
  int32_t* counters = static_cast<int32_t*>(scratch);
  RowVerdict* verdicts = reinterpret_cast<RowVerdict*>(static_cast<char*>(scratch) + kNoAllocCounterBytes);
  // the array keeps whatever the previous call left: the arrival counters must start at zero
  LASER_CUDA(cudaMemsetAsync(counters, 0, sizeof(int32_t) * size_t(B), as_stream(stream)));
  const int R = p->K + 1;
  accept_rows_kernel<<<B * R, kAcceptThreads, 0, as_stream(stream)>>>(
      logits, tokens, n_rows, seq_ids, R, V, p->mode, p->topk, double(p->p), counters, verdicts,
      n_accept, out_tokens, n_out, kv ? kv->seq_len : nullptr);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_accept_commit(laser_kv* kv, const int32_t* seq_ids,
                                           const float* logits, const int32_t* tokens,
                                           const int32_t* n_rows, int32_t B, int32_t V,
                                           const laser_params* p, int32_t* n_accept,
                                           int32_t* out_tokens, int32_t* n_out, void* stream) {
  using namespace laser;
  LASER_REQUIRE(p && logits && tokens && n_rows && n_accept && out_tokens && n_out, "null argument");
  LASER_REQUIRE(B >= 0 && B <= kMaxAcceptSeqs, "B = %d outside [0, %d]", B, kMaxAcceptSeqs);
  LASER_REQUIRE(V >= 1, "V = %d", V);
  LASER_REQUIRE(p->K >= 0 && p->K <= 1023, "K = %d outside [0, 1023]", p->K);
  LASER_REQUIRE(p->mode >= LASER_MODE_STRICT && p->mode <= LASER_MODE_RELAXED_ARGMAX, "mode = %d", p->mode);
  LASER_REQUIRE(p->mode == LASER_MODE_STRICT || p->mode == LASER_MODE_TOPP || p->topk >= 1,
                "topk = %d", p->topk);
  LASER_REQUIRE(kv == nullptr || seq_ids != nullptr, "seq_ids is required when committing");
  if (B == 0) return LASER_OK;
  const int R = p->K + 1;
  void* scratch = nullptr;
  const size_t counters_bytes = sizeof(int32_t) * kMaxAcceptSeqs;
  LASER_TRY(scratch_get(SCRATCH_ACCEPT, counters_bytes + sizeof(RowVerdict) * size_t(B) * R, &scratch));
  int32_t* counters = static_cast<int32_t*>(scratch);
  RowVerdict* verdicts = reinterpret_cast<RowVerdict*>(static_cast<char*>(scratch) + counters_bytes);
  accept_rows_kernel<<<B * R, kAcceptThreads, 0, as_stream(stream)>>>(
      logits, tokens, n_rows, seq_ids, R, V, p->mode, p->topk, double(p->p), counters, verdicts,
      n_accept, out_tokens, n_out, kv ? kv->seq_len : nullptr);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}
