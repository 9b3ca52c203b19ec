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
#include "verdict.cuh"

namespace laser {
namespace {

constexpr int kAcceptThreads = kVerdictThreads;
constexpr int kMaxAcceptSeqs = 1 << 16;  // counters live at the start of the scratch

struct RowVerdict { int32_t argmax; int32_t pass; };

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
  // pass 1: max and arg max; pass 2 (the row is now in L1/L2): the verdict on the draft token this
  // row verifies, if any.  The branch conditions are uniform across the CTA.
  float mx;
  int arg;
  cta_argmax(row, V, &mx, &arg);
  int pass = 0;
  if (i + 1 < nr) pass = cta_verdict(row, V, tokens[b * R + i + 1], mx, arg, mode, topk, p);

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
