// Verification of a token tree (Section 3.4, tree part): a node is verified when its parent is
// and its token passes the criterion (Eq. 4, Eq. 8 or the ablation variants) on the distribution
// of its parent's row; the verified node of greatest depth wins (the first in depth-first order
// among equals), its path is accepted and one more token comes from its own row.  The accepted
// path's K and V are then moved from their rows' cache slots to consecutive positions.
//
// One CTA per (sequence, row): arg max of the row itself (the token it would emit), and for a
// node the verdict on its token, read off its parent's row (max, rank, fp64 denominator).  The
// last CTA of a sequence to finish walks the tree.  Reductions have a fixed shape.
#include <algorithm>

#include "state.cuh"
#include "verdict.cuh"

namespace laser {
namespace {

constexpr int kThreads = kVerdictThreads;
constexpr int kMaxSeqs = 1 << 16;   // arrival counters at the start of the scratch
constexpr int kMaxTreeRows = 64;

struct NodeVerdict { int32_t argmax; int32_t pass; };

__global__ void __launch_bounds__(kThreads)
accept_tree_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens,
                   const int32_t* __restrict__ parents, const int32_t* __restrict__ n_rows, int32_t R, int32_t V,
                   int32_t mode, int32_t topk, double p, int32_t* __restrict__ counters,
                   NodeVerdict* __restrict__ verdicts, int32_t* __restrict__ n_accept,
                   int32_t* __restrict__ out_tokens, int32_t* __restrict__ n_out, int32_t* __restrict__ path_rows) {
  const int b = blockIdx.x / R, i = blockIdx.x % R;
  const int nr = min(n_rows[b], R);
  const int tid = threadIdx.x;
  if (nr <= 0) {
    if (i == 0) {
      if (tid == 0) { n_accept[b] = 0; n_out[b] = 0; }
      for (int j = tid; j < R; j += kThreads) { out_tokens[b * R + j] = -1; path_rows[b * R + j] = -1; }
    }
    return;
  }
  if (i >= nr) return;
  float mx;
  int arg;
  cta_argmax(logits + (size_t(b) * R + i) * V, V, &mx, &arg);
  int pass = 0;
  if (i > 0) {
    const int par = parents[b * R + i];
    if (par >= 0 && par < i) {      // a malformed parent verifies nothing
      const float* prow = logits + (size_t(b) * R + par) * V;
      float pmx;
      int parg;
      cta_argmax(prow, V, &pmx, &parg);
      pass = cta_verdict(prow, V, tokens[b * R + i], pmx, parg, mode, topk, p);
    }
  }
  __shared__ int s_last;
  if (tid == 0) {
    verdicts[b * R + i] = NodeVerdict{arg, pass};
    __threadfence();
    const int done = atomicAdd(&counters[b], 1);
    s_last = (done == nr - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // the last CTA walks the tree (depth-first order: a parent precedes its children)
  __shared__ int s_a, s_path[kMaxTreeRows];
  const volatile NodeVerdict* v = verdicts + b * R;
  if (tid == 0) {
    unsigned long long ok = 1ull;
    int depth[kMaxTreeRows];
    depth[0] = 0;
    int best = 0;
    for (int j = 1; j < nr; ++j) {
      const int par = parents[b * R + j];
      const bool good = par >= 0 && par < j && ((ok >> par) & 1ull) && v[j].pass;
      depth[j] = good ? depth[par] + 1 : 0;
      if (good) ok |= 1ull << j;
      if (good && depth[j] > depth[best]) best = j;
    }
    const int a = depth[best];
    for (int j = best, d = a; d > 0; --d) { s_path[d - 1] = j; j = parents[b * R + j]; }
    s_path[a] = best;     // the row that emits the extra token
    s_a = a;
    n_accept[b] = a;
    n_out[b] = a + 1;
    counters[b] = 0;      // ready for the next call
  }
  __syncthreads();
  const int a = s_a;
  for (int j = tid; j < R; j += kThreads) {
    out_tokens[b * R + j] = j < a ? tokens[b * R + s_path[j]] : (j == a ? v[s_path[a]].argmax : -1);
    path_rows[b * R + j] = j < a ? s_path[j] : -1;
  }
}

// Moves the K and V of the accepted rows to consecutive cache slots: slot ctx + path[j] ->
// ctx + j + 1, j ascending (a target is never a later source, since path[j] >= j + 1 and the
// rows ascend).  One block per (sequence, layer); a thread owns fixed 16-byte chunks of a token.
__global__ void compact_path_kernel(__nv_bfloat16* __restrict__ pages, size_t layer_elems, size_t page_elems,
                                    const int32_t* __restrict__ page_table, int pages_per_seq, int Hkv, int dh,
                                    const int32_t* __restrict__ seq_ids, const int32_t* __restrict__ seq_len,
                                    const int32_t* __restrict__ path_rows, const int32_t* __restrict__ n_accept,
                                    int row_stride, int max_seqs, int capacity) {
  const int b = blockIdx.x, layer = blockIdx.y;
  const int seq = seq_ids[b];
  if (seq < 0 || seq >= max_seqs) return;
  const int a = min(n_accept[b], row_stride - 1), ctx = seq_len[seq];
  const int32_t* pt = page_table + size_t(seq) * pages_per_seq;
  __nv_bfloat16* base = pages + size_t(layer) * layer_elems;
  const int chunks = 2 * Hkv * (dh / 8);     // 16-byte chunks of one token (K and V, all heads)
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    const int kvh = c / (dh / 8), off = (c % (dh / 8)) * 8;   // kvh = (K|V) * Hkv + head
    for (int j = 0; j < a; ++j) {
      const int row = path_rows[b * row_stride + j];
      const int src = ctx + row, dst = ctx + j + 1;
      if (row < j + 1 || src >= capacity || src == dst) continue;
      const uint4* s = reinterpret_cast<const uint4*>(base + size_t(pt[src >> 4]) * page_elems + (size_t(kvh) * 16 + (src & 15)) * dh + off);
      uint4* d = reinterpret_cast<uint4*>(base + size_t(pt[dst >> 4]) * page_elems + (size_t(kvh) * 16 + (dst & 15)) * dh + off);
      *d = *s;
    }
  }
}

__global__ void advance_len_kernel(const int32_t* __restrict__ seq_ids, const int32_t* __restrict__ n_out, int B,
                                   int max_seqs, int32_t* __restrict__ seq_len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B && seq_ids[b] >= 0 && seq_ids[b] < max_seqs) seq_len[seq_ids[b]] += n_out[b];
}

}  // namespace
}  // namespace laser

LASER_API laser_status laser_kv_compact_path(laser_kv* kv, const int32_t* seq_ids, const int32_t* path_rows,
                                             const int32_t* n_accept, int32_t B, int32_t row_stride, void* stream) {
  using namespace laser;
  LASER_REQUIRE(kv && seq_ids && path_rows && n_accept, "null argument");
  LASER_REQUIRE(B >= 0 && row_stride >= 1, "B = %d, row_stride = %d", B, row_stride);
  LASER_REQUIRE(kv->head_dim % 8 == 0, "head_dim = %d is not a multiple of 8", kv->head_dim);
  if (B == 0) return LASER_OK;
  const int capacity = int(std::min<int64_t>(kv->capacity_tokens(), INT32_MAX));
  compact_path_kernel<<<dim3(unsigned(B), unsigned(kv->n_layers)), 128, 0, as_stream(stream)>>>(
      kv->pages, kv->layer_elems(), kv->page_elems(), kv->page_table, kv->pages_per_seq, kv->n_kv_heads, kv->head_dim,
      seq_ids, kv->seq_len, path_rows, n_accept, row_stride, kv->max_seqs, capacity);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_accept_tree(laser_kv* kv, const int32_t* seq_ids, const float* logits,
                                         const int32_t* tokens, const int32_t* parents, const int32_t* n_rows,
                                         int32_t B, int32_t V, const laser_params* p, int32_t* n_accept,
                                         int32_t* out_tokens, int32_t* n_out, int32_t* path_rows, void* stream) {
  using namespace laser;
  LASER_REQUIRE(p && logits && tokens && parents && n_rows && n_accept && out_tokens && n_out && path_rows, "null argument");
  LASER_REQUIRE(B >= 0 && B <= kMaxSeqs, "B = %d outside [0, %d]", B, kMaxSeqs);
  LASER_REQUIRE(V >= 1, "V = %d", V);
  LASER_REQUIRE(p->K >= 0 && p->K + 1 <= kMaxTreeRows, "a token tree has at most %d rows (K + 1 = %d)", kMaxTreeRows, p->K + 1);
  LASER_REQUIRE(p->mode >= LASER_MODE_STRICT && p->mode <= LASER_MODE_RELAXED_ARGMAX, "mode = %d", p->mode);
  LASER_REQUIRE(p->mode == LASER_MODE_STRICT || p->mode == LASER_MODE_TOPP || p->topk >= 1, "topk = %d", p->topk);
  LASER_REQUIRE(kv == nullptr || seq_ids != nullptr, "seq_ids is required when committing");
  if (B == 0) return LASER_OK;
  const int R = p->K + 1;
  void* scratch = nullptr;
  const size_t counters_bytes = sizeof(int32_t) * kMaxSeqs;
  LASER_TRY(scratch_get(SCRATCH_ACCEPT_TREE, counters_bytes + sizeof(NodeVerdict) * size_t(B) * R, &scratch));
  int32_t* counters = static_cast<int32_t*>(scratch);
  NodeVerdict* verdicts = reinterpret_cast<NodeVerdict*>(static_cast<char*>(scratch) + counters_bytes);
  accept_tree_kernel<<<B * R, kThreads, 0, as_stream(stream)>>>(logits, tokens, parents, n_rows, R, V, p->mode, p->topk,
                                                              double(p->p), counters, verdicts, n_accept, out_tokens,
                                                              n_out, path_rows);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  if (kv) {   // commit: compact the accepted path, then advance the lengths by the emitted tokens
    LASER_TRY(laser_kv_compact_path(kv, seq_ids, path_rows, n_accept, B, R, stream));
    advance_len_kernel<<<ceil_div(B, 128), 128, 0, as_stream(stream)>>>(seq_ids, n_out, B, kv->max_seqs, kv->seq_len);
    count_launch();
    LASER_CUDA(cudaGetLastError());
  }
  return LASER_OK;
}
