// Generation loop: Draft-Then-Verify decoding (Section 2.1, Section 3) and, with no pool,
// plain greedy autoregressive decoding (Eq. 1).  All per-step state stays on the device;
// the host launches the step's kernels and reads back one integer (sequences still active).
#include <algorithm>
#include <vector>

#include "model.cuh"

namespace laser {
namespace {

struct GenState {
  int32_t* seq_tok;      // [B, max_total] prompt followed by generated tokens
  int32_t* seq_len;      // [B] tokens in seq_tok
  int32_t* prompt_len;   // [B]
  int32_t* out_len;      // [B] generated so far
  int32_t* done;         // [B]
  int32_t* cursor;       // [B] prompt tokens already cached
  unsigned long long* counters;  // steps, drafted, accepted, emitted
  int32_t* n_active;     // [1]
  int max_total;
};

// Prompt chunk for the prefill of sequences b0 .. b0 + nb - 1: up to Rs of the not yet cached prompt
// tokens (all but the last) of each.
__global__ void prefill_rows_kernel(GenState g, int b0, int Rs, int32_t* __restrict__ tokens, int32_t* __restrict__ n_rows) {
  const int i = blockIdx.x, b = b0 + i;
  const int remaining = g.prompt_len[b] - 1 - g.cursor[b];
  const int n = max(0, min(Rs, remaining));
  for (int j = threadIdx.x; j < Rs; j += blockDim.x)
    tokens[i * Rs + j] = j < n ? g.seq_tok[size_t(b) * g.max_total + g.cursor[b] + j] : -1;
  if (threadIdx.x == 0) n_rows[i] = n;
}

__global__ void prefill_advance_kernel(GenState g, int b0, int nb, const int32_t* __restrict__ n_rows, int32_t* __restrict__ kv_len) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= nb) return;
  g.cursor[b0 + i] += n_rows[i];
  kv_len[b0 + i] += n_rows[i];
}

// Tail (last n_max tokens, right-aligned) and pending token of every active sequence.
__global__ void step_prep_kernel(GenState g, int B, int n_max, int32_t* __restrict__ tails, int32_t* __restrict__ tail_len,
                                 int32_t* __restrict__ last) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int len = g.seq_len[b];
  const int tl = g.done[b] ? 0 : min(n_max, len);
  for (int j = 0; j < n_max; ++j) {
    const int src = len - n_max + j;
    tails[b * n_max + j] = (j >= n_max - tl) ? g.seq_tok[size_t(b) * g.max_total + src] : -1;
  }
  tail_len[b] = tl;
  last[b] = g.done[b] ? -1 : g.seq_tok[size_t(b) * g.max_total + len - 1];
}

__global__ void no_draft_kernel(int B, int K, int32_t* __restrict__ draft, int32_t* __restrict__ draft_len) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B * K) draft[i] = -1;
  if (i < B) draft_len[i] = 0;
}

// Truncate the emitted tokens to the room left, stop at EOS, append, advance the cache.
__global__ void step_append_kernel(GenState g, int B, int Rs, int max_new, int eos, const int32_t* __restrict__ n_rows,
                                   const int32_t* __restrict__ n_accept, const int32_t* __restrict__ out_tokens,
                                   const int32_t* __restrict__ n_out, int32_t* __restrict__ out, int32_t* __restrict__ kv_len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B && !g.done[b] && n_rows[b] > 0) {
    int n = min(n_out[b], max_new - g.out_len[b]);
    bool fin = false;
    for (int j = 0; j < n; ++j)
      if (eos >= 0 && out_tokens[b * Rs + j] == eos) { n = j + 1; fin = true; break; }
    for (int j = 0; j < n; ++j) {
      const int32_t t = out_tokens[b * Rs + j];
      out[size_t(b) * max_new + g.out_len[b] + j] = t;
      g.seq_tok[size_t(b) * g.max_total + g.seq_len[b] + j] = t;
    }
    g.out_len[b] += n;
    g.seq_len[b] += n;
    kv_len[b] += n;
    if (g.out_len[b] >= max_new) fin = true;
    atomicAdd(&g.counters[0], 1ULL);
    atomicAdd(&g.counters[1], (unsigned long long)(n_rows[b] - 1));
    atomicAdd(&g.counters[2], (unsigned long long)n_accept[b]);
    atomicAdd(&g.counters[3], (unsigned long long)n);
    if (fin) { g.done[b] = 1; atomicSub(g.n_active, 1); }
  }
}

// Work buffers of one laser_generate call, carved out of one allocation that the model keeps and only
// ever grows: requests are collected first, then placed (256-byte aligned) and cleared together.
struct DevBuf {
  struct Req { void** p; size_t bytes; };
  std::vector<Req> reqs;
  template <typename T>
  laser_status get(T** p, size_t count) {
    reqs.push_back(Req{reinterpret_cast<void**>(p), std::max<size_t>(count, 1) * sizeof(T)});
    return LASER_OK;
  }
  laser_status commit(laser_model* m, cudaStream_t stream) {
    size_t total = 0;
    for (const Req& r : reqs) total += (r.bytes + 255) & ~size_t(255);
    if (total > m->gen_bytes) {
      LASER_CUDA(cudaStreamSynchronize(stream));
      if (m->gen_buf) {
        LASER_CUDA(cudaFree(m->gen_buf));
        m->owned.erase(std::remove(m->owned.begin(), m->owned.end(), m->gen_buf), m->owned.end());
      }
      m->gen_buf = nullptr; m->gen_bytes = 0;
      LASER_CUDA(cudaMalloc(&m->gen_buf, total));
      m->owned.push_back(m->gen_buf);
      m->gen_bytes = total;
    }
    LASER_CUDA(cudaMemsetAsync(m->gen_buf, 0, total, stream));
    size_t off = 0;
    for (const Req& r : reqs) { *r.p = static_cast<char*>(m->gen_buf) + off; off += (r.bytes + 255) & ~size_t(255); }
    return LASER_OK;
  }
};

struct Events {
  cudaEvent_t e[5] = {};
  ~Events() { for (auto& x : e) if (x) cudaEventDestroy(x); }
};

}  // namespace
}  // namespace laser

using namespace laser;

LASER_API laser_status laser_generate(laser_model* m, laser_kv* kv, const laser_pool* pool, const int32_t* prompts,
                                      const int64_t* prompt_offsets, const int32_t* group_id, int32_t B,
                                      const laser_params* p, int32_t* out, int32_t* out_len, laser_stats* stats,
                                      void* stream_) {
  LASER_REQUIRE(m && kv && prompts && prompt_offsets && p && out && out_len, "null argument");
  LASER_REQUIRE(pool == nullptr || group_id != nullptr, "group_id is required with a pool");
  LASER_REQUIRE(B >= 1 && B <= m->cfg.max_batch && B <= kv->max_seqs, "B = %d outside [1, min(max_batch, max_seqs)]", B);
  LASER_REQUIRE(p->K == m->cfg.max_draft, "params K = %d differs from the model's max_draft = %d", p->K, m->cfg.max_draft);
  LASER_REQUIRE(p->max_new >= 1, "max_new = %d", p->max_new);
  LASER_REQUIRE(pool == nullptr || (p->K >= 1 && p->n_max >= 1 && p->n_max <= 8), "drafting needs K >= 1 and n_max in [1, 8]");
  LASER_REQUIRE(!p->temp_branches || pool != nullptr, "temporary branches are drafted beside a pool");
  LASER_REQUIRE(!p->tree || pool != nullptr, "tree drafting needs a pool");
  cudaStream_t stream = as_stream(stream_);
  const int K = p->K, Rs = K + 1, n_max = pool ? p->n_max : 1;
  int max_prompt = 0;
  for (int b = 0; b < B; ++b) {
    const int64_t len = prompt_offsets[b + 1] - prompt_offsets[b];
    LASER_REQUIRE(len >= 1, "prompt %d is empty", b);
    LASER_REQUIRE(len - 1 + p->max_new + K <= kv->capacity_tokens(),
                  "prompt %d (%lld tokens) + max_new + K does not fit the %lld tokens of its KV pages", b,
                  (long long)len, (long long)kv->capacity_tokens());
    max_prompt = std::max<int>(max_prompt, int(len));
  }
  const long long launches0 = g_launches;
  DevBuf buf;
  GenState g{};
  g.max_total = max_prompt + p->max_new + Rs;
  int32_t *tokens, *n_rows, *tails, *tail_len, *last, *draft, *draft_len, *match_n, *seq_ids, *gid;
  int32_t *n_accept, *out_tokens, *n_out, *d_out, *draft_par, *parents, *path_rows;
  float* logits;
  LASER_TRY(buf.get(&g.seq_tok, size_t(B) * g.max_total));
  LASER_TRY(buf.get(&g.seq_len, size_t(B)));
  LASER_TRY(buf.get(&g.prompt_len, size_t(B)));
  LASER_TRY(buf.get(&g.out_len, size_t(B)));
  LASER_TRY(buf.get(&g.done, size_t(B)));
  LASER_TRY(buf.get(&g.cursor, size_t(B)));
  LASER_TRY(buf.get(&g.counters, size_t(4)));
  LASER_TRY(buf.get(&g.n_active, size_t(1)));
  LASER_TRY(buf.get(&tokens, std::max(size_t(B) * Rs, size_t(m->R_pad))));
  LASER_TRY(buf.get(&n_rows, size_t(B)));
  LASER_TRY(buf.get(&tails, size_t(B) * n_max));
  LASER_TRY(buf.get(&tail_len, size_t(B)));
  LASER_TRY(buf.get(&last, size_t(B)));
  LASER_TRY(buf.get(&draft, size_t(B) * std::max(K, 1)));
  LASER_TRY(buf.get(&draft_len, size_t(B)));
  LASER_TRY(buf.get(&match_n, size_t(B)));
  LASER_TRY(buf.get(&seq_ids, size_t(B)));
  LASER_TRY(buf.get(&gid, size_t(B)));
  LASER_TRY(buf.get(&draft_par, size_t(B) * std::max(K, 1)));
  LASER_TRY(buf.get(&parents, size_t(B) * Rs));
  LASER_TRY(buf.get(&path_rows, size_t(B) * Rs));
  LASER_TRY(buf.get(&n_accept, size_t(B)));
  LASER_TRY(buf.get(&out_tokens, size_t(B) * Rs));
  LASER_TRY(buf.get(&n_out, size_t(B)));
  LASER_TRY(buf.get(&d_out, size_t(B) * p->max_new));
  const bool fused = p->fused_accept && !(pool && p->tree);   // chain steps without stored logits
  LASER_TRY(buf.get(&logits, fused ? size_t(4) : size_t(B) * Rs * m->cfg.vocab));
  LASER_TRY(buf.commit(m, stream));

  // host -> device: prompts, lengths, ids
  std::vector<int32_t> h_len(B), h_ids(B);
  for (int b = 0; b < B; ++b) {
    h_len[b] = int32_t(prompt_offsets[b + 1] - prompt_offsets[b]);
    h_ids[b] = b;
    LASER_CUDA(cudaMemcpyAsync(g.seq_tok + size_t(b) * g.max_total, prompts + prompt_offsets[b], size_t(h_len[b]) * 4,
                               cudaMemcpyHostToDevice, stream));
  }
  LASER_CUDA(cudaMemcpyAsync(g.seq_len, h_len.data(), size_t(B) * 4, cudaMemcpyHostToDevice, stream));
  LASER_CUDA(cudaMemcpyAsync(g.prompt_len, h_len.data(), size_t(B) * 4, cudaMemcpyHostToDevice, stream));
  LASER_CUDA(cudaMemcpyAsync(seq_ids, h_ids.data(), size_t(B) * 4, cudaMemcpyHostToDevice, stream));
  if (pool) LASER_CUDA(cudaMemcpyAsync(gid, group_id, size_t(B) * 4, cudaMemcpyHostToDevice, stream));
  LASER_CUDA(cudaMemsetAsync(kv->seq_len, 0, size_t(B) * 4, stream));
  LASER_CUDA(cudaMemsetAsync(d_out, 0xff, size_t(B) * p->max_new * 4, stream));
  int32_t h_active = B;
  LASER_CUDA(cudaMemcpyAsync(g.n_active, &h_active, 4, cudaMemcpyHostToDevice, stream));

  Events ev;
  for (auto& x : ev.e) LASER_CUDA(cudaEventCreate(&x));
  float ms_prefill = 0, ms_draft = 0, ms_verify = 0, ms_accept = 0, ms;
  LASER_CUDA(cudaEventRecord(ev.e[0], stream));

  // prefill: every prompt token but the last.  A pass of Rs rows per sequence would read a sequence's
  // whole cached prefix once per Rs prompt tokens; instead the model's row workspace is given to few
  // sequences at a time, up to 128 rows each, and the LM head is left out.
  const int chunk = std::max(Rs, std::min(128, m->R_pad / 16 * 16));
  const int group = std::max(1, std::min(B, m->R_pad / chunk));
  int n_pass = 0;
  for (int b0 = 0; b0 < B; b0 += group) {
    const int nb = std::min(group, B - b0);
    int longest = 0;
    for (int b = b0; b < b0 + nb; ++b) longest = std::max(longest, h_len[b] - 1);
    for (int it = 0; it < ceil_div(longest, chunk); ++it, ++n_pass) {
      prefill_rows_kernel<<<nb, 32, 0, stream>>>(g, b0, chunk, tokens, n_rows);
      LASER_TRY(prefill_rows(m, kv, seq_ids + b0, tokens, n_rows, nb, chunk, stream));
      prefill_advance_kernel<<<ceil_div(nb, 128), 128, 0, stream>>>(g, b0, nb, n_rows, kv->seq_len);
      count_launch(2);
      if ((n_pass & 15) == 15) LASER_TRY(laser_check(m, stream));   // do not keep launching after a device-side error
    }
  }
  LASER_CUDA(cudaEventRecord(ev.e[1], stream));
  LASER_CUDA(cudaStreamSynchronize(stream));
  LASER_CUDA(cudaEventElapsedTime(&ms_prefill, ev.e[0], ev.e[1]));

  laser_params acc = *p;
  int64_t verify_calls = 0;
  int32_t h_status = 0;
  const int max_steps = p->max_new + 1;
  for (int step = 0; step < max_steps && h_active > 0; ++step) {
    LASER_CUDA(cudaEventRecord(ev.e[0], stream));
    step_prep_kernel<<<ceil_div(B, 128), 128, 0, stream>>>(g, B, n_max, tails, tail_len, last);
    count_launch();
    if (pool) {
      // temporary branch: the sequence's prompt and generated tokens (seq_tok) are searched as well
      if (p->tree)
        LASER_TRY(laser_draft_tree(pool, tails, tail_len, gid, p->temp_branches ? g.seq_tok : nullptr,
                                   p->temp_branches ? g.seq_len : nullptr, p->temp_branches ? g.max_total : 0, B, p, draft,
                                   draft_par, draft_len, match_n, stream));
      else if (p->temp_branches)
        LASER_TRY(laser_draft_temp(pool, tails, tail_len, gid, g.seq_tok, g.seq_len, g.max_total, B, p, draft, draft_len,
                                   match_n, stream));
      else
        LASER_TRY(laser_draft(pool, tails, tail_len, gid, B, p, draft, draft_len, match_n, stream));
    } else {
      no_draft_kernel<<<ceil_div(B * std::max(K, 1), 128), 128, 0, stream>>>(B, K, draft, draft_len);
      count_launch();
    }
    const bool tree = pool && p->tree;
    if (tree) LASER_TRY(laser_make_rows_tree(last, draft, draft_par, draft_len, B, K, tokens, parents, n_rows, stream));
    else LASER_TRY(laser_make_rows(last, draft, draft_len, B, K, tokens, n_rows, stream));
    LASER_CUDA(cudaEventRecord(ev.e[1], stream));
    if (tree) LASER_TRY(laser_verify_step_tree(m, kv, seq_ids, tokens, parents, n_rows, B, logits, stream));
    else if (fused) LASER_TRY(laser_verify_accept(m, kv, seq_ids, tokens, n_rows, B, &acc, 0, nullptr, n_accept, out_tokens, n_out, stream));
    else LASER_TRY(laser_verify_step(m, kv, seq_ids, tokens, n_rows, B, logits, stream));
    ++verify_calls;
    LASER_CUDA(cudaEventRecord(ev.e[2], stream));
    if (fused && !tree) {
      // the verdict came with the forward
    } else if (tree) {
      // verdict, then the accepted path's K/V to consecutive slots (the lengths advance in step_append)
      LASER_TRY(laser_accept_tree(nullptr, nullptr, logits, tokens, parents, n_rows, B, m->cfg.vocab, &acc, n_accept,
                                  out_tokens, n_out, path_rows, stream));
      LASER_TRY(laser_kv_compact_path(kv, seq_ids, path_rows, n_accept, B, Rs, stream));
    } else {
      LASER_TRY(laser_accept_commit(nullptr, nullptr, logits, tokens, n_rows, B, m->cfg.vocab, &acc, n_accept, out_tokens,
                                    n_out, stream));
    }
    step_append_kernel<<<ceil_div(B, 128), 128, 0, stream>>>(g, B, Rs, p->max_new, p->eos_id, n_rows, n_accept,
                                                            out_tokens, n_out, d_out, kv->seq_len);
    count_launch();
    LASER_CUDA(cudaEventRecord(ev.e[3], stream));
    LASER_CUDA(cudaMemcpyAsync(&h_active, g.n_active, 4, cudaMemcpyDeviceToHost, stream));
    LASER_CUDA(cudaMemcpyAsync(&h_status, m->status, 4, cudaMemcpyDeviceToHost, stream));
    LASER_CUDA(cudaStreamSynchronize(stream));
    if (h_status != 0) break;   // a device-side error (capacity, a wait that ran out): stop at once, laser_check reports it
    LASER_CUDA(cudaEventElapsedTime(&ms, ev.e[0], ev.e[1])); ms_draft += ms;
    LASER_CUDA(cudaEventElapsedTime(&ms, ev.e[1], ev.e[2])); ms_verify += ms;
    LASER_CUDA(cudaEventElapsedTime(&ms, ev.e[2], ev.e[3])); ms_accept += ms;
  }
  LASER_TRY(laser_check(m, stream));
  LASER_CUDA(cudaMemcpyAsync(out, d_out, size_t(B) * p->max_new * 4, cudaMemcpyDeviceToHost, stream));
  LASER_CUDA(cudaMemcpyAsync(out_len, g.out_len, size_t(B) * 4, cudaMemcpyDeviceToHost, stream));
  unsigned long long h_cnt[4] = {};
  LASER_CUDA(cudaMemcpyAsync(h_cnt, g.counters, sizeof(h_cnt), cudaMemcpyDeviceToHost, stream));
  LASER_CUDA(cudaStreamSynchronize(stream));
  if (h_active > 0) { set_error("generation did not finish in %d steps", max_steps); return LASER_ERR_TIMEOUT; }
  if (stats) {
    stats->steps = int64_t(h_cnt[0]); stats->drafted = int64_t(h_cnt[1]);
    stats->accepted = int64_t(h_cnt[2]); stats->emitted = int64_t(h_cnt[3]);
    stats->launches = g_launches - launches0;
    stats->verify_calls = verify_calls;
    stats->ms_prefill = ms_prefill; stats->ms_draft = ms_draft; stats->ms_verify = ms_verify;
    stats->ms_accept = ms_accept; stats->ms_total = ms_prefill + ms_draft + ms_verify + ms_accept;
  }
  return LASER_OK;
}
