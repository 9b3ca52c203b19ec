// Target model M and its paged KV cache; the verify forward q_i = M(x_<=t, x~_<i) of
// Eq. 3 / Eq. 6 for a Llama-style decoder (RMSNorm, rotary embedding with rotate-half
// pairing, causal attention, SwiGLU, no biases).
//
// One step processes R = B * (K+1) rows.  The residual stream, the norm statistics and the
// softmax stay in fp32; GEMM operands, Q and the K/V cache are bf16.  K and V of all rows
// are written to the pages before attention, so attention reads cache and new rows alike.
#include <cmath>

#include "model.cuh"
#include "tma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;


// ---- row bookkeeping -------------------------------------------------------------------
// One block per row: position, cache slot, capacity check, rotary angles (fp64 -> fp32).
// With `parents` (token tree, Section 3.3) a row's position is ctx + its depth, its cache slot
// stays ctx + row index, and row_mask gets the rows it attends to (its ancestors and itself).
__global__ void prep_rows_kernel(const int32_t* __restrict__ seq_ids, const int32_t* __restrict__ n_rows,
                                 const int32_t* __restrict__ parents, unsigned long long* __restrict__ row_mask,
                                 int B, int Rs, int R_pad, const int32_t* __restrict__ seq_len,
                                 int max_seqs, int capacity, int half, double theta, int head_dim,
                                 int32_t* __restrict__ row_pos, int32_t* __restrict__ row_seq,
                                 int32_t* __restrict__ row_ctx, int32_t* __restrict__ row_n,
                                 float* __restrict__ rope, int32_t* __restrict__ status) {
  const int r = blockIdx.x;
  const int b = r / Rs, i = r % Rs;
  int pos = -1, seq = 0;
  __shared__ int s_rpos;
  int rpos = 0;                      // position the rotary embedding uses
  unsigned long long mask = 0ull;
  if (r < B * Rs) {
    seq = seq_ids[b];
    int nr = min(max(n_rows[b], 0), Rs);
    int ctx = 0;
    if (seq < 0 || seq >= max_seqs) {
      nr = 0; seq = 0;
      if (threadIdx.x == 0) atomicCAS(status, 0, LASER_ERR_INVALID_ARG);
    } else {
      ctx = seq_len[seq];
      if (ctx + nr > capacity) {
        nr = 0;
        if (threadIdx.x == 0) atomicCAS(status, 0, LASER_ERR_CAPACITY);
      }
    }
    if (i < nr) pos = ctx + i;
    rpos = max(pos, 0);
    if (parents && i < nr && threadIdx.x == 0) {
      int depth = 0, j = i;
      mask = 1ull << i;
      while (j > 0) {                // parents are earlier rows: at most i steps
        const int pj = parents[b * Rs + j];
        if (pj < 0 || pj >= j) { atomicCAS(status, 0, LASER_ERR_INVALID_ARG); break; }
        j = pj;
        mask |= 1ull << j;
        ++depth;
      }
      rpos = ctx + depth;
    }
    if (i == 0 && threadIdx.x == 0) { row_ctx[b] = ctx; row_n[b] = nr; }
  }
  if (threadIdx.x == 0) { row_pos[r] = pos; row_seq[r] = seq; s_rpos = rpos; if (row_mask) row_mask[r] = mask; }
  __syncthreads();
  rpos = s_rpos;
  for (int j = threadIdx.x; j < half; j += blockDim.x) {
    const double inv_freq = pow(theta, -2.0 * double(j) / double(head_dim));
    double s, c;
    sincos(double(rpos) * inv_freq, &s, &c);
    rope[(size_t(r) * half + j) * 2] = float(c);
    rope[(size_t(r) * half + j) * 2 + 1] = float(s);
  }
}

__device__ __forceinline__ float block_sum(float v, float* red) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < nw; ++w) t += red[w];
  return t;
}

// Embedding gather: resid = emb[token]; xb = bf16(resid * gain of the first norm); the sum of
// squares of the row goes to tile plane 0 (the consumer GEMM turns it into the RMSNorm scale).
__global__ void __launch_bounds__(256)
embed_kernel(const int32_t* __restrict__ tokens, int R, int d, int vocab, const bf16* __restrict__ emb,
             const bf16* __restrict__ gain, float* __restrict__ resid, bf16* __restrict__ xb,
             float* __restrict__ sumsq, const int32_t* __restrict__ n_rows, int Rs, int32_t* __restrict__ row_draft,
             int split) {
  __shared__ float red[8];
  const int r = blockIdx.x;
  const int tok = r < R ? tokens[r] : -1;
  if (row_draft && threadIdx.x == 0) {   // fused acceptance: the draft token that this row's distribution verifies
    int dt = -1;
    if (r < R && (r % Rs) + 1 < min(n_rows[r / Rs], Rs)) dt = tokens[r + 1];
    row_draft[r] = dt;
  }
  const bool ok = tok >= 0 && tok < vocab;
  float ss = 0.f;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    const float x = ok ? __bfloat162float(emb[size_t(tok) * d + j]) : 0.f;
    resid[size_t(r) * d + j] = x;
    const float y = x * __bfloat162float(gain[j]);
    const bf16 hi = __float2bfloat16(y);
    if (split) {   // operand as a hi + lo pair: [hi | lo] in a row of 2 d
      xb[size_t(r) * (2 * d) + j] = hi;
      xb[size_t(r) * (2 * d) + d + j] = __float2bfloat16(y - __bfloat162float(hi));
    } else {
      xb[size_t(r) * d + j] = hi;
    }
    ss += x * x;
  }
  ss = block_sum(ss, red);
  if (threadIdx.x == 0) sumsq[r] = ss;
}

// Causal attention of the step's rows over the paged cache: grid (sequence, head).
// Scores of one row go to shared memory, softmax in fp32, then thread d accumulates
// sum_j p_j V[j][d].
// qf (optional): the queries in fp32 instead of q; out_split: the output as hi + lo bf16 pairs, rows of 2 H dh.
__global__ void __launch_bounds__(128)
attention_kernel(const bf16* __restrict__ q, const float* __restrict__ qf, int out_split, const int32_t* __restrict__ seq_ids,
                 const int32_t* __restrict__ row_ctx, const int32_t* __restrict__ row_n, int Rs, int H,
                 int Hkv, int dh, const int32_t* __restrict__ page_table, int pages_per_seq,
                 const bf16* __restrict__ pages_layer, size_t page_elems, bf16* __restrict__ out,
                 const unsigned long long* __restrict__ row_mask) {
  extern __shared__ float smem[];
  float* s_q = smem;            // [dh]
  float* s_sc = smem + dh;      // [ctx + rows]
  __shared__ float red[4];
  const int b = blockIdx.x, h = blockIdx.y, hk = h / (H / Hkv);
  const int nr = row_n[b], ctx = row_ctx[b];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int32_t* pt = page_table + size_t(seq_ids[b]) * pages_per_seq;
  const float scale = rsqrtf(float(dh));
  for (int i = 0; i < Rs; ++i) {
    const size_t r = size_t(b) * Rs + i;
    bf16* o = out + r * H * dh * (out_split ? 2 : 1) + size_t(h) * dh;
    bf16* o_lo = o + size_t(H) * dh;
    if (i >= nr) {
      for (int d = tid; d < dh; d += 128) {
        o[d] = __float2bfloat16(0.f);
        if (out_split) o_lo[d] = __float2bfloat16(0.f);
      }
      continue;
    }
    __syncthreads();
    for (int d = tid; d < dh; d += 128)
      s_q[d] = (qf ? qf[r * H * dh + size_t(h) * dh + d] : __bfloat162float(q[r * H * dh + size_t(h) * dh + d])) * scale;
    __syncthreads();
    // chain: the cache and rows 0..i; token tree: the cache and the rows of the mask
    const int n = row_mask ? ctx + nr : ctx + i + 1;
    const unsigned long long vis = row_mask ? row_mask[r] : ~0ull;
    float mx = -INFINITY;
    for (int j = tid; j < n; j += 128) {
      const bf16* kp = pages_layer + size_t(pt[j / 16]) * page_elems + size_t(hk) * 16 * dh + size_t(j % 16) * dh;
      float s = 0.f;
      for (int d = 0; d < dh; d += 8) {
        const uint4 u = *reinterpret_cast<const uint4*>(kp + d);
        const bf16* e = reinterpret_cast<const bf16*>(&u);
#pragma unroll
        for (int x = 0; x < 8; ++x) s += s_q[d + x] * __bfloat162float(e[x]);
      }
      if (j >= ctx && !((vis >> (j - ctx)) & 1ull)) s = -INFINITY;
      s_sc[j] = s;
      mx = fmaxf(mx, s);
    }
    for (int o2 = 16; o2; o2 >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o2));
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    float sum = 0.f;
    for (int j = tid; j < n; j += 128) {
      const float e = __expf(s_sc[j] - mx);
      s_sc[j] = e;
      sum += e;
    }
    for (int o2 = 16; o2; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    sum = red[0] + red[1] + red[2] + red[3];
    for (int d = tid; d < dh; d += 128) {
      float acc = 0.f;
      for (int j = 0; j < n; ++j) {
        const bf16* vp = pages_layer + size_t(pt[j / 16]) * page_elems + (size_t(Hkv) + hk) * 16 * dh + size_t(j % 16) * dh;
        acc += s_sc[j] * __bfloat162float(vp[d]);
      }
      const float y = acc / sum;
      o[d] = __float2bfloat16(y);
      if (out_split) o_lo[d] = __float2bfloat16(y - __bfloat162float(o[d]));
    }
  }
}

// K/V copy between contiguous [n, Hkv*dh] arrays and the pages of one sequence and layer.
__global__ void kv_copy_kernel(bf16* __restrict__ pages_layer, size_t page_elems, const int32_t* __restrict__ pt,
                               int Hkv, int dh, int pos0, int n, bf16* __restrict__ k, bf16* __restrict__ v,
                               int to_pages) {
  const int w = Hkv * dh;
  for (size_t idx = size_t(blockIdx.x) * blockDim.x + threadIdx.x; idx < size_t(n) * w;
       idx += size_t(gridDim.x) * blockDim.x) {
    const int t = int(idx / w), c = int(idx % w), h = c / dh, d = c % dh;
    const int pos = pos0 + t;
    bf16* kp = pages_layer + size_t(pt[pos / 16]) * page_elems + size_t(h) * 16 * dh + size_t(pos % 16) * dh + d;
    bf16* vp = kp + size_t(Hkv) * 16 * dh;
    if (to_pages) { *kp = k[idx]; *vp = v[idx]; } else { k[idx] = *kp; v[idx] = *vp; }
  }
}

__global__ void set_len_kernel(int32_t* __restrict__ seq_len, const int32_t* __restrict__ src, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) seq_len[i] = src[i];
}

template <typename T>
laser_status model_alloc(laser_model* m, T** p, size_t count) {
  LASER_CUDA(cudaMalloc(reinterpret_cast<void**>(p), std::max<size_t>(count, 1) * sizeof(T)));
  LASER_CUDA(cudaMemset(*p, 0, std::max<size_t>(count, 1) * sizeof(T)));
  m->owned.push_back(*p);
  return LASER_OK;
}

// Returns `first` if the pieces are adjacent in memory, else a fused device copy.
laser_status fuse_rows(laser_model* m, const void* const* pieces, const size_t* elems, int n,
                       const bf16** out) {
  bool adjacent = true;
  for (int i = 1; i < n; ++i)
    adjacent = adjacent && (static_cast<const bf16*>(pieces[i]) == static_cast<const bf16*>(pieces[i - 1]) + elems[i - 1]);
  if (adjacent) { *out = static_cast<const bf16*>(pieces[0]); return LASER_OK; }
  size_t total = 0;
  for (int i = 0; i < n; ++i) total += elems[i];
  bf16* buf = nullptr;
  LASER_TRY(model_alloc(m, &buf, total));
  size_t off = 0;
  for (int i = 0; i < n; ++i) {
    LASER_CUDA(cudaMemcpy(buf + off, pieces[i], elems[i] * sizeof(bf16), cudaMemcpyDeviceToDevice));
    off += elems[i];
  }
  *out = buf;
  return LASER_OK;
}

}  // namespace
}  // namespace laser

using namespace laser;

LASER_API laser_status laser_profile_enable(laser_model* m, int32_t on) {
  LASER_REQUIRE(m, "null model");
  m->profile = on != 0;
  return LASER_OK;
}

LASER_API laser_status laser_profile_read(laser_model* m, int32_t cls, double* ms, int64_t* launches) {
  LASER_REQUIRE(m && ms && launches && cls >= 0 && cls < 2, "bad argument");
  LASER_CUDA(cudaDeviceSynchronize());
  double total = 0;
  const size_t n = m->prof_used[cls] / 2;
  for (size_t i = 0; i < n; ++i) {
    float t = 0;
    LASER_CUDA(cudaEventElapsedTime(&t, m->prof_events[cls][2 * i], m->prof_events[cls][2 * i + 1]));
    total += t;
  }
  m->prof_used[cls] = 0;
  *ms = total; *launches = int64_t(n);
  return LASER_OK;
}

LASER_API laser_status laser_model_free(laser_model* m) {
  if (!m) return LASER_OK;
  gemm_state_free(m);
  for (auto& v : m->prof_events) for (cudaEvent_t e : v) cudaEventDestroy(e);
  for (void* p : m->owned) cudaFree(p);
  delete m;
  return LASER_OK;
}

LASER_API laser_status laser_model_create(const laser_model_cfg* cfg, const laser_weights* w, laser_model** out) {
  LASER_REQUIRE(cfg && w && out, "null argument");
  LASER_REQUIRE(cfg->n_layers >= 0 && cfg->d_model >= 16 && cfg->n_heads >= 1 && cfg->n_kv_heads >= 1 &&
                cfg->d_ffn >= 16 && cfg->vocab >= 8, "bad model shape");
  LASER_REQUIRE(cfg->n_heads % cfg->n_kv_heads == 0, "n_heads must be a multiple of n_kv_heads");
  LASER_REQUIRE(cfg->head_dim >= 16 && cfg->head_dim <= 128 && 128 % cfg->head_dim == 0,
                "head_dim = %d (must be 16, 32, 64 or 128)", cfg->head_dim);
  LASER_REQUIRE(cfg->d_model % 8 == 0 && cfg->d_ffn % 8 == 0 && cfg->vocab % 8 == 0,
                "d_model, d_ffn and vocab must be multiples of 8");
  LASER_REQUIRE(cfg->page_size == 16, "page_size must be 16");
  LASER_REQUIRE(cfg->max_draft >= 0 && cfg->max_draft <= 63 && cfg->max_batch >= 1, "max_draft / max_batch");
  LASER_REQUIRE(w->tok_emb && w->lm_head && w->final_norm, "null weight");
  // the epilogues read four norm gains at a time
  LASER_REQUIRE((reinterpret_cast<uintptr_t>(w->final_norm) & 7) == 0, "final_norm must be 8-byte aligned");
  for (int l = 0; l < cfg->n_layers; ++l)
    LASER_REQUIRE(w->attn_norm[l] && w->ffn_norm[l] && (reinterpret_cast<uintptr_t>(w->attn_norm[l]) & 7) == 0 &&
                  (reinterpret_cast<uintptr_t>(w->ffn_norm[l]) & 7) == 0, "norm gains of layer %d must be non-null and 8-byte aligned", l);
  laser_model* m = new laser_model();
  struct Guard { laser_model* p; ~Guard() { if (p) laser_model_free(p); } } guard{m};
  m->cfg = *cfg;
  m->rows_per_seq = cfg->max_draft + 1;
  m->R = cfg->max_batch * m->rows_per_seq;
  m->R_pad = ceil_div(m->R, 16) * 16;
  const int d = cfg->d_model, f = cfg->d_ffn, L = cfg->n_layers;
  m->dq = cfg->n_heads * cfg->head_dim;
  m->dkv = cfg->n_kv_heads * cfg->head_dim;
  m->dqkv = m->dq + 2 * m->dkv;
  m->tok_emb = static_cast<const bf16*>(w->tok_emb);
  m->lm_head = static_cast<const bf16*>(w->lm_head);
  m->final_norm = static_cast<const bf16*>(w->final_norm);
  for (int l = 0; l < L; ++l) {
    LASER_REQUIRE(w->wq[l] && w->wk[l] && w->wv[l] && w->wo[l] && w->w_gate[l] && w->w_up[l] && w->w_down[l] &&
                  w->attn_norm[l] && w->ffn_norm[l], "null weight in layer %d", l);
    const void* qkv[3] = {w->wq[l], w->wk[l], w->wv[l]};
    const size_t qkv_e[3] = {size_t(m->dq) * d, size_t(m->dkv) * d, size_t(m->dkv) * d};
    const bf16* fused = nullptr;
    LASER_TRY(fuse_rows(m, qkv, qkv_e, 3, &fused));
    m->wqkv.push_back(fused);
    const void* gu[2] = {w->w_gate[l], w->w_up[l]};
    const size_t gu_e[2] = {size_t(f) * d, size_t(f) * d};
    LASER_TRY(fuse_rows(m, gu, gu_e, 2, &fused));
    m->wgu.push_back(fused);
    m->wo.push_back(static_cast<const bf16*>(w->wo[l]));
    m->wdown.push_back(static_cast<const bf16*>(w->w_down[l]));
    m->attn_norm.push_back(static_cast<const bf16*>(w->attn_norm[l]));
    m->ffn_norm.push_back(static_cast<const bf16*>(w->ffn_norm[l]));
  }
  const size_t Rp = size_t(m->R_pad);
  LASER_TRY(model_alloc(m, &m->resid, Rp * d));
  m->precise = cfg->precise != 0;
  const size_t pair = m->precise ? 2 : 1;     // hi + lo parts side by side in a row
  LASER_TRY(model_alloc(m, &m->xn, Rp * d * pair));
  LASER_TRY(model_alloc(m, &m->q, Rp * m->dq));
  if (m->precise) LASER_TRY(model_alloc(m, &m->qf, Rp * m->dq));
  LASER_TRY(model_alloc(m, &m->attn, Rp * m->dq * pair));
  LASER_TRY(model_alloc(m, &m->act, Rp * f * pair));
  LASER_TRY(model_alloc(m, &m->sumsq, size_t(ceil_div(d, 128)) * Rp));
  LASER_TRY(model_alloc(m, &m->rope, Rp * (cfg->head_dim / 2) * 2));
  LASER_TRY(model_alloc(m, &m->row_pos, Rp));
  LASER_TRY(model_alloc(m, &m->row_seq, Rp));
  LASER_TRY(model_alloc(m, &m->row_ctx, size_t(cfg->max_batch)));
  LASER_TRY(model_alloc(m, &m->row_n, size_t(cfg->max_batch)));
  LASER_TRY(model_alloc(m, &m->row_mask, size_t(m->R_pad)));
  const size_t v_tiles = size_t(ceil_div(cfg->vocab, 128));
  LASER_TRY(model_alloc(m, &m->row_draft, Rp));
  LASER_TRY(model_alloc(m, &m->draft_logit, Rp));
  LASER_TRY(model_alloc(m, &m->top_val, Rp * v_tiles));
  LASER_TRY(model_alloc(m, &m->top_idx, Rp * v_tiles));
  LASER_TRY(model_alloc(m, &m->tile_sum, Rp * v_tiles));
  LASER_TRY(model_alloc(m, &m->status, size_t(1)));
  guard.p = nullptr;
  *out = m;
  return LASER_OK;
}

LASER_API laser_status laser_kv_free(laser_kv* kv) {
  if (!kv) return LASER_OK;
  cudaFree(kv->pages); cudaFree(kv->page_table); cudaFree(kv->seq_len);
  delete kv;
  return LASER_OK;
}

LASER_API laser_status laser_kv_create(const laser_model* m, int32_t max_seqs, int64_t n_pages, laser_kv** out) {
  LASER_REQUIRE(m && out, "null argument");
  LASER_REQUIRE(max_seqs >= 1 && n_pages >= max_seqs, "max_seqs = %d, n_pages = %lld", max_seqs, (long long)n_pages);
  laser_kv* kv = new laser_kv();
  struct Guard { laser_kv* p; ~Guard() { if (p) laser_kv_free(p); } } guard{kv};
  kv->n_layers = m->cfg.n_layers; kv->n_kv_heads = m->cfg.n_kv_heads; kv->head_dim = m->cfg.head_dim;
  kv->max_seqs = max_seqs; kv->n_pages = n_pages;
  kv->pages_per_seq = int32_t(std::min<int64_t>(n_pages / max_seqs, 1 << 20));
  const size_t elems = std::max<size_t>(1, size_t(kv->n_layers) * kv->layer_elems());
  LASER_CUDA(cudaMalloc(reinterpret_cast<void**>(&kv->pages), elems * sizeof(__nv_bfloat16)));
  // masked keys still enter P*V with weight 0, so the pages must never hold NaN/Inf patterns
  LASER_CUDA(cudaMemset(kv->pages, 0, elems * sizeof(__nv_bfloat16)));
  LASER_CUDA(cudaMalloc(reinterpret_cast<void**>(&kv->page_table), size_t(max_seqs) * kv->pages_per_seq * 4));
  LASER_CUDA(cudaMalloc(reinterpret_cast<void**>(&kv->seq_len), size_t(max_seqs) * 4));
  LASER_CUDA(cudaMemset(kv->seq_len, 0, size_t(max_seqs) * 4));
  std::vector<int32_t> table(size_t(max_seqs) * kv->pages_per_seq);
  for (int s = 0; s < max_seqs; ++s)
    for (int j = 0; j < kv->pages_per_seq; ++j) table[size_t(s) * kv->pages_per_seq + j] = j * max_seqs + s;
  LASER_CUDA(cudaMemcpy(kv->page_table, table.data(), table.size() * 4, cudaMemcpyHostToDevice));
  const uint64_t map_rows = uint64_t(kv->n_layers) * uint64_t(n_pages) * 2 * kv->n_kv_heads * 16;
  if (kv->head_dim % 64 == 0 && map_rows > 0 && map_rows < (uint64_t(1) << 31)) {
    LASER_TRY(encode_bf16_2d(&kv->pages_map, kv->pages, map_rows, uint64_t(kv->head_dim), 16));
    kv->has_pages_map = true;
  }
  guard.p = nullptr;
  *out = kv;
  return LASER_OK;
}

LASER_API laser_status laser_kv_set_page_table(laser_kv* kv, const int32_t* table) {
  LASER_REQUIRE(kv && table, "null argument");
  const size_t n = size_t(kv->max_seqs) * kv->pages_per_seq;
  std::vector<uint8_t> seen(size_t(kv->n_pages), 0);
  for (size_t i = 0; i < n; ++i) {
    LASER_REQUIRE(table[i] >= 0 && table[i] < kv->n_pages && !seen[table[i]], "page table entry %zu invalid or repeated", i);
    seen[table[i]] = 1;
  }
  LASER_CUDA(cudaDeviceSynchronize());
  LASER_CUDA(cudaMemcpy(kv->page_table, table, n * 4, cudaMemcpyHostToDevice));
  return LASER_OK;
}

LASER_API laser_status laser_kv_set_len(laser_kv* kv, const int32_t* seq_ids, const int32_t* lens, int32_t n, void* stream) {
  LASER_REQUIRE(kv && seq_ids && lens && n >= 0, "bad argument");
  for (int i = 0; i < n; ++i) {
    LASER_REQUIRE(seq_ids[i] >= 0 && seq_ids[i] < kv->max_seqs, "seq id %d out of range", seq_ids[i]);
    LASER_REQUIRE(lens[i] >= 0 && lens[i] <= kv->capacity_tokens(), "length %d out of range", lens[i]);
  }
  for (int i = 0; i < n; ++i)
    LASER_CUDA(cudaMemcpyAsync(kv->seq_len + seq_ids[i], lens + i, 4, cudaMemcpyHostToDevice, as_stream(stream)));
  LASER_CUDA(cudaStreamSynchronize(as_stream(stream)));
  return LASER_OK;
}

LASER_API laser_status laser_kv_reset(laser_kv* kv, void* stream) {
  LASER_REQUIRE(kv, "null argument");
  LASER_CUDA(cudaMemsetAsync(kv->seq_len, 0, size_t(kv->max_seqs) * 4, as_stream(stream)));
  return LASER_OK;
}

LASER_API laser_status laser_kv_set_len_dev(laser_kv* kv, const int32_t* lens_dev, int32_t n, void* stream) {
  LASER_REQUIRE(kv && lens_dev && n >= 0 && n <= kv->max_seqs, "bad argument");
  if (n == 0) return LASER_OK;
  set_len_kernel<<<ceil_div(n, 256), 256, 0, as_stream(stream)>>>(kv->seq_len, lens_dev, n);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_kv_get_len(const laser_kv* kv, const int32_t* seq_ids, int32_t* lens, int32_t n, void* stream) {
  LASER_REQUIRE(kv && seq_ids && lens && n >= 0, "bad argument");
  for (int i = 0; i < n; ++i) LASER_REQUIRE(seq_ids[i] >= 0 && seq_ids[i] < kv->max_seqs, "seq id %d out of range", seq_ids[i]);
  for (int i = 0; i < n; ++i)
    LASER_CUDA(cudaMemcpyAsync(lens + i, kv->seq_len + seq_ids[i], 4, cudaMemcpyDeviceToHost, as_stream(stream)));
  LASER_CUDA(cudaStreamSynchronize(as_stream(stream)));
  return LASER_OK;
}

static laser_status kv_copy(const laser_kv* kv, int32_t seq, int32_t layer, int32_t pos0, int32_t n,
                            void* k, void* v, int to_pages, void* stream) {
  LASER_REQUIRE(kv && k && v, "null argument");
  LASER_REQUIRE(seq >= 0 && seq < kv->max_seqs && layer >= 0 && layer < kv->n_layers, "seq / layer out of range");
  LASER_REQUIRE(pos0 >= 0 && n >= 0 && int64_t(pos0) + n <= kv->capacity_tokens(), "positions [%d, %d) outside the sequence's pages", pos0, pos0 + n);
  if (n == 0) return LASER_OK;
  const size_t total = size_t(n) * kv->n_kv_heads * kv->head_dim;
  kv_copy_kernel<<<unsigned(std::min<size_t>(ceil_div<size_t>(total, 256), 4096)), 256, 0, as_stream(stream)>>>(
      kv->pages + size_t(layer) * kv->layer_elems(), kv->page_elems(), kv->page_table + size_t(seq) * kv->pages_per_seq,
      kv->n_kv_heads, kv->head_dim, pos0, n, static_cast<__nv_bfloat16*>(k), static_cast<__nv_bfloat16*>(v), to_pages);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_kv_import(laser_kv* kv, int32_t seq, int32_t layer, int32_t pos0, int32_t n,
                                       const void* k, const void* v, void* stream) {
  return kv_copy(kv, seq, layer, pos0, n, const_cast<void*>(k), const_cast<void*>(v), 1, stream);
}
LASER_API laser_status laser_kv_export(const laser_kv* kv, int32_t seq, int32_t layer, int32_t pos0, int32_t n,
                                       void* k, void* v, void* stream) {
  return kv_copy(kv, seq, layer, pos0, n, k, v, 0, stream);
}

LASER_API laser_status laser_check(laser_model* m, void* stream) {
  LASER_REQUIRE(m, "null model");
  int32_t st = 0;
  LASER_CUDA(cudaMemcpyAsync(&st, m->status, 4, cudaMemcpyDeviceToHost, as_stream(stream)));
  LASER_CUDA(cudaStreamSynchronize(as_stream(stream)));
  if (st != 0) {
    LASER_CUDA(cudaMemsetAsync(m->status, 0, 4, as_stream(stream)));
    set_error(st == LASER_ERR_CAPACITY ? "a sequence outgrew its KV pages"
              : st == LASER_ERR_TIMEOUT ? "a device-side wait ran out" : "a step was given a bad sequence id");
    return st;
  }
  return LASER_OK;
}

// fused: 0 = LM head stores logits (none at all if logits is null); otherwise acceptance is fused into the LM head:
// the number of largest logits kept per vocabulary tile (1..4), negative when the tile sums of exp are wanted too
static laser_status verify_impl(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                                const int32_t* parents, const int32_t* n_rows, int32_t B, int32_t Rs, float* logits, void* stream_,
                                int fused = 0);

LASER_API laser_status laser_verify_step(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                                         const int32_t* n_rows, int32_t B, float* logits, void* stream) {
  LASER_REQUIRE(m && logits, "null argument");
  return verify_impl(m, kv, seq_ids, tokens, nullptr, n_rows, B, m->rows_per_seq, logits, stream);
}

LASER_API laser_status laser_verify_step_tree(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                                              const int32_t* parents, const int32_t* n_rows, int32_t B, float* logits,
                                              void* stream) {
  LASER_REQUIRE(parents, "null argument");
  LASER_REQUIRE(m && m->rows_per_seq <= 64, "a token tree has at most 64 rows (K + 1 = %d)", m ? m->rows_per_seq : 0);
  LASER_REQUIRE(logits, "null argument");
  return verify_impl(m, kv, seq_ids, tokens, parents, n_rows, B, m->rows_per_seq, logits, stream);
}

namespace laser {
// Prompt processing (the x_<=t of Eq. 3): the same forward over B sequences with Rs rows each, any Rs
// with B * Rs inside the model's row workspace; only K and V are wanted, so the LM head is left out.
laser_status prefill_rows(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                          const int32_t* n_rows, int32_t B, int32_t Rs, cudaStream_t stream) {
  return verify_impl(m, kv, seq_ids, tokens, nullptr, n_rows, B, Rs, nullptr, stream);
}
// The verify forward whose LM head leaves, per (row, vocabulary tile), what the acceptance rule needs
// (see GemmEpilogue) in the model's buffers; logits may be null.
laser_status verify_fused(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                          const int32_t* n_rows, int32_t B, float* logits, int top_n, bool sums, cudaStream_t stream) {
  return verify_impl(m, kv, seq_ids, tokens, nullptr, n_rows, B, m->rows_per_seq, logits, stream, sums ? -top_n : top_n);
}
}  // namespace laser

// The forward over B sequences of Rs rows each; logits == nullptr: no LM head (prompt processing).
static laser_status verify_impl(laser_model* m, laser_kv* kv, const int32_t* seq_ids, const int32_t* tokens,
                                const int32_t* parents, const int32_t* n_rows, int32_t B, int32_t Rs, float* logits, void* stream_,
                                int fused) {
  LASER_REQUIRE(m && kv && seq_ids && tokens && n_rows, "null argument");
  LASER_REQUIRE(B >= 1 && Rs >= 1 && B <= m->cfg.max_batch && int64_t(B) * Rs <= m->R_pad,
                "B = %d sequences of %d rows outside the model's %d rows (max_batch = %d)", B, Rs, m->R_pad, m->cfg.max_batch);
  LASER_REQUIRE(kv->n_layers == m->cfg.n_layers && kv->n_kv_heads == m->cfg.n_kv_heads && kv->head_dim == m->cfg.head_dim,
                "cache was created for another model shape");
  // the LM head stores four logits at a time
  LASER_REQUIRE((reinterpret_cast<uintptr_t>(logits) & 15) == 0, "logits must be 16-byte aligned");
  cudaStream_t stream = as_stream(stream_);
  const laser_model_cfg& c = m->cfg;
  const int R = B * Rs, Rp = ceil_div(R, 16) * 16;
  const int d = c.d_model, f = c.d_ffn, dh = c.head_dim, H = c.n_heads, Hkv = c.n_kv_heads;
  const int capacity = int(std::min<int64_t>(kv->capacity_tokens(), INT32_MAX));

  // Every row of the workspace is (re)marked: a GEMM's last token tile may reach past this call's
  // rows, and whatever it finds there must be inactive (no cache write) and finite.
  const bool tree = parents != nullptr;
  prep_rows_kernel<<<m->R_pad, 64, 0, stream>>>(seq_ids, n_rows, parents, tree ? m->row_mask : nullptr, B, Rs, Rp, kv->seq_len, kv->max_seqs, capacity, dh / 2,
                                          double(c.rope_theta), dh, m->row_pos, m->row_seq, m->row_ctx, m->row_n,
                                          m->rope, m->status);
  const __nv_bfloat16* first_gain = c.n_layers > 0 ? m->attn_norm[0] : m->final_norm;
  embed_kernel<<<m->R_pad, 256, 0, stream>>>(tokens, R, d, c.vocab, m->tok_emb, first_gain, m->resid, m->xn, m->sumsq, n_rows, Rs,
                                             fused ? m->row_draft : nullptr, m->precise ? 1 : 0);
  count_launch(2);
  const bool use_tma_attn = attention_tma_supported(m, kv);
  const size_t attn_smem = (size_t(dh) + size_t(capacity) + 8) * sizeof(float);
  if (!use_tma_attn && attn_smem > 48 * 1024) {
    LASER_REQUIRE(attn_smem <= 200 * 1024, "KV capacity of %d tokens per sequence exceeds the attention kernel's limit", capacity);
    LASER_CUDA(cudaFuncSetAttribute(attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(attn_smem)));
  }
  const int d_tiles = ceil_div(d, 128);
  GemmEpilogue base;
  base.R_rows = m->R_pad;
  base.sumsq_ld = m->R_pad;
  base.inv_d = 1.f / float(d);
  base.eps = c.rms_eps;
  base.out_split = m->precise ? 1 : 0;
  int norm_tiles = 1;  // tile planes holding the sums of squares of the current residual
  for (int l = 0; l < c.n_layers; ++l) {
    __nv_bfloat16* pages_l = kv->pages + size_t(l) * kv->layer_elems();
    {  // QKV projection of the normalised residual; rotary embedding; Q store; cache write
      GemmEpilogue e = base;
      e.sumsq_in = m->sumsq; e.sumsq_in_tiles = norm_tiles;
      e.q = m->q; e.pages_layer = pages_l; e.page_elems = kv->page_elems(); e.page_table = kv->page_table;
      e.pages_per_seq = kv->pages_per_seq; e.row_pos = m->row_pos; e.row_seq = m->row_seq; e.rope = m->rope;
      e.H = H; e.Hkv = Hkv; e.dh = dh;
      if (m->precise) { e.a_lo_off = d; e.qf = m->qf; }
      ProfScope ps(m, 0, stream);
      LASER_TRY(gemm_fused(m, m->xn, m->wqkv[l], Rp, m->dqkv, d, EPI_QKV, e, stream));
    }
    {
      ProfScope ps(m, 1, stream);
      if (use_tma_attn) {
        LASER_TRY(attention_tma_launch(m, kv, l, seq_ids, B, Rs, tree, stream));
      } else {
        attention_kernel<<<dim3(B, H), 128, attn_smem, stream>>>(m->q, m->qf, m->precise ? 1 : 0, seq_ids, m->row_ctx, m->row_n, Rs, H, Hkv, dh,
                                                                kv->page_table, kv->pages_per_seq, pages_l,
                                                                kv->page_elems(), m->attn, tree ? m->row_mask : nullptr);
        count_launch();
      }
    }
    {  // output projection; residual add; operand and statistics of the FFN norm
      GemmEpilogue e = base;
      e.resid = m->resid; e.xb = m->xn; e.gain_next = m->ffn_norm[l]; e.sumsq_out = m->sumsq;
      if (m->precise) e.a_lo_off = m->dq;
      ProfScope ps(m, 0, stream);
      LASER_TRY(gemm_fused(m, m->attn, m->wo[l], Rp, d, m->dq, EPI_RESID, e, stream));
    }
    {  // gate and up projections of the normalised residual; SwiGLU
      GemmEpilogue e = base;
      e.sumsq_in = m->sumsq; e.sumsq_in_tiles = d_tiles;
      e.act = m->act; e.f = f;
      if (m->precise) e.a_lo_off = d;
      ProfScope ps(m, 0, stream);
      LASER_TRY(gemm_fused(m, m->xn, m->wgu[l], Rp, 2 * f, d, EPI_SWIGLU, e, stream));
    }
    {  // down projection; residual add; operand and statistics of the next norm
      GemmEpilogue e = base;
      e.resid = m->resid; e.xb = m->xn; e.sumsq_out = m->sumsq;
      e.gain_next = l + 1 < c.n_layers ? m->attn_norm[l + 1] : m->final_norm;
      if (m->precise) e.a_lo_off = f;
      ProfScope ps(m, 0, stream);
      LASER_TRY(gemm_fused(m, m->act, m->wdown[l], Rp, d, f, EPI_RESID, e, stream));
    }
    norm_tiles = d_tiles;
  }
  if (logits || fused) {  // final norm (as a row scale) and LM head straight into the caller's logits
    GemmEpilogue e = base;
    e.sumsq_in = m->sumsq; e.sumsq_in_tiles = norm_tiles;
    e.out = logits; e.ldo = c.vocab; e.R_store = R;
    if (m->precise) e.a_lo_off = d;
    if (fused) {   // ... or into what the acceptance rule needs of every (row, vocabulary tile)
      e.row_draft = m->row_draft; e.draft_logit = m->draft_logit; e.top_val = m->top_val; e.top_idx = m->top_idx;
      e.tile_sum = fused < 0 ? m->tile_sum : nullptr;
      e.top_n = fused < 0 ? -fused : fused; e.n_vtiles = ceil_div(c.vocab, 128);
    }
    ProfScope ps(m, 0, stream);
    LASER_TRY(gemm_fused(m, m->xn, m->lm_head, Rp, c.vocab, d, fused ? EPI_VERDICT : EPI_PLAIN, e, stream));
  }
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}
