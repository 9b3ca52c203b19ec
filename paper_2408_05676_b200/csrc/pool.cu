// Customized Retrieval Pool (Section 3.2) and draft retrieval, Retrieve(D, tail, K) of Eq. 5
// (Section 3.3).
//
// Index: for every n in [n_min, n_max] one open-addressing hash table keyed by a 64-bit
// hash of (group, n-gram) whose entries point at a run of a position array sorted by
// (hash, position).  A run lists, ascending, every position where that n-gram ends inside
// that group - exactly the nodes a per-group trie reaches with the n-gram as prefix, with
// multiplicity.  A hash collision only merges runs; every position read at lookup time is
// checked against the actual pool tokens and the group bounds, so results never depend on
// the hash.
//
// Lookup: one warp per query.  All 32 lanes probe 32 consecutive slots (512 B, coalesced);
// the run is read 32 positions at a time, verified, and compacted; the greedy
// highest-frequency walk votes over at most 64 occurrences held two per lane.  Queries that
// need more than 64 occurrences (max_occ = 0 or > 64) go to a work list served by one CTA
// per query with a shared-memory histogram over the vocabulary.
//
// The (key, position) sort of the one-off build uses the radix sort of CUB, the header
// library shipped with the CUDA toolkit; nothing on the per-step path does.
#include <cub/device/device_radix_sort.cuh>

#include <algorithm>

#include "common.cuh"

struct laser_pool {
  int64_t n_tokens = 0;
  int32_t n_groups = 0, n_min = 0, n_max = 0;
  int32_t vocab_bound = 0;  // largest token id + 1
  int32_t* tokens = nullptr;         // dev [n_tokens]
  int64_t* group_offsets = nullptr;  // dev [n_groups + 1]
  struct Level {
    uint4* table = nullptr;    // {key.lo, key.hi, start, count}
    uint64_t mask = 0;         // slots - 1
    uint32_t* positions = nullptr;
    int64_t n_positions = 0, n_keys = 0;
  } level[9];                  // indexed by n
  int64_t device_bytes = 0;
};

namespace laser {
namespace {

constexpr int kMaxN = 8;
constexpr int kMaxK = 64;
constexpr uint64_t kEmpty = ~0ULL;

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ULL;
  x ^= x >> 27; x *= 0x94d049bb133111ebULL;
  x ^= x >> 31;
  return x;
}
__host__ __device__ __forceinline__ uint64_t key_begin(int g, int n) {
  return mix64((uint64_t(uint32_t(g)) << 8) | uint64_t(n));
}
__host__ __device__ __forceinline__ uint64_t key_push(uint64_t h, int32_t tok) {
  return mix64(h ^ (uint64_t(uint32_t(tok)) * 0x9E3779B97F4A7C15ULL));
}
__host__ __device__ __forceinline__ uint64_t key_end(uint64_t h) { return h == kEmpty ? 0 : h; }

__device__ __forceinline__ int group_of(const int64_t* __restrict__ goff, int G, int64_t p) {
  int lo = 0, hi = G;  // largest g with goff[g] <= p (skips empty groups)
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (goff[mid] <= p) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void make_keys_kernel(const int32_t* __restrict__ tok, int64_t N,
                                 const int64_t* __restrict__ goff, int G, int n,
                                 uint64_t* __restrict__ keys, uint32_t* __restrict__ pos,
                                 unsigned long long* __restrict__ n_valid, int* __restrict__ max_tok) {
  int64_t p = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  bool valid = false;
  uint64_t h = kEmpty;
  int mt = -1;
  if (p < N) {
    const int g = group_of(goff, G, p);
    valid = (p - n + 1 >= goff[g]);
    if (valid) {
      h = key_begin(g, n);
      for (int j = 0; j < n; ++j) {
        const int32_t t = tok[p - n + 1 + j];
        if (t < 0) { valid = false; break; }
        h = key_push(h, t);
      }
      h = valid ? key_end(h) : kEmpty;
    }
    mt = tok[p];
    keys[p] = h;
    pos[p] = uint32_t(p);
  }
  const unsigned ball = __ballot_sync(0xffffffffu, valid);
  for (int o = 16; o; o >>= 1) mt = max(mt, __shfl_xor_sync(0xffffffffu, mt, o));
  if ((threadIdx.x & 31) == 0) {
    if (ball) atomicAdd(n_valid, (unsigned long long)__popc(ball));
    atomicMax(max_tok, mt);
  }
}

__global__ void count_heads_kernel(const uint64_t* __restrict__ keys, int64_t n,
                                   unsigned long long* __restrict__ n_heads) {
  int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const bool head = i < n && (i == 0 || keys[i] != keys[i - 1]);
  const unsigned ball = __ballot_sync(0xffffffffu, head);
  if ((threadIdx.x & 31) == 0 && ball) atomicAdd(n_heads, (unsigned long long)__popc(ball));
}

__global__ void insert_heads_kernel(const uint64_t* __restrict__ keys, int64_t n,
                                    uint4* __restrict__ table, uint64_t mask) {
  int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t k = keys[i];
  if (i != 0 && keys[i - 1] == k) return;
  int64_t lo = i, hi = n;  // hi -> first index with a different key
  while (hi - lo > 1) {
    int64_t mid = (lo + hi) >> 1;
    if (keys[mid] == k) lo = mid; else hi = mid;
  }
  const uint32_t count = uint32_t(hi - i);
  unsigned long long* slots = reinterpret_cast<unsigned long long*>(table);
  uint64_t s = k & mask;
  for (uint64_t tries = 0; tries <= mask; ++tries, s = (s + 1) & mask) {
    const unsigned long long old = atomicCAS(&slots[2 * s], (unsigned long long)kEmpty, (unsigned long long)k);
    if (old == kEmpty) {
      reinterpret_cast<uint32_t*>(table)[4 * s + 2] = uint32_t(i);
      reinterpret_cast<uint32_t*>(table)[4 * s + 3] = count;
      return;
    }
  }
}

// ---------------------------------------------------------------------------------------
struct PoolView {
  const int32_t* tok;
  const int64_t* goff;
  int G;
  const uint4* table[kMaxN + 1];
  uint64_t mask[kMaxN + 1];
  const uint32_t* positions[kMaxN + 1];
};

struct DraftArgs {
  const int32_t* tails; const int32_t* tail_len; const int32_t* group_id;
  int B, K, n_min, n_max, min_draft, max_occ;
  int32_t* draft; int32_t* draft_len; int32_t* match_n;
  int32_t* work;  // [0] = count, [1..] = query ids for the large-run path
};

// Warp-cooperative probe: returns true and (start, count) if the key is present.
__device__ __forceinline__ bool probe(const uint4* __restrict__ table, uint64_t mask, uint64_t key,
                                      int lane, uint32_t& start, uint32_t& count) {
  uint64_t s = key & mask;
  for (uint64_t tries = 0; tries <= mask; tries += 32, s = (s + 32) & mask) {
    const uint4 e = __ldg(&table[(s + lane) & mask]);
    const uint64_t k = (uint64_t(e.y) << 32) | e.x;
    const unsigned hit = __ballot_sync(0xffffffffu, k == key);
    const unsigned empty = __ballot_sync(0xffffffffu, k == kEmpty);
    if (hit) {  // linear probing without deletions: no empty slot lies before the hit
      const int src = __ffs(hit) - 1;
      start = __shfl_sync(0xffffffffu, e.z, src);
      count = __shfl_sync(0xffffffffu, e.w, src);
      return true;
    }
    if (empty) return false;
  }
  return false;
}

__device__ __forceinline__ bool is_occurrence(const int32_t* __restrict__ tok, int64_t lo, int64_t hi,
                                              int64_t p, const int32_t* tail, int n) {
  if (p - n + 1 < lo || p >= hi) return false;
  for (int j = 0; j < n; ++j)
    if (tok[p - n + 1 + j] != tail[j]) return false;
  return true;
}

constexpr int kDraftWarps = 4;

__global__ void __launch_bounds__(kDraftWarps * 32)
draft_warp_kernel(PoolView pv, DraftArgs a) {
  __shared__ uint32_t s_occ[kDraftWarps][64];
  __shared__ int32_t s_tok[kDraftWarps][64];
  __shared__ int32_t s_cur[kDraftWarps][kMaxK];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.x * kDraftWarps + warp;
  if (q >= a.B) return;
  int32_t* out = a.draft + size_t(q) * a.K;
  const int g = a.group_id[q];
  int best_len = 0, best_n = 0;
  bool overflow = false;
  if (g >= 0 && g < pv.G) {
    const int64_t lo = pv.goff[g], hi = pv.goff[g + 1];
    const int tl = min(max(a.tail_len[q], 0), a.n_max);
    for (int n = tl; n >= a.n_min && !overflow; --n) {
      int32_t tn[kMaxN];  // the last n tail tokens, oldest first
      bool bad = false;
      uint64_t h = key_begin(g, n);
      for (int j = 0; j < n; ++j) {
        tn[j] = a.tails[size_t(q) * a.n_max + a.n_max - n + j];
        bad |= tn[j] < 0;
        h = key_push(h, tn[j]);
      }
      if (bad) continue;
      uint32_t start, count;
      if (!probe(pv.table[n], pv.mask[n], key_end(h), lane, start, count)) continue;
      const uint32_t* plist = pv.positions[n] + start;
      // gather verified occurrences, ascending, into s_occ
      const int want = (a.max_occ > 0 && a.max_occ <= 64) ? a.max_occ : 65;
      int n_occ = 0;
      for (uint32_t base = 0; base < count && n_occ < want; base += 32) {
        const uint32_t idx = base + lane;
        const int64_t p = idx < count ? int64_t(plist[idx]) : -1;
        const bool ok = idx < count && is_occurrence(pv.tok, lo, hi, p, tn, n);
        const unsigned ball = __ballot_sync(0xffffffffu, ok);
        const int slot = n_occ + __popc(ball & ((1u << lane) - 1));
        if (ok && slot < 64) s_occ[warp][slot] = uint32_t(p);
        n_occ += __popc(ball);
      }
      if (want == 65 && n_occ > 64) { overflow = true; break; }
      n_occ = min(n_occ, min(want, 64));
      if (n_occ == 0) continue;
      __syncwarp();
      // greedy highest-frequency walk
      const int64_t p0 = lane < n_occ ? int64_t(s_occ[warp][lane]) : -1;
      const int64_t p1 = lane + 32 < n_occ ? int64_t(s_occ[warp][lane + 32]) : -1;
      bool al0 = p0 >= 0, al1 = p1 >= 0;
      int len = 0;
      bool go = true;
      // The continuation of every occurrence is fetched eight depths at a time, all loads issued before
      // the first vote: the walk then costs one memory round trip per eight tokens, not one per token.
      for (int jb = 1; jb <= a.K && go; jb += 8) {
        int32_t r0[8], r1[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = jb + u;
          r0[u] = (al0 && j <= a.K && p0 + j < hi) ? pv.tok[p0 + j] : -1;
          r1[u] = (al1 && j <= a.K && p1 + j < hi) ? pv.tok[p1 + j] : -1;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = jb + u;
          if (j > a.K) { go = false; break; }
          const int32_t t0 = al0 ? r0[u] : -1, t1 = al1 ? r1[u] : -1;
          al0 = t0 >= 0; al1 = t1 >= 0;
          if (!__any_sync(0xffffffffu, al0 || al1)) { go = false; break; }
          s_tok[warp][lane] = t0;
          s_tok[warp][lane + 32] = t1;
          __syncwarp();
          uint32_t c0 = 0, c1 = 0;
          for (int e = 0; e < n_occ; ++e) {
            const int32_t x = s_tok[warp][e];
            c0 += (x == t0); c1 += (x == t1);
          }
          unsigned long long cand = 0;
          if (al0) cand = (uint64_t(c0) << 32) | uint32_t(0x7fffffff - t0);
          if (al1) cand = max(cand, (unsigned long long)((uint64_t(c1) << 32) | uint32_t(0x7fffffff - t1)));
          for (int o = 16; o; o >>= 1) cand = max(cand, __shfl_xor_sync(0xffffffffu, cand, o));
          const int32_t pick = 0x7fffffff - int32_t(uint32_t(cand));
          if (lane == 0) s_cur[warp][j - 1] = pick;
          al0 = al0 && t0 == pick; al1 = al1 && t1 == pick;
          len = j;
          __syncwarp();
        }
      }
      if (len > best_len) {
        for (int j = lane; j < len; j += 32) out[j] = s_cur[warp][j];
        best_len = len; best_n = n;
      }
      __syncwarp();
      if (best_len >= max(a.min_draft, 1)) break;
    }
  }
  if (overflow) {  // hand the whole query to the large-run kernel
    if (lane == 0) { const int w = atomicAdd(&a.work[0], 1); a.work[1 + w] = q; }
    return;
  }
  for (int j = best_len + lane; j < a.K; j += 32) out[j] = -1;
  if (lane == 0) { a.draft_len[q] = best_len; a.match_n[q] = best_len ? best_n : 0; }
}

// Temporary branches (Section 3.2): the same retrieval with the sequence's own text (prompt +
// generated tokens) searched as one more document.  Its occurrences of the tail that still have
// a following token come first in the occurrence list, the group's follow, and the list is cut
// to max_occ (1..64).  An occurrence is tagged with bit 31 when it lies in the history.
struct TempArgs {
  const int32_t* hist; const int32_t* hist_len; int64_t hist_stride;
};

__global__ void __launch_bounds__(kDraftWarps * 32)
draft_temp_kernel(PoolView pv, DraftArgs a, TempArgs t) {
  __shared__ uint32_t s_occ[kDraftWarps][64];
  __shared__ int32_t s_tok[kDraftWarps][64];
  __shared__ int32_t s_cur[kDraftWarps][kMaxK];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = blockIdx.x * kDraftWarps + warp;
  if (q >= a.B) return;
  int32_t* out = a.draft + size_t(q) * a.K;
  const int g = a.group_id[q];
  const bool has_group = g >= 0 && g < pv.G;
  const int64_t lo = has_group ? pv.goff[g] : 0, hi = has_group ? pv.goff[g + 1] : 0;
  const int32_t* h = t.hist + size_t(q) * t.hist_stride;
  const int hl = max(t.hist_len[q], 0);
  const int cap = a.max_occ;
  int best_len = 0, best_n = 0;
  const int tl = min(max(a.tail_len[q], 0), a.n_max);
  for (int n = tl; n >= a.n_min; --n) {
    int32_t tn[kMaxN];  // the last n tail tokens, oldest first
    bool bad = false;
    uint64_t key = key_begin(g, n);
    for (int j = 0; j < n; ++j) {
      tn[j] = a.tails[size_t(q) * a.n_max + a.n_max - n + j];
      bad |= tn[j] < 0;
      key = key_push(key, tn[j]);
    }
    if (bad) continue;
    int n_occ = 0;
    for (int base = 0; base + 1 < hl && n_occ < cap; base += 32) {   // the history, ascending
      const int idx = base + lane;
      bool ok = idx >= n - 1 && idx + 1 < hl;
      for (int j = 0; ok && j < n; ++j) ok = h[idx - n + 1 + j] == tn[j];
      const unsigned ball = __ballot_sync(0xffffffffu, ok);
      const int slot = n_occ + __popc(ball & ((1u << lane) - 1));
      if (ok && slot < 64) s_occ[warp][slot] = uint32_t(idx) | 0x80000000u;
      n_occ += __popc(ball);
    }
    n_occ = min(n_occ, cap);
    uint32_t start = 0, count = 0;
    if (has_group && n_occ < cap && probe(pv.table[n], pv.mask[n], key_end(key), lane, start, count)) {
      const uint32_t* plist = pv.positions[n] + start;
      for (uint32_t base = 0; base < count && n_occ < cap; base += 32) {   // the group, ascending
        const uint32_t idx = base + lane;
        const int64_t p = idx < count ? int64_t(plist[idx]) : -1;
        const bool ok = idx < count && is_occurrence(pv.tok, lo, hi, p, tn, n);
        const unsigned ball = __ballot_sync(0xffffffffu, ok);
        const int slot = n_occ + __popc(ball & ((1u << lane) - 1));
        if (ok && slot < 64) s_occ[warp][slot] = uint32_t(p);
        n_occ += __popc(ball);
      }
      n_occ = min(n_occ, cap);
    }
    if (n_occ == 0) continue;
    __syncwarp();
    // greedy highest-frequency walk over both sources
    const uint32_t e0 = lane < n_occ ? s_occ[warp][lane] : 0u, e1 = lane + 32 < n_occ ? s_occ[warp][lane + 32] : 0u;
    bool al0 = lane < n_occ, al1 = lane + 32 < n_occ;
    auto next_token = [&](uint32_t e, int j) -> int32_t {
      if (e & 0x80000000u) {
        const int idx = int(e & 0x7fffffffu) + j;
        return idx < hl ? h[idx] : -1;
      }
      const int64_t p = int64_t(e) + j;
      return p < hi ? pv.tok[p] : -1;
    };
    int len = 0;
    for (int j = 1; j <= a.K; ++j) {
      const int32_t t0 = al0 ? next_token(e0, j) : -1;
      const int32_t t1 = al1 ? next_token(e1, j) : -1;
      al0 = t0 >= 0; al1 = t1 >= 0;
      if (!__any_sync(0xffffffffu, al0 || al1)) break;
      s_tok[warp][lane] = t0;
      s_tok[warp][lane + 32] = t1;
      __syncwarp();
      uint32_t c0 = 0, c1 = 0;
      for (int e = 0; e < n_occ; ++e) {
        const int32_t x = s_tok[warp][e];
        c0 += (x == t0); c1 += (x == t1);
      }
      unsigned long long cand = 0;
      if (al0) cand = (uint64_t(c0) << 32) | uint32_t(0x7fffffff - t0);
      if (al1) cand = max(cand, (unsigned long long)((uint64_t(c1) << 32) | uint32_t(0x7fffffff - t1)));
      for (int o = 16; o; o >>= 1) cand = max(cand, __shfl_xor_sync(0xffffffffu, cand, o));
      const int32_t pick = 0x7fffffff - int32_t(uint32_t(cand));
      if (lane == 0) s_cur[warp][j - 1] = pick;
      al0 = al0 && t0 == pick; al1 = al1 && t1 == pick;
      len = j;
      __syncwarp();
    }
    if (len > best_len) {
      for (int j = lane; j < len; j += 32) out[j] = s_cur[warp][j];
      best_len = len; best_n = n;
    }
    __syncwarp();
    if (best_len >= max(a.min_draft, 1)) break;
  }
  for (int j = best_len + lane; j < a.K; j += 32) out[j] = -1;
  if (lane == 0) { a.draft_len[q] = best_len; a.match_n[q] = best_len ? best_n : 0; }
}

// Tree-based drafting (Section 3.3): the sub-tree under the matched tail, cut to its K most
// frequent nodes, listed depth-first.  One warp per query.  The occurrences (history first if
// given, then the group's, at most max_occ <= 64) each carry a continuation of up to K tokens; a
// trie node is a pair (occurrence o, depth d) = the first d tokens of o's continuation, owned by
// the first occurrence that has that prefix.  Pairwise common-prefix lengths give every node's
// frequency; nodes are taken best first by (frequency descending, depth ascending, token path
// ascending) -- along one occurrence that is by increasing depth, so each occurrence offers one
// candidate per round -- and the kept nodes are ranked into depth-first order, children by
// (frequency descending, token ascending).
constexpr int kTreeK = 32;   // nodes of a drafted tree (one lane ranks one node)

__global__ void __launch_bounds__(32)
draft_tree_kernel(PoolView pv, DraftArgs a, TempArgs t, int32_t* __restrict__ draft_parents) {
  __shared__ uint32_t s_occ[64];
  __shared__ int32_t s_cont[64][kTreeK];
  __shared__ uint8_t s_len[64], s_own[64];         // continuation length; first depth the occurrence owns
  __shared__ uint8_t s_lcp[64][64];
  __shared__ uint8_t s_freq[64][kTreeK];           // frequency of node (o, d) at [o][d-1]
  __shared__ int s_sel_o[kTreeK], s_sel_d[kTreeK], s_rank[kTreeK];
  const int lane = threadIdx.x, q = blockIdx.x;
  if (q >= a.B) return;
  int32_t* out = a.draft + size_t(q) * a.K;
  int32_t* outp = draft_parents + size_t(q) * a.K;
  const int K = a.K;
  const int g = a.group_id[q];
  const bool has_group = g >= 0 && g < pv.G;
  const int64_t lo = has_group ? pv.goff[g] : 0, hi = has_group ? pv.goff[g + 1] : 0;
  const int32_t* h = t.hist ? t.hist + size_t(q) * t.hist_stride : nullptr;
  const int hl = t.hist ? max(t.hist_len[q], 0) : 0;
  const int cap = a.max_occ;
  int best_len = 0, best_n = 0;
  const int tl = min(max(a.tail_len[q], 0), a.n_max);
  for (int n = tl; n >= a.n_min; --n) {
    int32_t tn[kMaxN];
    bool bad = false;
    uint64_t key = key_begin(g, n);
    for (int j = 0; j < n; ++j) {
      tn[j] = a.tails[size_t(q) * a.n_max + a.n_max - n + j];
      bad |= tn[j] < 0;
      key = key_push(key, tn[j]);
    }
    if (bad) continue;
    // ---- occurrences ----
    int n_occ = 0;
    for (int base = 0; base + 1 < hl && n_occ < cap; base += 32) {
      const int idx = base + lane;
      bool ok = idx >= n - 1 && idx + 1 < hl;
      for (int j = 0; ok && j < n; ++j) ok = h[idx - n + 1 + j] == tn[j];
      const unsigned ball = __ballot_sync(0xffffffffu, ok);
      const int slot = n_occ + __popc(ball & ((1u << lane) - 1));
      if (ok && slot < 64) s_occ[slot] = uint32_t(idx) | 0x80000000u;
      n_occ += __popc(ball);
    }
    n_occ = min(n_occ, cap);
    uint32_t start = 0, count = 0;
    if (has_group && n_occ < cap && probe(pv.table[n], pv.mask[n], key_end(key), lane, start, count)) {
      const uint32_t* plist = pv.positions[n] + start;
      for (uint32_t base = 0; base < count && n_occ < cap; base += 32) {
        const uint32_t idx = base + lane;
        const int64_t p = idx < count ? int64_t(plist[idx]) : -1;
        const bool ok = idx < count && is_occurrence(pv.tok, lo, hi, p, tn, n);
        const unsigned ball = __ballot_sync(0xffffffffu, ok);
        const int slot = n_occ + __popc(ball & ((1u << lane) - 1));
        if (ok && slot < 64) s_occ[slot] = uint32_t(p);
        n_occ += __popc(ball);
      }
      n_occ = min(n_occ, cap);
    }
    if (n_occ == 0) continue;
    __syncwarp();
    // ---- continuations ----
    for (int o = lane; o < n_occ; o += 32) {
      const uint32_t e = s_occ[o];
      int len = 0;
      for (int j = 1; j <= K; ++j) {
        int32_t tok;
        if (e & 0x80000000u) { const int idx = int(e & 0x7fffffffu) + j; tok = idx < hl ? h[idx] : -1; }
        else { const int64_t p = int64_t(e) + j; tok = p < hi ? pv.tok[p] : -1; }
        if (tok < 0) break;
        s_cont[o][len++] = tok;
      }
      s_len[o] = uint8_t(len);
    }
    __syncwarp();
    // ---- pairwise common-prefix lengths ----
    for (int pr = lane; pr < n_occ * n_occ; pr += 32) {
      const int o = pr / n_occ, o2 = pr % n_occ;
      const int lim = min(int(s_len[o]), int(s_len[o2]));
      int l = 0;
      while (l < lim && s_cont[o][l] == s_cont[o2][l]) ++l;
      s_lcp[o][o2] = uint8_t(l);
    }
    __syncwarp();
    // ---- node frequencies; the depth from which an occurrence owns its nodes ----
    for (int o = lane; o < n_occ; o += 32) {
      uint8_t hist_l[kTreeK + 1];
      for (int d = 0; d <= K; ++d) hist_l[d] = 0;
      int shared_before = 0;
      for (int o2 = 0; o2 < n_occ; ++o2) {
        const int l = s_lcp[o][o2];
        ++hist_l[l];
        if (o2 < o) shared_before = max(shared_before, l);
      }
      int run = 0;
      for (int d = int(s_len[o]); d >= 1; --d) { run += hist_l[d]; s_freq[o][d - 1] = uint8_t(run); }
      s_own[o] = uint8_t(shared_before + 1);
    }
    __syncwarp();
    // ---- best-first selection: each occurrence offers its shallowest untaken own node ----
    int nd0 = lane < n_occ ? int(s_own[lane]) : 255, nd1 = lane + 32 < n_occ ? int(s_own[lane + 32]) : 255;
    int m = 0;
    auto pack = [&](int o, int d) -> unsigned {   // smaller = better; ties are resolved by the token path below
      const unsigned f = s_freq[o][d - 1];
      return ((255u - f) << 16) | (unsigned(d) << 8) | unsigned(o);
    };
    auto path_less = [&](int o, int o2, int d) -> bool {   // same frequency and depth, different nodes
      const int l = s_lcp[o][o2];
      return s_cont[o][l] < s_cont[o2][l];
    };
    auto node_better = [&](unsigned x, unsigned y) -> bool {
      if (y == 0xffffffffu) return x != 0xffffffffu;
      if (x == 0xffffffffu) return false;
      if ((x >> 8) != (y >> 8)) return (x >> 8) < (y >> 8);
      const int o = int(x & 255u), o2 = int(y & 255u), d = int((x >> 8) & 255u);
      if (o == o2) return false;
      return path_less(o, o2, d);
    };
    while (m < K) {
      unsigned c0 = (nd0 <= (lane < n_occ ? int(s_len[lane]) : 0)) ? pack(lane, nd0) : 0xffffffffu;
      const unsigned c1 = (nd1 <= (lane + 32 < n_occ ? int(s_len[lane + 32]) : 0)) ? pack(lane + 32, nd1) : 0xffffffffu;
      if (node_better(c1, c0)) c0 = c1;
      for (int off = 16; off; off >>= 1) {
        const unsigned other = __shfl_xor_sync(0xffffffffu, c0, off);
        if (node_better(other, c0)) c0 = other;
      }
      if (c0 == 0xffffffffu) break;
      const int o = int(c0 & 255u), d = int((c0 >> 8) & 255u);
      if (lane == 0) { s_sel_o[m] = o; s_sel_d[m] = d; }
      if (o == lane) ++nd0;
      if (o == lane + 32) ++nd1;
      ++m;
    }
    __syncwarp();
    if (m > best_len) {
      // ---- depth-first rank of every kept node (lane k ranks node k) ----
      int rank = 0;
      const int ok_ = lane < m ? s_sel_o[lane] : 0, dk = lane < m ? s_sel_d[lane] : 0;
      if (lane < m) {
        for (int j = 0; j < m; ++j) {
          if (j == lane) continue;
          const int oj = s_sel_o[j], dj = s_sel_d[j];
          const int l = min(int(s_lcp[oj][ok_]), min(dj, dk));
          bool before;
          if (l == dj) before = true;                 // j is an ancestor of this node
          else if (l == dk) before = false;           // this node is an ancestor of j
          else {                                      // they part at depth l + 1: compare those siblings
            const int fj = s_freq[oj][l], fk = s_freq[ok_][l];
            before = fj > fk || (fj == fk && s_cont[oj][l] < s_cont[ok_][l]);
          }
          rank += before;
        }
        s_rank[lane] = rank;
      }
      __syncwarp();
      if (lane < m) {
        int parent_row = 0;
        if (dk > 1)
          for (int j = 0; j < m; ++j)
            if (s_sel_d[j] == dk - 1 && int(s_lcp[s_sel_o[j]][ok_]) >= dk - 1) { parent_row = s_rank[j] + 1; break; }
        out[rank] = s_cont[ok_][dk - 1];
        outp[rank] = parent_row;
      }
      best_len = m; best_n = n;
    }
    __syncwarp();
    if (best_len >= max(a.min_draft, 1)) break;
  }
  for (int j = best_len + lane; j < K; j += 32) { out[j] = -1; outp[j] = -1; }
  if (lane == 0) { a.draft_len[q] = best_len; a.match_n[q] = best_len ? best_n : 0; }
}

__global__ void make_tree_rows_kernel(const int32_t* __restrict__ last, const int32_t* __restrict__ draft,
                                      const int32_t* __restrict__ dpar, const int32_t* __restrict__ dlen, int B, int K,
                                      int32_t* __restrict__ tokens, int32_t* __restrict__ parents,
                                      int32_t* __restrict__ n_rows) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * (K + 1)) return;
  const int b = i / (K + 1), j = i % (K + 1);
  const int32_t lt = last[b];
  const int m = lt < 0 ? 0 : min(max(dlen[b], 0), K);
  tokens[i] = lt < 0 ? -1 : (j == 0 ? lt : (j <= m ? draft[b * K + j - 1] : -1));
  parents[i] = (lt >= 0 && j >= 1 && j <= m) ? dpar[b * K + j - 1] : -1;
  if (j == 0) n_rows[b] = lt < 0 ? 0 : 1 + m;
}

// Large-run path: one CTA per query, votes through a shared-memory histogram over the
// vocabulary.  Occurrences are streamed from the run at every depth; one is alive at depth
// j if its tokens match the tail and its continuation agrees with the draft so far.
constexpr int kBigThreads = 256;

__global__ void __launch_bounds__(kBigThreads)
draft_cta_kernel(PoolView pv, DraftArgs a, int vocab_bound) {
  extern __shared__ uint32_t s_hist[];
  __shared__ int32_t s_cur[kMaxK];
  __shared__ uint32_t s_start, s_count, s_cut;
  __shared__ int s_found;
  __shared__ unsigned long long s_red[kBigThreads / 32];
  __shared__ uint8_t s_flag[kBigThreads];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int v = tid; v < vocab_bound; v += kBigThreads) s_hist[v] = 0;
  __syncthreads();
  const int n_work = a.work[0];
  for (int w = blockIdx.x; w < n_work; w += gridDim.x) {
    const int q = a.work[1 + w];
    int32_t* out = a.draft + size_t(q) * a.K;
    const int g = a.group_id[q];
    const int64_t lo = pv.goff[g], hi = pv.goff[g + 1];
    const int tl = min(max(a.tail_len[q], 0), a.n_max);
    int best_len = 0, best_n = 0;
    for (int n = tl; n >= a.n_min; --n) {
      int32_t tn[kMaxN];
      bool bad = false;
      uint64_t h = key_begin(g, n);
      for (int j = 0; j < n; ++j) {
        tn[j] = a.tails[size_t(q) * a.n_max + a.n_max - n + j];
        bad |= tn[j] < 0;
        h = key_push(h, tn[j]);
      }
      if (bad) continue;
      if (warp == 0) {
        uint32_t st = 0, ct = 0;
        const bool f = probe(pv.table[n], pv.mask[n], key_end(h), lane, st, ct);
        if (lane == 0) { s_found = f; s_start = st; s_count = ct; s_cut = ct; }
      }
      __syncthreads();
      const bool found = s_found;
      const uint32_t count = s_count;
      const uint32_t* plist = pv.positions[n] + s_start;
      __syncthreads();
      if (!found) continue;
      if (a.max_occ > 0) {  // cut the run after the max_occ-th verified occurrence
        uint32_t total = 0;
        for (uint32_t base = 0; base < count; base += kBigThreads) {
          const uint32_t idx = base + tid;
          const bool ok = idx < count && is_occurrence(pv.tok, lo, hi, int64_t(plist[idx]), tn, n);
          s_flag[tid] = ok;
          const uint32_t c = __syncthreads_count(ok);
          if (total + c >= uint32_t(a.max_occ)) {
            if (tid == 0) {
              uint32_t run = total, i = 0;
              for (; i < kBigThreads; ++i) { run += s_flag[i]; if (run == uint32_t(a.max_occ)) break; }
              s_cut = min(count, base + i + 1);
            }
            break;
          }
          total += c;
          __syncthreads();
        }
        __syncthreads();
      }
      const uint32_t cut = s_cut;
      int len = 0;
      for (int j = 1; j <= a.K; ++j) {
        unsigned long long cand = 0;
        for (int phase = 0; phase < 3; ++phase) {
          for (uint32_t idx = tid; idx < cut; idx += kBigThreads) {
            const int64_t p = plist[idx];
            if (!is_occurrence(pv.tok, lo, hi, p, tn, n) || p + j >= hi) continue;
            bool alive = true;
            for (int c = 1; c < j; ++c) alive = alive && pv.tok[p + c] == s_cur[c - 1];
            const int32_t t = pv.tok[p + j];
            if (!alive || t < 0) continue;
            if (phase == 0) atomicAdd(&s_hist[t], 1u);
            else if (phase == 1) cand = max(cand, (unsigned long long)((uint64_t(s_hist[t]) << 32) | uint32_t(0x7fffffff - t)));
            else s_hist[t] = 0;
          }
          __syncthreads();
        }
        for (int o = 16; o; o >>= 1) cand = max(cand, __shfl_xor_sync(0xffffffffu, cand, o));
        if (lane == 0) s_red[warp] = cand;
        __syncthreads();
        cand = 0;
        for (int x = 0; x < kBigThreads / 32; ++x) cand = max(cand, s_red[x]);
        __syncthreads();
        if (cand == 0) break;
        if (tid == 0) s_cur[j - 1] = 0x7fffffff - int32_t(uint32_t(cand));
        len = j;
        __syncthreads();
      }
      if (len > best_len) {
        for (int j = tid; j < len; j += kBigThreads) out[j] = s_cur[j];
        best_len = len; best_n = n;
      }
      __syncthreads();
      if (best_len >= max(a.min_draft, 1)) break;
    }
    for (int j = best_len + tid; j < a.K; j += kBigThreads) out[j] = -1;
    if (tid == 0) { a.draft_len[q] = best_len; a.match_n[q] = best_len ? best_n : 0; }
    __syncthreads();
  }
}

__global__ void make_rows_kernel(const int32_t* __restrict__ last, const int32_t* __restrict__ draft,
                                 const int32_t* __restrict__ dlen, int B, int K,
                                 int32_t* __restrict__ tokens, int32_t* __restrict__ n_rows) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * (K + 1)) return;
  const int b = i / (K + 1), j = i % (K + 1);
  const int32_t lt = last[b];
  const int m = lt < 0 ? 0 : min(max(dlen[b], 0), K);
  tokens[i] = lt < 0 ? -1 : (j == 0 ? lt : (j <= m ? draft[b * K + j - 1] : -1));
  if (j == 0) n_rows[b] = lt < 0 ? 0 : 1 + m;
}

template <typename T>
laser_status dev_alloc(T** p, size_t count, int64_t* bytes) {
  LASER_CUDA(cudaMalloc(reinterpret_cast<void**>(p), std::max<size_t>(count, 1) * sizeof(T)));
  *bytes += int64_t(count * sizeof(T));
  return LASER_OK;
}

}  // namespace
}  // namespace laser

LASER_API laser_status laser_pool_free(laser_pool* pool) {
  if (!pool) return LASER_OK;
  cudaFree(pool->tokens);
  cudaFree(pool->group_offsets);
  for (auto& lv : pool->level) { cudaFree(lv.table); cudaFree(lv.positions); }
  delete pool;
  return LASER_OK;
}

LASER_API laser_status laser_pool_build(const int32_t* tokens, int64_t n_tokens,
                                        const int64_t* group_offsets, int32_t n_groups,
                                        int32_t n_min, int32_t n_max, void* stream_,
                                        laser_pool** out) {
  using namespace laser;
  LASER_REQUIRE(tokens && group_offsets && out, "null argument");
  LASER_REQUIRE(n_tokens >= 1 && n_tokens < (int64_t(1) << 31), "n_tokens = %lld outside [1, 2^31)", (long long)n_tokens);
  LASER_REQUIRE(n_groups >= 1, "n_groups = %d", n_groups);
  LASER_REQUIRE(n_min >= 1 && n_min <= n_max && n_max <= kMaxN, "suffix range [%d, %d] outside [1, %d]", n_min, n_max, kMaxN);
  LASER_REQUIRE(group_offsets[0] == 0 && group_offsets[n_groups] == n_tokens, "group_offsets must span [0, n_tokens]");
  for (int g = 0; g < n_groups; ++g)
    LASER_REQUIRE(group_offsets[g] <= group_offsets[g + 1], "group_offsets not ascending at %d", g);
  cudaStream_t stream = as_stream(stream_);
  laser_pool* P = new laser_pool();
  P->n_tokens = n_tokens; P->n_groups = n_groups; P->n_min = n_min; P->n_max = n_max;
  struct Guard { laser_pool* p; ~Guard() { if (p) laser_pool_free(p); } } guard{P};

  LASER_TRY(dev_alloc(&P->tokens, size_t(n_tokens), &P->device_bytes));
  LASER_TRY(dev_alloc(&P->group_offsets, size_t(n_groups) + 1, &P->device_bytes));
  LASER_CUDA(cudaMemcpyAsync(P->tokens, tokens, size_t(n_tokens) * 4, cudaMemcpyDefault, stream));
  LASER_CUDA(cudaMemcpyAsync(P->group_offsets, group_offsets, (size_t(n_groups) + 1) * 8,
                             cudaMemcpyHostToDevice, stream));

  // transient build buffers
  uint64_t *keys = nullptr, *keys_alt = nullptr;
  uint32_t *pos = nullptr, *pos_alt = nullptr;
  void* cub_tmp = nullptr;
  unsigned long long* counters = nullptr;  // [0] valid keys, [1] heads
  int* max_tok = nullptr;
  struct Tmp { void** p; ~Tmp() { cudaFree(*p); } };
  Tmp t1{(void**)&keys}, t2{(void**)&keys_alt}, t3{(void**)&pos}, t4{(void**)&pos_alt},
      t5{&cub_tmp}, t6{(void**)&counters}, t7{(void**)&max_tok};
  const size_t N = size_t(n_tokens);
  LASER_CUDA(cudaMalloc(&keys, N * 8));
  LASER_CUDA(cudaMalloc(&keys_alt, N * 8));
  LASER_CUDA(cudaMalloc(&pos, N * 4));
  LASER_CUDA(cudaMalloc(&pos_alt, N * 4));
  LASER_CUDA(cudaMalloc(&counters, 16));
  LASER_CUDA(cudaMalloc(&max_tok, 4));
  LASER_CUDA(cudaMemsetAsync(max_tok, 0xff, 4, stream));
  size_t cub_bytes = 0;
  {
    cub::DoubleBuffer<uint64_t> kb(keys, keys_alt);
    cub::DoubleBuffer<uint32_t> vb(pos, pos_alt);
    LASER_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, cub_bytes, kb, vb, int64_t(N), 0, 64, stream));
  }
  LASER_CUDA(cudaMalloc(&cub_tmp, std::max<size_t>(cub_bytes, 16)));

  const int threads = 256;
  const unsigned blocks = unsigned(ceil_div<size_t>(N, threads));
  for (int n = n_min; n <= n_max; ++n) {
    auto& lv = P->level[n];
    LASER_CUDA(cudaMemsetAsync(counters, 0, 16, stream));
    make_keys_kernel<<<blocks, threads, 0, stream>>>(P->tokens, n_tokens, P->group_offsets, n_groups, n,
                                                     keys, pos, counters, max_tok);
    cub::DoubleBuffer<uint64_t> kb(keys, keys_alt);
    cub::DoubleBuffer<uint32_t> vb(pos, pos_alt);
    LASER_CUDA(cub::DeviceRadixSort::SortPairs(cub_tmp, cub_bytes, kb, vb, int64_t(N), 0, 64, stream));
    unsigned long long h_cnt[2] = {0, 0};
    LASER_CUDA(cudaMemcpyAsync(h_cnt, counters, 8, cudaMemcpyDeviceToHost, stream));
    LASER_CUDA(cudaStreamSynchronize(stream));
    const int64_t n_valid = int64_t(h_cnt[0]);  // invalid keys (all ones) sort to the end
    count_heads_kernel<<<unsigned(ceil_div<int64_t>(std::max<int64_t>(n_valid, 1), threads)), threads, 0, stream>>>(
        kb.Current(), n_valid, counters + 1);
    LASER_CUDA(cudaMemcpyAsync(h_cnt + 1, counters + 1, 8, cudaMemcpyDeviceToHost, stream));
    LASER_CUDA(cudaStreamSynchronize(stream));
    lv.n_keys = int64_t(h_cnt[1]);
    lv.n_positions = n_valid;
    uint64_t slots = 64;
    while (slots < 2 * uint64_t(lv.n_keys)) slots <<= 1;
    lv.mask = slots - 1;
    LASER_TRY(dev_alloc(&lv.table, size_t(slots), &P->device_bytes));
    LASER_CUDA(cudaMemsetAsync(lv.table, 0xff, size_t(slots) * sizeof(uint4), stream));
    LASER_TRY(dev_alloc(&lv.positions, size_t(n_valid), &P->device_bytes));
    if (n_valid > 0) {
      LASER_CUDA(cudaMemcpyAsync(lv.positions, vb.Current(), size_t(n_valid) * 4, cudaMemcpyDeviceToDevice, stream));
      insert_heads_kernel<<<unsigned(ceil_div<int64_t>(n_valid, threads)), threads, 0, stream>>>(
          kb.Current(), n_valid, lv.table, lv.mask);
    }
    LASER_CUDA(cudaGetLastError());
    LASER_CUDA(cudaStreamSynchronize(stream));
  }
  int h_max = -1;
  LASER_CUDA(cudaMemcpyAsync(&h_max, max_tok, 4, cudaMemcpyDeviceToHost, stream));
  LASER_CUDA(cudaStreamSynchronize(stream));
  P->vocab_bound = h_max + 1;
  guard.p = nullptr;
  *out = P;
  return LASER_OK;
}

LASER_API laser_status laser_pool_info(const laser_pool* pool, int64_t* n_tokens, int64_t* n_keys,
                                       int64_t* device_bytes) {
  using namespace laser;
  LASER_REQUIRE(pool, "null pool");
  if (n_tokens) *n_tokens = pool->n_tokens;
  if (n_keys) { *n_keys = 0; for (int n = pool->n_min; n <= pool->n_max; ++n) *n_keys += pool->level[n].n_keys; }
  if (device_bytes) *device_bytes = pool->device_bytes;
  return LASER_OK;
}

LASER_API laser_status laser_draft(const laser_pool* pool, const int32_t* tails, const int32_t* tail_len,
                                   const int32_t* group_id, int32_t B, const laser_params* p,
                                   int32_t* draft, int32_t* draft_len, int32_t* match_n, void* stream_) {
  using namespace laser;
  LASER_REQUIRE(pool && tails && tail_len && group_id && p && draft && draft_len && match_n, "null argument");
  LASER_REQUIRE(B >= 0, "B = %d", B);
  LASER_REQUIRE(p->K >= 1 && p->K <= kMaxK, "K = %d outside [1, %d]", p->K, kMaxK);
  LASER_REQUIRE(p->n_min >= pool->n_min && p->n_max <= pool->n_max && p->n_min <= p->n_max,
                "suffix range [%d, %d] outside the pool's [%d, %d]", p->n_min, p->n_max, pool->n_min, pool->n_max);
  LASER_REQUIRE(p->max_occ >= 0 && p->min_draft >= 0, "max_occ / min_draft negative");
  if (B == 0) return LASER_OK;
  cudaStream_t stream = as_stream(stream_);
  PoolView pv{};
  pv.tok = pool->tokens; pv.goff = pool->group_offsets; pv.G = pool->n_groups;
  for (int n = pool->n_min; n <= pool->n_max; ++n) {
    pv.table[n] = pool->level[n].table; pv.mask[n] = pool->level[n].mask;
    pv.positions[n] = pool->level[n].positions;
  }
  const bool big = (p->max_occ == 0 || p->max_occ > 64);
  const size_t smem = size_t(pool->vocab_bound) * sizeof(uint32_t);
  if (big && smem > 200 * 1024) {
    set_error("vocabulary bound %d too large for the unlimited-occurrence path", pool->vocab_bound);
    return LASER_ERR_UNSUPPORTED;
  }
  void* scratch = nullptr;
  LASER_TRY(scratch_get(SCRATCH_DRAFT, sizeof(int32_t) * (size_t(B) + 1), &scratch));
  DraftArgs a{tails, tail_len, group_id, B, p->K, p->n_min, p->n_max, p->min_draft, p->max_occ,
              draft, draft_len, match_n, static_cast<int32_t*>(scratch)};
  LASER_CUDA(cudaMemsetAsync(scratch, 0, sizeof(int32_t), stream));
  draft_warp_kernel<<<ceil_div(B, kDraftWarps), kDraftWarps * 32, 0, stream>>>(pv, a);
  count_launch();
  if (big) {
    LASER_CUDA(cudaFuncSetAttribute(draft_cta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
    draft_cta_kernel<<<std::min(B, 296), kBigThreads, smem, stream>>>(pv, a, pool->vocab_bound);
    count_launch();
  }
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_draft_temp(const laser_pool* pool, const int32_t* tails, const int32_t* tail_len,
                                        const int32_t* group_id, const int32_t* hist, const int32_t* hist_len,
                                        int64_t hist_stride, int32_t B, const laser_params* p,
                                        int32_t* draft, int32_t* draft_len, int32_t* match_n, void* stream_) {
  using namespace laser;
  LASER_REQUIRE(pool && tails && tail_len && group_id && hist && hist_len && p && draft && draft_len && match_n, "null argument");
  LASER_REQUIRE(B >= 0 && hist_stride >= 0, "B = %d, hist_stride = %lld", B, (long long)hist_stride);
  LASER_REQUIRE(p->K >= 1 && p->K <= kMaxK, "K = %d outside [1, %d]", p->K, kMaxK);
  LASER_REQUIRE(p->n_min >= pool->n_min && p->n_max <= pool->n_max && p->n_min <= p->n_max,
                "suffix range [%d, %d] outside the pool's [%d, %d]", p->n_min, p->n_max, pool->n_min, pool->n_max);
  LASER_REQUIRE(p->max_occ >= 1 && p->max_occ <= 64 && p->min_draft >= 0,
                "max_occ = %d: the temporary-branch draft keeps 1..64 occurrences", p->max_occ);
  if (B == 0) return LASER_OK;
  cudaStream_t stream = as_stream(stream_);
  PoolView pv{};
  pv.tok = pool->tokens; pv.goff = pool->group_offsets; pv.G = pool->n_groups;
  for (int n = pool->n_min; n <= pool->n_max; ++n) {
    pv.table[n] = pool->level[n].table; pv.mask[n] = pool->level[n].mask;
    pv.positions[n] = pool->level[n].positions;
  }
  DraftArgs a{tails, tail_len, group_id, B, p->K, p->n_min, p->n_max, p->min_draft, p->max_occ,
              draft, draft_len, match_n, nullptr};
  TempArgs t{hist, hist_len, hist_stride};
  draft_temp_kernel<<<ceil_div(B, kDraftWarps), kDraftWarps * 32, 0, stream>>>(pv, a, t);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_draft_tree(const laser_pool* pool, const int32_t* tails, const int32_t* tail_len,
                                        const int32_t* group_id, const int32_t* hist, const int32_t* hist_len,
                                        int64_t hist_stride, int32_t B, const laser_params* p, int32_t* draft,
                                        int32_t* draft_parents, int32_t* draft_len, int32_t* match_n, void* stream_) {
  using namespace laser;
  LASER_REQUIRE(pool && tails && tail_len && group_id && p && draft && draft_parents && draft_len && match_n, "null argument");
  LASER_REQUIRE((hist == nullptr) == (hist_len == nullptr), "hist and hist_len come together");
  LASER_REQUIRE(B >= 0 && hist_stride >= 0, "B = %d, hist_stride = %lld", B, (long long)hist_stride);
  LASER_REQUIRE(p->K >= 1 && p->K <= kTreeK, "K = %d outside [1, %d]", p->K, kTreeK);
  LASER_REQUIRE(p->n_min >= pool->n_min && p->n_max <= pool->n_max && p->n_min <= p->n_max,
                "suffix range [%d, %d] outside the pool's [%d, %d]", p->n_min, p->n_max, pool->n_min, pool->n_max);
  LASER_REQUIRE(p->max_occ >= 1 && p->max_occ <= 64 && p->min_draft >= 0,
                "max_occ = %d: tree drafting keeps 1..64 occurrences", p->max_occ);
  if (B == 0) return LASER_OK;
  PoolView pv{};
  pv.tok = pool->tokens; pv.goff = pool->group_offsets; pv.G = pool->n_groups;
  for (int n = pool->n_min; n <= pool->n_max; ++n) {
    pv.table[n] = pool->level[n].table; pv.mask[n] = pool->level[n].mask;
    pv.positions[n] = pool->level[n].positions;
  }
  DraftArgs a{tails, tail_len, group_id, B, p->K, p->n_min, p->n_max, p->min_draft, p->max_occ,
              draft, draft_len, match_n, nullptr};
  TempArgs t{hist, hist_len, hist_stride};
  draft_tree_kernel<<<B, 32, 0, as_stream(stream_)>>>(pv, a, t, draft_parents);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_make_rows_tree(const int32_t* last_token, const int32_t* draft, const int32_t* draft_parents,
                                            const int32_t* draft_len, int32_t B, int32_t K, int32_t* tokens,
                                            int32_t* parents, int32_t* n_rows, void* stream) {
  using namespace laser;
  LASER_REQUIRE(last_token && draft && draft_parents && draft_len && tokens && parents && n_rows, "null argument");
  LASER_REQUIRE(B >= 0 && K >= 0, "B = %d, K = %d", B, K);
  if (B == 0) return LASER_OK;
  make_tree_rows_kernel<<<ceil_div(B * (K + 1), 256), 256, 0, as_stream(stream)>>>(last_token, draft, draft_parents, draft_len,
                                                                                  B, K, tokens, parents, n_rows);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

LASER_API laser_status laser_make_rows(const int32_t* last_token, const int32_t* draft,
                                       const int32_t* draft_len, int32_t B, int32_t K,
                                       int32_t* tokens, int32_t* n_rows, void* stream) {
  using namespace laser;
  LASER_REQUIRE(last_token && draft && draft_len && tokens && n_rows, "null argument");
  LASER_REQUIRE(B >= 0 && K >= 0, "B = %d, K = %d", B, K);
  if (B == 0) return LASER_OK;
  make_rows_kernel<<<ceil_div(B * (K + 1), 256), 256, 0, as_stream(stream)>>>(last_token, draft, draft_len, B, K, tokens, n_rows);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}
