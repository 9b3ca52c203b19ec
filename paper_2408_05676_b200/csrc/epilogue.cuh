// Fused epilogues of the dense contractions of the verify forward: what happens to a finished
// 128-feature x token-row accumulator tile (RMSNorm scale, rotary embedding + cache write, residual
// add + next norm's operand, SwiGLU, logits, or the acceptance rule's per-tile record).  Values that
// another SM may have written during the running kernel (the residual stream) are read past L1.
#pragma once
#include "model.cuh"

namespace laser {

using bf16 = __nv_bfloat16;
constexpr int kBM = 128;          // weight rows per tile (MMA M)
constexpr int kBK = 64;           // K elements per stage = one 128-byte swizzle span of bf16
constexpr int kVerdictRow = 132;  // floats per staged token row where one lane reads one row (16-byte reads of 8 lanes hit 8 bank groups)

__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  return make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
}

// hi = bf16(x), lo = bf16(x - hi): the pair carries about 16 significant bits of x
__device__ __forceinline__ void split4_bf16(float a, float b, float c, float d, uint2& hi, uint2& lo) {
  const __nv_bfloat162 h01 = __floats2bfloat162_rn(a, b), h23 = __floats2bfloat162_rn(c, d);
  const __nv_bfloat162 l01 = __floats2bfloat162_rn(a - __low2float(h01), b - __high2float(h01));
  const __nv_bfloat162 l23 = __floats2bfloat162_rn(c - __low2float(h23), d - __high2float(h23));
  hi = make_uint2(*reinterpret_cast<const uint32_t*>(&h01), *reinterpret_cast<const uint32_t*>(&h23));
  lo = make_uint2(*reinterpret_cast<const uint32_t*>(&l01), *reinterpret_cast<const uint32_t*>(&l23));
}

// ---- fused epilogues: one warp finishes one token row r of a 128-feature tile; lane l holds
//      features n0 + 4l .. 4l+3 in v.  What depends on the feature alone is worked out once per
//      thread (LaneCtx); rows are finished without branches (`live` predicates the stores), so
//      that the rows of a group interleave. ------------------------------------------------------
struct LaneCtx {
  int n;            // first of the lane's four features
  bool in_range;    // n < N (N is a multiple of 8: then all four features are valid)
  bool vec_out;     // EPI_PLAIN: the four results may be stored as one float4
  // EPI_QKV
  int kind;         // 0 = Q, 1 = K, 2 = V
  int idx;          // offset of the feature inside its head
  int shift;        // lanes between a feature and its rotation partner
  float sg;         // sign of the partner's term
  size_t kv_off;    // offset of (K or V, head, idx) inside a page
  int rope_off;     // offset of the lane's first (cos, sin) pair inside a row of the table
};

template <int EPI>
__device__ __forceinline__ LaneCtx make_lane_ctx(const GemmEpilogue& e, int n0, int lane, int N) {
  LaneCtx c;
  c.n = n0 + 4 * lane;
  c.in_range = c.n < N;
  c.vec_out = c.n + 3 < N && (e.ldo & 3) == 0;
  c.kind = 0; c.idx = 0; c.shift = 0; c.sg = 0.f; c.kv_off = 0; c.rope_off = 0;
  if (EPI == EPI_QKV) {
    const int dh = e.dh, half = dh >> 1, dq = e.H * dh, dkv = e.Hkv * dh;
    c.shift = dh >> 3;
    c.kind = c.n < dq ? 0 : (c.n < dq + dkv ? 1 : 2);
    c.idx = c.n % dh;          // four consecutive features stay inside one half of one head
    c.sg = c.idx < half ? -1.f : 1.f;
    c.rope_off = (c.idx % half) * 2;
    if (c.kind) {
      const int h = (c.n - dq - (c.kind - 1) * dkv) / dh;
      c.kv_off = (size_t(c.kind - 1) * e.Hkv + h) * 16 * dh + c.idx;
    }
  }
  return c;
}

__device__ __forceinline__ void epi_plain(const GemmEpilogue& e, const LaneCtx& c, int r, bool live, float4 v, float rstd, int N) {
  if (!live || r >= e.R_store) return;
  float* o = e.out + size_t(r) * e.ldo + c.n;
  v.x *= rstd; v.y *= rstd; v.z *= rstd; v.w *= rstd;
  if (c.vec_out) {
    *reinterpret_cast<float4*>(o) = v;
  } else {
    if (c.n < N) o[0] = v.x;
    if (c.n + 1 < N) o[1] = v.y;
    if (c.n + 2 < N) o[2] = v.z;
    if (c.n + 3 < N) o[3] = v.w;
  }
}

// Order-preserving map of finite floats (and infinities) onto unsigned integers, and back
__device__ __forceinline__ uint32_t f32_to_ordered(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_f32(uint32_t o) {
  return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}

// Acceptance fused into the LM head (Eq. 4, Eq. 7, Eq. 8): the warp holds the 128 logits of (row r, vocabulary
// tile wt).  It leaves the tile's top_n largest logits with their token ids (equal logits: smaller id first), the
// tile's sum of exp(l - tile max) where the rule needs a probability, and - from the tile that holds it - the logit
// of the row's draft token.  From these a second, small kernel takes the row's arg max, the draft's rank among the
// first top_n and its softmax probability without a row of logits ever being stored.  The reductions are warp-wide
// integer max / min over order-preserving keys: exact, the same from run to run.
__device__ __forceinline__ void epi_verdict(const GemmEpilogue& e, const LaneCtx& c, int r, bool live, int lane, float4 v,
                                            float rstd, int N, int wt, int draft) {
  float x[4] = {v.x * rstd, v.y * rstd, v.z * rstd, v.w * rstd};
  live = live && r < e.R_store;
  if (e.out && live) {
    float* o = e.out + size_t(r) * e.ldo + c.n;
    if (c.vec_out) {
      *reinterpret_cast<float4*>(o) = make_float4(x[0], x[1], x[2], x[3]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) if (c.n + i < N) o[i] = x[i];
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (x[i] == 0.f) x[i] = 0.f;                 // -0 and +0 are one value and must map to one key
    if (c.n + i >= N) x[i] = -INFINITY;          // beyond the vocabulary
  }
  const int off = draft - c.n;          // `draft` is the row's draft token (-1: none), read before the tile was ready
  if (live && draft >= 0 && off >= 0 && off < 4 && c.n + off < N) e.draft_logit[r] = off == 0 ? x[0] : off == 1 ? x[1] : off == 2 ? x[2] : x[3];
  float tv[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
  int ti[4] = {0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff};
  uint32_t taken = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (q < e.top_n) {   // uniform over the launch
      float bv = -INFINITY;
      int bi = 0x7fffffff, bslot = -1;
#pragma unroll
      for (int i = 0; i < 4; ++i)   // ids ascend with i: a strict comparison keeps the smaller id on ties
        if (!((taken >> i) & 1u) && c.n + i < N && (bslot < 0 || x[i] > bv)) { bv = x[i]; bi = c.n + i; bslot = i; }
      const uint32_t key = bslot < 0 ? 0u : f32_to_ordered(bv);
      const uint32_t best = __reduce_max_sync(0xffffffffu, key);
      const int who = __reduce_min_sync(0xffffffffu, (key == best && bslot >= 0) ? bi : 0x7fffffff);
      if (bslot >= 0 && bi == who) taken |= 1u << bslot;
      if (who != 0x7fffffff) { tv[q] = ordered_to_f32(best); ti[q] = who; }
    }
  }
  float s = 0.f;
  if (e.tile_sum) {
#pragma unroll
    for (int i = 0; i < 4; ++i) if (c.n + i < N) s += expf(x[i] - tv[0]);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  }
  if (live && lane == 0) {
    const size_t at = size_t(r) * e.n_vtiles + wt;
    e.top_val[at] = make_float4(tv[0], tv[1], tv[2], tv[3]);
    e.top_idx[at] = make_int4(ti[0], ti[1], ti[2], ti[3]);
    if (e.tile_sum) e.tile_sum[at] = s;
  }
}

// The same per (row, vocabulary tile) record as epi_verdict, for a tile staged whole in this CTA's shared memory
// (rows of kVerdictRow floats): one lane per token row walks the row's 128 logits in ascending token id, keeping
// the TOPN largest in registers (a later equal logit never displaces an earlier one: smaller id first), then sums
// exp(l - tile max) in a second walk where the rule has a probability.
template <int TOPN>
__device__ __forceinline__ void verdict_rows(const GemmEpilogue& e, uint32_t tile_smem, int NT, int r0, int n0t, int wt, int N,
                                             int warp, int lane, const float* s_rstd, const int* s_draft, bool ok) {
  const int nch = min(32, (N - n0t) >> 2);       // 16-byte chunks of the tile inside the vocabulary (N % 8 == 0)
  for (int jb = warp * 32; jb < NT; jb += 6 * 32) {
    const int j = jb + lane, r = r0 + j;
    if (j >= NT) continue;
    const bool live = ok && r < e.R_store;
    const float rstd = s_rstd[j];
    const uint32_t row = tile_smem + uint32_t(j) * (kVerdictRow * 4);
    float tv[TOPN];
    int ti[TOPN];
#pragma unroll
    for (int q = 0; q < TOPN; ++q) { tv[q] = -INFINITY; ti[q] = 0x7fffffff; }
#pragma unroll 4
    for (int c = 0; c < nch; ++c) {
      float4 a;
      asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "r"(row + uint32_t(c) * 16));
      const float x[4] = {a.x * rstd, a.y * rstd, a.z * rstd, a.w * rstd};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (x[i] > tv[TOPN - 1]) {
          tv[TOPN - 1] = x[i]; ti[TOPN - 1] = n0t + 4 * c + i;
#pragma unroll
          for (int q = TOPN - 1; q > 0; --q)
            if (tv[q] > tv[q - 1]) {
              const float fv = tv[q]; tv[q] = tv[q - 1]; tv[q - 1] = fv;
              const int fi = ti[q]; ti[q] = ti[q - 1]; ti[q - 1] = fi;
            }
        }
      }
    }
    float s = 0.f;
    if (e.tile_sum) {
#pragma unroll 4
      for (int c = 0; c < nch; ++c) {
        float4 a;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "r"(row + uint32_t(c) * 16));
        s += (__expf(a.x * rstd - tv[0]) + __expf(a.y * rstd - tv[0])) + (__expf(a.z * rstd - tv[0]) + __expf(a.w * rstd - tv[0]));
      }
    }
    if (!live) continue;
    const int off = s_draft[j] - n0t;
    if (off >= 0 && off < 4 * nch) {
      float dl;
      asm volatile("ld.shared.f32 %0, [%1];" : "=f"(dl) : "r"(row + uint32_t(off) * 4));
      e.draft_logit[r] = dl * rstd;
    }
    const size_t at = size_t(r) * e.n_vtiles + wt;
    e.top_val[at] = make_float4(tv[0], TOPN > 1 ? tv[TOPN > 1 ? 1 : 0] : -INFINITY, TOPN > 2 ? tv[TOPN > 2 ? 2 : 0] : -INFINITY,
                                TOPN > 3 ? tv[TOPN > 3 ? 3 : 0] : -INFINITY);
    e.top_idx[at] = make_int4(ti[0], TOPN > 1 ? ti[TOPN > 1 ? 1 : 0] : 0x7fffffff, TOPN > 2 ? ti[TOPN > 2 ? 2 : 0] : 0x7fffffff,
                              TOPN > 3 ? ti[TOPN > 3 ? 3 : 0] : 0x7fffffff);
    if (e.tile_sum) e.tile_sum[at] = s;
  }
}

// resid += acc; xb = bf16(resid * gain of the next norm); per-tile sum of squares for that norm
__device__ __forceinline__ void epi_resid(const GemmEpilogue& e, const LaneCtx& c, int r, bool live, int lane, float4 v, int N,
                                          int tile, float4 x, uint2 g2) {
  float ss = 0.f;
  x.x += v.x; x.y += v.y; x.z += v.z; x.w += v.w;
  if (live && c.in_range) {
    *reinterpret_cast<float4*>(e.resid + size_t(r) * N + c.n) = x;
    const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&g2.x), g23 = *reinterpret_cast<const __nv_bfloat162*>(&g2.y);
    const float y0 = x.x * __low2float(g01), y1 = x.y * __high2float(g01), y2 = x.z * __low2float(g23), y3 = x.w * __high2float(g23);
    if (e.out_split) {
      uint2 hi, lo;
      split4_bf16(y0, y1, y2, y3, hi, lo);
      *reinterpret_cast<uint2*>(e.xb + size_t(r) * (2 * N) + c.n) = hi;
      *reinterpret_cast<uint2*>(e.xb + size_t(r) * (2 * N) + N + c.n) = lo;
    } else {
      *reinterpret_cast<uint2*>(e.xb + size_t(r) * N + c.n) = pack4_bf16(y0, y1, y2, y3);
    }
    ss = x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
  }
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (live && lane == 0) e.sumsq_out[size_t(tile) * e.sumsq_ld + r] = ss;
}

// Tile rows 0..63 = gate features f0.., rows 64..127 = up features f0..: lanes 0-15 hold four
// gate values each, lanes 16-31 the four up values of the same features.  Each pair of lanes
// (l, l+16) trades two values, so that every lane finishes two features: act = silu(g) * u.
__device__ __forceinline__ void epi_swiglu(const GemmEpilogue& e, int r, bool live, int f0, int lane, float4 v, float rstd) {
  const bool lo = lane < 16;
  const float t0 = __shfl_xor_sync(0xffffffffu, lo ? v.z : v.x, 16);
  const float t1 = __shfl_xor_sync(0xffffffffu, lo ? v.w : v.y, 16);
  const float g0 = (lo ? v.x : t0) * rstd, g1 = (lo ? v.y : t1) * rstd;
  const float u0 = (lo ? t0 : v.z) * rstd, u1 = (lo ? t1 : v.w) * rstd;
  const int fidx = f0 + 4 * (lane & 15) + (lo ? 0 : 2);
  if (live && fidx < e.f) {  // f is a multiple of 8 (checked on the host)
    const float a0 = __fdividef(g0, 1.f + __expf(-g0)) * u0, a1 = __fdividef(g1, 1.f + __expf(-g1)) * u1;
    const __nv_bfloat162 a = __floats2bfloat162_rn(a0, a1);
    if (e.out_split) {
      *reinterpret_cast<__nv_bfloat162*>(e.act + size_t(r) * (2 * e.f) + fidx) = a;
      *reinterpret_cast<__nv_bfloat162*>(e.act + size_t(r) * (2 * e.f) + e.f + fidx) =
          __floats2bfloat162_rn(a0 - __low2float(a), a1 - __high2float(a));
    } else {
      *reinterpret_cast<__nv_bfloat162*>(e.act + size_t(r) * e.f + fidx) = a;
    }
  }
}

// rotary embedding of Q and K (pair i, i + dh/2), bf16 rounding, Q store, K/V page write
__device__ __forceinline__ void epi_qkv(const GemmEpilogue& e, const LaneCtx& c, int r, bool live, float4 v, float rstd,
                                        int pos, int page, float4 cs01, float4 cs23) {
  v.x *= rstd; v.y *= rstd; v.z *= rstd; v.w *= rstd;
  float4 pv;
  pv.x = __shfl_xor_sync(0xffffffffu, v.x, c.shift); pv.y = __shfl_xor_sync(0xffffffffu, v.y, c.shift);
  pv.z = __shfl_xor_sync(0xffffffffu, v.z, c.shift); pv.w = __shfl_xor_sync(0xffffffffu, v.w, c.shift);
  float4 y = v;
  if (c.kind < 2) {
    y.x = v.x * cs01.x + c.sg * pv.x * cs01.y;
    y.y = v.y * cs01.z + c.sg * pv.y * cs01.w;
    y.z = v.z * cs23.x + c.sg * pv.z * cs23.y;
    y.w = v.w * cs23.z + c.sg * pv.w * cs23.w;
  }
  if (!live || !c.in_range) return;
  if (c.kind == 0) {
    if (pos < 0) y = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e.qf) *reinterpret_cast<float4*>(e.qf + size_t(r) * (e.H * e.dh) + c.n) = y;
    else *reinterpret_cast<uint2*>(e.q + size_t(r) * (e.H * e.dh) + c.n) = pack4_bf16(y.x, y.y, y.z, y.w);
  } else if (pos >= 0) {
    bf16* dst = e.pages_layer + size_t(page) * e.page_elems + c.kv_off + size_t(pos & 15) * e.dh;
    *reinterpret_cast<uint2*>(dst) = pack4_bf16(y.x, y.y, y.z, y.w);
  }
}

}  // namespace laser
