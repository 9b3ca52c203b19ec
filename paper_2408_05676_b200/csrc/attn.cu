// Causal attention of the verify forward (Eq. 3 / Eq. 6, chain form of the mask): the K+1
// rows of a sequence against its paged bf16 KV cache, which already holds the rows' own K/V.
//
// One CTA per (sequence, head, group of TPC 16-row tiles).  A producer warp walks the sequence's
// page table and streams each 16-token page of K and V through TMA (128-byte swizzle) into a ring
// of shared-memory stages; four consumer warps compute S = Q K^T and O += P V with warp-level MMA
// (the rows are few, far below a tensor-memory tile), keep an online softmax with warp-shuffle row
// reductions, and merge their partial (max, sum, O) through shared memory at the end.  With up to
// 16 rows per sequence (TPC = 1) the four warps take pages round-robin; with more rows (K + 1 > 16
// or a large token tree, TPC = 2) two warps serve each of two row tiles and both tiles use the same
// staged page, so a page is still read from HBM once per 32 rows.  Every mbarrier wait is bounded.
#include "model.cuh"
#include "tma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
constexpr int kConsumers = 4;
constexpr int kAttnThreads = (kConsumers + 1) * 32;
constexpr int kStages = 4;   // a multiple of kConsumers: stage s always serves warp s % 4
constexpr int kCtasPerSm = 4;  // registers and shared memory are sized for four resident CTAs

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// PR (precise mode): the queries come in fp32 (qf) and enter the score MMA as hi + lo bf16 pairs, the probabilities
// enter the value MMA as pairs as well, and the output is written as pairs ([hi | lo] rows of 2 H DH).
template <int DH, int TPC, bool PR>
__global__ void __launch_bounds__(kAttnThreads, PR ? 3 : kCtasPerSm)
attn_paged_kernel(const __grid_constant__ CUtensorMap kvmap, const bf16* __restrict__ q, const float* __restrict__ qf,
                  const int32_t* __restrict__ seq_ids, const int32_t* __restrict__ row_ctx,
                  const int32_t* __restrict__ row_n, int Rs, int H, int Hkv,
                  const int32_t* __restrict__ page_table, int pages_per_seq, int layer_row0,
                  bf16* __restrict__ out, int32_t* __restrict__ status,
                  const unsigned long long* __restrict__ row_mask) {
  constexpr int HALVES = DH / 64;                 // 64-element (128-byte) column blocks per row
  constexpr int SUB = 16 * 128;                   // bytes of one 16-token x 64-element sub-tile
  constexpr int STAGE = 2 * HALVES * SUB;         // K then V
  constexpr int QLD = DH + 8;                     // padded row of the Q tile (elements)
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[kStages], empty_bar[kStages];
  __shared__ float s_m[kConsumers][16], s_l[kConsumers][16], s_wgt[kConsumers][16];
  __shared__ int abort_flag;

  // Programmatic dependent launch: let the next kernel start its prologue.  The kernel before this
  // one produces Q and the K/V of the step's own rows; pages that lie wholly below the committed
  // length were written by earlier steps, so the producer requests those before it waits for that
  // kernel, and the wait and the Q tile overlap their flight.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int b = blockIdx.x, h = blockIdx.y, mt = blockIdx.z;
  const int hk = h / (H / Hkv);
  const int nr = row_n[b], ctx = row_ctx[b];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NPG = kConsumers / TPC;           // consumer warps that share a row tile (they split the pages)
  const int cta_row0 = mt * 16 * TPC;              // first row of the CTA's tiles
  const int tile = TPC == 1 ? 0 : (warp & (TPC - 1)), pgrp = TPC == 1 ? warp : (warp / TPC);
  const int row0 = cta_row0 + tile * 16;           // first row of this warp's tile
  constexpr int OW = PR ? 2 : 1;                    // output row = OW x H x DH elements
  bf16* obase = out + (size_t(b) * Rs + cta_row0) * H * DH * OW + size_t(h) * DH;
  if (cta_row0 >= nr) {  // nothing active in these tiles: zero their rows
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int idx = tid; idx < 16 * TPC * DH; idx += kAttnThreads) {
      const int r = idx / DH, d = idx % DH;
      if (cta_row0 + r < Rs) {
        obase[size_t(r) * H * DH * OW + d] = __float2bfloat16(0.f);
        if (PR) obase[size_t(r) * H * DH * OW + size_t(H) * DH + d] = __float2bfloat16(0.f);
      }
    }
    return;
  }
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  uint8_t* tiles_ptr = smem_raw + (tiles - raw);
  const uint32_t q_smem = tiles + kStages * STAGE;
  bf16* q_ptr = reinterpret_cast<bf16*>(tiles_ptr + kStages * STAGE);
  const int n_keys = ctx + nr;
  const int n_pg = (n_keys + 15) >> 4;

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), TPC); }
    mbar_fence_init();
    tma_prefetch_map(&kvmap);
  }
  __syncthreads();   // barriers initialised

  if (warp == kConsumers) {  // producer
    if (lane == 0) {
      const int32_t* pt = page_table + size_t(seq_ids[b]) * pages_per_seq;
      const int n_early = min(min(ctx >> 4, n_pg), kStages);   // whole pages of older tokens that fit the ring
      bool ok = true;
      int issued = 0;
      const uint64_t kv_policy = make_policy_evict_first();   // a page is read once per step
      for (int p = 0; p < n_pg && ok; ++p) {
        const int s = p % kStages;
        if (p == n_early) asm volatile("griddepcontrol.wait;" ::: "memory");   // from here on: pages the kernel before may write
        if (p >= kStages) ok = mbar_wait(smem_u32(&empty_bar[s]), ((p / kStages) - 1) & 1, &abort_flag);
        if (!ok) break;
        const uint32_t bar = smem_u32(&full_bar[s]);
        const uint32_t dst = tiles + uint32_t(s) * STAGE;
        mbar_expect_tx(bar, STAGE);
        const int phys = pt[p];
        const int rowk = layer_row0 + ((phys * 2) * Hkv + hk) * 16;
        const int rowv = layer_row0 + ((phys * 2 + 1) * Hkv + hk) * 16;
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) {
          tma_load_2d_hint(dst + hf * SUB, &kvmap, hf * 64, rowk, bar, kv_policy);
          tma_load_2d_hint(dst + (HALVES + hf) * SUB, &kvmap, hf * 64, rowv, bar, kv_policy);
        }
        issued = p + 1;
      }
      if (!ok)
        for (int p = max(0, issued - kStages); p < issued; ++p) mbar_drain(smem_u32(&full_bar[p % kStages]), (p / kStages) & 1);
    }
    return;
  }

  // ---- consumers ----
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // Q tiles: rows of this sequence, zero beyond the active ones
  constexpr int QLO = 16 * TPC * QLD;             // PR: the lo parts of the Q tile follow the hi parts
  for (int idx = tid; idx < 16 * TPC * (DH / 8); idx += kConsumers * 32) {
    const int r = idx / (DH / 8), c = idx % (DH / 8);
    uint4 v = make_uint4(0, 0, 0, 0), vl = v;
    if (cta_row0 + r < nr) {
      const size_t at = (size_t(b) * Rs + cta_row0 + r) * H * DH + size_t(h) * DH + c * 8;
      if (PR) {
        const float4 f0 = *reinterpret_cast<const float4*>(qf + at), f1 = *reinterpret_cast<const float4*>(qf + at + 4);
        const float f[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const __nv_bfloat162 hh = __floats2bfloat162_rn(f[2 * x], f[2 * x + 1]);
          hi[x] = *reinterpret_cast<const uint32_t*>(&hh);
          lo[x] = pack_bf16(f[2 * x] - __low2float(hh), f[2 * x + 1] - __high2float(hh));
        }
        v = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        vl = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      } else {
        v = *reinterpret_cast<const uint4*>(q + at);
      }
    }
    *reinterpret_cast<uint4*>(q_ptr + r * QLD + c * 8) = v;
    if (PR) *reinterpret_cast<uint4*>(q_ptr + QLO + r * QLD + c * 8) = vl;
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  const int g = lane >> 2, qd = lane & 3;
  const float sl2 = rsqrtf(float(DH)) * 1.4426950408889634f;
  // Q fragments are re-read from shared memory for every page: keeping them in registers
  // would cost 32 registers per thread and one resident CTA per SM
  const uint32_t q_frag = q_smem + uint32_t((tile * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * QLD + (lane >> 4) * 8) * 2;
  float o[DH / 8][4];
#pragma unroll
  for (int t = 0; t < DH / 8; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  // last key each of this lane's two rows may see; inactive rows copy the last active row
  const int lim0 = ctx + min(row0 + g, nr - 1), lim1 = ctx + min(row0 + g + 8, nr - 1);
  // token tree: of the step's own rows a row sees those of its mask (ancestors and itself)
  const unsigned long long vis0 = row_mask ? row_mask[size_t(b) * Rs + min(row0 + g, nr - 1)] : 0ull;
  const unsigned long long vis1 = row_mask ? row_mask[size_t(b) * Rs + min(row0 + g + 8, nr - 1)] : 0ull;

  for (int p = pgrp; p < n_pg; p += NPG) {
    const int s = p % kStages;
    if (!mbar_wait(smem_u32(&full_bar[s]), (p / kStages) & 1, &abort_flag)) break;
    const uint32_t kbase = tiles + uint32_t(s) * STAGE, vbase = kbase + HALVES * SUB;
    float sc[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) sc[t][0] = sc[t][1] = sc[t][2] = sc[t][3] = 0.f;
    {
      const int mat = lane >> 3, key = (lane & 7) + (mat >> 1) * 8;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
        const int c = (ks & 3) * 2 + (mat & 1);
        uint32_t kb[4], qa[4];
        ldsm_x4(qa, q_frag + ks * 32);
        ldsm_x4(kb, kbase + (ks >> 2) * SUB + key * 128 + ((c ^ (key & 7)) << 4));
        mma16816(sc[0], qa, kb[0], kb[1]);
        mma16816(sc[1], qa, kb[2], kb[3]);
        if (PR) {
          ldsm_x4(qa, q_frag + QLO * 2 + ks * 32);
          mma16816(sc[0], qa, kb[0], kb[1]);
          mma16816(sc[1], qa, kb[2], kb[3]);
        }
      }
    }
    // causal mask, online softmax (rows g and g+8 of the tile)
    const int key0 = p * 16 + 2 * qd;
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int key = key0 + t * 8 + c;
        if (row_mask) {
          const int rel = key - ctx;   // >= 0: one of this step's rows (or the padding of the last page)
          if (rel >= 0 && (rel >= 64 || !((vis0 >> rel) & 1ull))) sc[t][c] = -INFINITY;
          if (rel >= 0 && (rel >= 64 || !((vis1 >> rel) & 1ull))) sc[t][2 + c] = -INFINITY;
        } else {
          if (key > lim0) sc[t][c] = -INFINITY;
          if (key > lim1) sc[t][2 + c] = -INFINITY;
        }
        mx0 = fmaxf(mx0, sc[t][c]);
        mx1 = fmaxf(mx1, sc[t][2 + c]);
      }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
    const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
    const float al0 = exp2f((m_run[0] - mu0) * sl2), al1 = exp2f((m_run[1] - mu1) * sl2);
    m_run[0] = mn0; m_run[1] = mn1;
    uint32_t pf[4], pl[4] = {0u, 0u, 0u, 0u};
    float ps0 = 0.f, ps1 = 0.f;
    {
      const float p00 = exp2f((sc[0][0] - mu0) * sl2), p01 = exp2f((sc[0][1] - mu0) * sl2);
      const float p02 = exp2f((sc[0][2] - mu1) * sl2), p03 = exp2f((sc[0][3] - mu1) * sl2);
      const float p10 = exp2f((sc[1][0] - mu0) * sl2), p11 = exp2f((sc[1][1] - mu0) * sl2);
      const float p12 = exp2f((sc[1][2] - mu1) * sl2), p13 = exp2f((sc[1][3] - mu1) * sl2);
      ps0 = p00 + p01 + p10 + p11;
      ps1 = p02 + p03 + p12 + p13;
      pf[0] = pack_bf16(p00, p01);   // row g,   keys 2q..   (k low)
      pf[1] = pack_bf16(p02, p03);   // row g+8, keys 2q..
      pf[2] = pack_bf16(p10, p11);   // row g,   keys 8+2q.. (k high)
      pf[3] = pack_bf16(p12, p13);   // row g+8, keys 8+2q..
      if (PR) {
        auto lo_of = [](uint32_t packed, float a, float b) {
          const __nv_bfloat162 hh = *reinterpret_cast<const __nv_bfloat162*>(&packed);
          return pack_bf16(a - __low2float(hh), b - __high2float(hh));
        };
        pl[0] = lo_of(pf[0], p00, p01); pl[1] = lo_of(pf[1], p02, p03);
        pl[2] = lo_of(pf[2], p10, p11); pl[3] = lo_of(pf[3], p12, p13);
      }
    }
    l_run[0] = l_run[0] * al0 + ps0;
    l_run[1] = l_run[1] * al1 + ps1;
#pragma unroll
    for (int t = 0; t < DH / 8; ++t) { o[t][0] *= al0; o[t][1] *= al0; o[t][2] *= al1; o[t][3] *= al1; }
    {
      const int mat = lane >> 3, key = (lane & 7) + (mat & 1) * 8;
#pragma unroll
      for (int j = 0; j < DH / 16; ++j) {
        const int c = (j & 3) * 2 + (mat >> 1);
        uint32_t vb[4];
        ldsm_x4_t(vb, vbase + (j >> 2) * SUB + key * 128 + ((c ^ (key & 7)) << 4));
        mma16816(o[2 * j], pf, vb[0], vb[1]);
        mma16816(o[2 * j + 1], pf, vb[2], vb[3]);
        if (PR) {
          mma16816(o[2 * j], pl, vb[0], vb[1]);
          mma16816(o[2 * j + 1], pl, vb[2], vb[3]);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
  }

  // ---- merge the four partial results ----
  l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1); l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
  l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1); l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
  asm volatile("bar.sync 1, 128;" ::: "memory");   // every page consumed: the stages are free
  float* s_o = reinterpret_cast<float*>(tiles_ptr);  // [consumer][16][DH]
  if (qd == 0) { s_m[warp][g] = m_run[0]; s_m[warp][g + 8] = m_run[1]; s_l[warp][g] = l_run[0]; s_l[warp][g + 8] = l_run[1]; }
#pragma unroll
  for (int t = 0; t < DH / 8; ++t) {
    *reinterpret_cast<float2*>(s_o + (warp * 16 + g) * DH + t * 8 + 2 * qd) = make_float2(o[t][0], o[t][1]);
    *reinterpret_cast<float2*>(s_o + (warp * 16 + g + 8) * DH + t * 8 + 2 * qd) = make_float2(o[t][2], o[t][3]);
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  // weight of each warp's partial result per row, normalisation included: e_w / sum_w e_w l_w
  if (tid < 16 * kConsumers) {
    const int r = tid % 16, wsel = tid / 16, tsel = TPC == 1 ? 0 : (wsel & (TPC - 1));
    float mt_ = -INFINITY;
#pragma unroll
    for (int w = 0; w < kConsumers; ++w)
      if (TPC == 1 || (w & (TPC - 1)) == tsel) mt_ = fmaxf(mt_, s_m[w][r]);
    float den = 0.f, mine = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumers; ++w) {
      if (TPC != 1 && (w & (TPC - 1)) != tsel) continue;
      const float e = s_m[w][r] == -INFINITY ? 0.f : exp2f((s_m[w][r] - mt_) * sl2);
      den += e * s_l[w][r];
      if (w == wsel) mine = e;
    }
    const bool live = cta_row0 + tsel * 16 + r < nr && den > 0.f && !abort_flag;
    s_wgt[wsel][r] = live ? mine / den : 0.f;
  }
  asm volatile("bar.sync 1, 128;" ::: "memory");
  for (int idx = tid; idx < 16 * TPC * (DH / 4); idx += kConsumers * 32) {   // four features per thread
    const int rr = idx / (DH / 4), d = (idx % (DH / 4)) * 4;      // rr: row within the CTA's tiles
    const int tsel = rr / 16, r = rr % 16;
    if (cta_row0 + rr >= Rs) continue;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < kConsumers; ++w) {
      if (TPC != 1 && (w & (TPC - 1)) != tsel) continue;
      const float e = s_wgt[w][r];
      const float4 x = *reinterpret_cast<const float4*>(s_o + (w * 16 + r) * DH + d);
      acc.x += e * x.x; acc.y += e * x.y; acc.z += e * x.z; acc.w += e * x.w;
    }
    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    *reinterpret_cast<uint2*>(obase + size_t(rr) * H * DH * OW + d) =
        make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    if (PR)   // the part of the result that the first bf16 value leaves
      *reinterpret_cast<uint2*>(obase + size_t(rr) * H * DH * OW + size_t(H) * DH + d) =
          make_uint2(pack_bf16(acc.x - __low2float(lo), acc.y - __high2float(lo)), pack_bf16(acc.z - __low2float(hi), acc.w - __high2float(hi)));
  }
  if (tid == 0 && abort_flag) atomicCAS(status, 0, LASER_ERR_TIMEOUT);
}

}  // namespace

bool attention_tma_supported(const laser_model* m, const laser_kv* kv) {
  return kv->has_pages_map && (m->cfg.head_dim == 64 || m->cfg.head_dim == 128);
}

laser_status attention_tma_launch(laser_model* m, laser_kv* kv, int layer, const int32_t* seq_ids, int B, int Rs, bool tree,
                                  cudaStream_t stream) {
  const int dh = m->cfg.head_dim, H = m->cfg.n_heads, Hkv = m->cfg.n_kv_heads;
  const int64_t rows_per_layer = int64_t(kv->n_pages) * 2 * Hkv * 16;
  const int layer_row0 = int(rows_per_layer * layer);
  const int tiles = ceil_div(Rs, 16), tpc = tiles > 1 ? 2 : 1;   // row tiles of a sequence; tiles per CTA
  const bool pr = m->precise;
  const size_t smem = 1024 + size_t(kStages) * (2 * (dh / 64) * 16 * 128) + size_t(16) * tpc * (dh + 8) * 2 * (pr ? 2 : 1);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(B), unsigned(H), unsigned(ceil_div(tiles, tpc)));
  cfg.blockDim = dim3(kAttnThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const __nv_bfloat16* q = m->q;
  const int32_t *rc = m->row_ctx, *rn = m->row_n, *pt = kv->page_table;
  const unsigned long long* mask = tree ? m->row_mask : nullptr;
  const float* qf = m->qf;
#define LASER_ATTN_LAUNCH(DH_, TPC_, PR_)                                                                                \
  do {                                                                                                                   \
    LASER_CUDA(cudaFuncSetAttribute(attn_paged_kernel<DH_, TPC_, PR_>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem))); \
    LASER_CUDA(cudaLaunchKernelEx(&cfg, attn_paged_kernel<DH_, TPC_, PR_>, kv->pages_map, q, qf, seq_ids, rc, rn, Rs, H, Hkv, pt, \
                                  kv->pages_per_seq, layer_row0, m->attn, m->status, mask));                              \
  } while (0)
  if (pr) {
    if (dh == 128 && tpc == 1) LASER_ATTN_LAUNCH(128, 1, true);
    else if (dh == 128) LASER_ATTN_LAUNCH(128, 2, true);
    else if (tpc == 1) LASER_ATTN_LAUNCH(64, 1, true);
    else LASER_ATTN_LAUNCH(64, 2, true);
  } else if (dh == 128 && tpc == 1) LASER_ATTN_LAUNCH(128, 1, false);
  else if (dh == 128) LASER_ATTN_LAUNCH(128, 2, false);
  else if (tpc == 1) LASER_ATTN_LAUNCH(64, 1, false);
  else LASER_ATTN_LAUNCH(64, 2, false);
#undef LASER_ATTN_LAUNCH
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

}  // namespace laser
