// Dense contractions of the verify forward (QKV, O, gate/up, down, LM head) with their
// element-wise neighbours fused in: acc[r][n] = sum_k A[r][k] * W[n][k], bf16 operands, fp32
// accumulation, followed by RMSNorm scaling / rotary embedding + cache write / residual add /
// SwiGLU in the epilogue.
//
// Shape of the problem: few token rows (batch x (K+1), e.g. 144) against large weight
// matrices, so the step is bound by streaming the weights from HBM.  The weight rows take the
// 128-wide M side of tcgen05.mma and the token rows the N side (NT <= 192, no padding of the
// rows to 128); the accumulator is a 128 x NT fp32 tile in tensor memory.
//
// One CTA per (token tile, weight tile, K range); the CTAs that share an output tile form a
// thread-block cluster along K.  Two CTAs fit on an SM and kernels are chained with
// programmatic dependent launch, so while one CTA runs its epilogue, exits, or a CTA of the
// next kernel starts up in its place, the other CTA of the SM keeps streaming weights.
//   warp 0     TMA producer: weight and activation tiles (128-byte swizzle) into a ring of
//              shared-memory stages; weight tiles are requested before the dependency wait,
//              since they do not depend on the previous kernel;
//   warp 1     MMA issuer: tcgen05.mma into a TMEM accumulator, tcgen05.commit frees stages;
//   warps 2-5  move the finished accumulator to shared memory (the free stages); then, after a
//              cluster barrier, all six warps sum the partial tiles of the cluster through
//              distributed shared memory in rank order (run-to-run identical, no partial sums
//              in global memory) for the token columns this CTA owns and apply the fused epilogue.
// Variants chosen by the host per launch: two weight tiles per CTA (MT = 2, one CTA per SM, token
// tiles of up to 256 rows) where several token tiles make the launch L2->SM-bound; activations as
// hi + lo bf16 pairs (the model's precise mode: every weight block is multiplied with both parts
// into the same accumulator); and, for the LM head, an epilogue that leaves what the acceptance
// rule needs per (row, vocabulary tile) instead of the logits.
// Every mbarrier wait is bounded: on expiry the CTA records LASER_ERR_TIMEOUT, drains its
// copies, still joins the cluster barriers, frees its tensor memory and exits.
#include <map>
#include <tuple>
#include <type_traits>

#include "epilogue.cuh"
#include "tma.cuh"
#include "umma.cuh"

namespace laser {
namespace {

constexpr int kTcThreads = 192;
constexpr int kMaxStages = 6;
constexpr int kMaxNT = 192;       // token rows per tile: accumulator staging must fit shared memory
#ifndef LASER_WIDE_NT
#define LASER_WIDE_NT 256
#endif
constexpr int kMaxNTWide = LASER_WIDE_NT;   // ... with two weight tiles per CTA (one CTA per SM); 256 = the largest MMA N
constexpr int kSmemBudget = 110 * 1024;  // shared memory of one CTA: two CTAs per SM
constexpr int kSmemBudgetWide = 200 * 1024;  // with two weight tiles per CTA: one CTA per SM
constexpr int kAccCols = 256;     // tensor-memory columns between the accumulators of a CTA's weight tiles

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  return remote;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t cluster_addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr));
  return v;
}
__device__ __forceinline__ void st_shared_f32(uint32_t addr, float v) {
  asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v));
}
// MT = weight tiles per CTA.  1: the form for few token rows (the step is bound by the weight stream;
// two CTAs per SM).  2: for several token tiles, where the launches are bound by L2->SM traffic: a CTA
// multiplies two 128-row weight tiles with the same staged activation tile (two accumulators), so the
// activation bytes per flop halve; one CTA per SM, no K split.
template <int EPI, int MT>
__global__ void __launch_bounds__(kTcThreads, MT == 1 ? 2 : 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA, const GemmEpilogue e,
               int N, int NT, int total_kb, int kb_per_split, int splits, int stages, int tmem_cols,
               int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ float s_rstd[MT == 1 ? kMaxNT : kMaxNTWide];
  __shared__ int s_pos[MT == 1 ? kMaxNT : kMaxNTWide], s_page[MT == 1 ? kMaxNT : kMaxNTWide];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its prologue
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
  const uint32_t w_bytes = kBM * 128, a_bytes = uint32_t(NT) * 128, stage_bytes = MT * w_bytes + a_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int krank = blockIdx.x % splits, ttile = blockIdx.x / splits;   // cluster rank = K range
  const int wtile = blockIdx.y;
  const int r0 = ttile * NT, n0 = wtile * kBM * MT;           // wtile counts groups of MT weight tiles
  const int kb0 = krank * kb_per_split;
  const int nkb = max(0, min(kb_per_split, total_kb - kb0));
  // Activations given as hi + lo bf16 pairs ([hi | lo] side by side in a row, lo starting at column a_lo_off): K
  // block g multiplies weight block g / 2 with the hi (g even) or lo (g odd) part, into the same accumulator.
  const int wshift = e.a_lo_off ? 1 : 0;
  const int slice = (NT + splits - 1) / splits;            // token columns finished by one CTA of the cluster
  const int own = max(0, min(slice, NT - krank * slice));

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
    mbar_init(smem_u32(&acc_bar), 1);
    mbar_fence_init();
    // The first weight stages are requested here, before tensor memory is allocated and the CTA's
    // threads meet: they depend on nothing, and a CTA that starts late (once an earlier kernel's CTA
    // has left its slot) has its first bytes on the way that much sooner.
    const uint64_t w_policy0 = make_policy_evict_first();
    for (int kb = 0; kb < min(stages, nkb); ++kb) {
      const uint32_t bar = smem_u32(&full_bar[kb]), dst = tiles + uint32_t(kb) * stage_bytes;
      const int wk = ((kb0 + kb) >> wshift) * kBK;
      mbar_expect_tx(bar, stage_bytes);
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        const int T = wtile * MT + t;
        if (EPI == EPI_SWIGLU) {   // 64 gate rows and the 64 up rows of the same features (the map's box is 64 rows)
          tma_load_2d_hint(dst + t * w_bytes, &tmW, wk, T * 64, bar, w_policy0);
          tma_load_2d_hint(dst + t * w_bytes + w_bytes / 2, &tmW, wk, e.f + T * 64, bar, w_policy0);
        } else {                   // 128 consecutive rows: one copy (the map's box is 128 rows)
          tma_load_2d_hint(dst + t * w_bytes, &tmW, wk, T * kBM, bar, w_policy0);
        }
      }
    }
    tma_prefetch_map(&tmA);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_slot;
  // floats between consecutive token rows of the staged accumulator; the verdict epilogue reads one row per lane
  // and pads the rows so that those reads spread over the banks
  constexpr int kRow = EPI == EPI_VERDICT ? kVerdictRow : kBM;

  // gains of the next norm for the first weight tile: a weight, not a result of the kernel before, so
  // requested now, long before the epilogue uses it
  uint2 gain4_first = make_uint2(0u, 0u);
  if (EPI == EPI_RESID && n0 + 4 * lane < N) gain4_first = *reinterpret_cast<const uint2*>(e.gain_next + n0 + 4 * lane);
  bool acc_ok = true;
  // accumulator t from tensor memory to shared memory, token-major [NT][128] (epilogue warps; a warp may
  // only touch its own 32 TMEM lanes)
  auto drain = [&](int t) {
    const int quarter = warp & 3;
    const uint32_t src = tmem_acc + uint32_t(t) * kAccCols + (uint32_t(quarter * 32) << 16);
    const uint32_t dst0 = tiles + uint32_t((quarter * 32 + lane) * 4);
    for (int c = 0; c < NT; c += 48) {   // three loads in flight, one wait; reads past NT stay inside the allocation
      uint32_t v0[16], v1[16], v2[16];
      if (acc_ok && nkb > 0) {
        tmem_ld16(src + uint32_t(c), v0);
        if (c + 16 < NT) tmem_ld16(src + uint32_t(c + 16), v1);
        if (c + 32 < NT) tmem_ld16(src + uint32_t(c + 32), v2);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int x = 0; x < 16; ++x) v0[x] = v1[x] = v2[x] = 0u;
      }
      const uint32_t dst = dst0 + uint32_t(c) * (kRow * 4);
#pragma unroll
      for (int x = 0; x < 16; ++x) {
        if (c + x < NT) st_shared_f32(dst + x * (kRow * 4), __uint_as_float(v0[x]));
        if (c + 16 + x < NT) st_shared_f32(dst + (16 + x) * (kRow * 4), __uint_as_float(v1[x]));
        if (c + 32 + x < NT) st_shared_f32(dst + (32 + x) * (kRow * 4), __uint_as_float(v2[x]));
      }
    }
  };

  if (warp == 0) {
    if (lane == 0) {  // ---- TMA producer ----
      const uint32_t full0 = smem_u32(&full_bar[0]);
      // weights are read once per step: they must not push the activations, the residual stream and the
      // cache pages of this step out of L2; every CTA of the launch reads the activations
      const uint64_t w_policy = make_policy_evict_first(), a_policy = make_policy_evict_last();
      auto load = [&](uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar, uint64_t pol) { tma_load_2d_hint(dst, tm, x, y, bar, pol); };
      auto expect = [&](int s) { mbar_expect_tx(smem_u32(&full_bar[s]), stage_bytes); };
      auto load_w = [&](int kb, int s) {
        const int k = ((kb0 + kb) >> wshift) * kBK;
        const uint32_t dst = tiles + uint32_t(s) * stage_bytes, bar = full0 + uint32_t(s) * 8;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          const int T = wtile * MT + t;
          if (EPI == EPI_SWIGLU) {
            load(dst + t * w_bytes, &tmW, k, T * 64, bar, w_policy);
            load(dst + t * w_bytes + w_bytes / 2, &tmW, k, e.f + T * 64, bar, w_policy);
          } else {
            load(dst + t * w_bytes, &tmW, k, T * kBM, bar, w_policy);
          }
        }
      };
      auto load_a = [&](int kb, int s) {
        const int g = kb0 + kb;
        load(tiles + uint32_t(s) * stage_bytes + MT * w_bytes, &tmA, (g & wshift) * e.a_lo_off + (g >> wshift) * kBK, r0,
             full0 + uint32_t(s) * 8, a_policy);
      };
      // The ring was filled with weight tiles at the start of the kernel (they do not depend on the
      // kernel before this one); only now wait for that kernel's results (the activations).
      const int pre = min(stages, nkb);
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int kb = 0; kb < pre; ++kb) load_a(kb, kb);
      bool ok = true;
      int kb = pre;
      // (slot and round are counted, not divided out: this loop is one thread, and it paces the weight stream)
      for (int s = 0, par = 0; kb < nkb; ++kb) {
        ok = mbar_wait_hot(smem_u32(&empty_bar[s]), par, &abort_flag);
        if (!ok) break;
        expect(s);
        load_w(kb, s);
        load_a(kb, s);
        if (++s == stages) { s = 0; par ^= 1; }
      }
      if (!ok)  // drain copies still in flight before the CTA may exit
        for (int j = max(0, kb - stages); j < kb; ++j) mbar_drain(smem_u32(&full_bar[j % stages]), (j / stages) & 1);
    }
  } else if (warp == 1) {
    if (lane == 0) {  // ---- MMA issuer ----
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(NT >> 3) << 17) | (uint32_t(kBM >> 4) << 24);
      bool ok = true;
      for (int kb = 0, s = 0, par = 0; kb < nkb && ok; ++kb) {
        ok = mbar_wait_hot(smem_u32(&full_bar[s]), par, &abort_flag);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t w_addr = tiles + uint32_t(s) * stage_bytes;
        const uint64_t adesc = umma_desc(w_addr + MT * w_bytes);
#pragma unroll
        for (int t = 0; t < MT; ++t) {
          const uint64_t wdesc = umma_desc(w_addr + t * w_bytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)  // 16 bf16 = 32 bytes further along K inside the swizzle span
            umma_bf16(tmem_acc + uint32_t(t) * kAccCols, wdesc + uint64_t(k * 2), adesc + uint64_t(k * 2), idesc, (kb | k) != 0);
        }
        umma_commit(smem_u32(&empty_bar[s]));
        if (++s == stages) { s = 0; par ^= 1; }
      }
      // arrives when every MMA issued so far has finished
      umma_commit(smem_u32(&acc_bar));
    }
  } else {
    // ---- epilogue warps, part 1: everything that can be done before the accumulator is ready ----
    asm volatile("griddepcontrol.wait;" ::: "memory");   // what follows reads earlier kernels' results
    for (int j = threadIdx.x - 64; j < NT; j += 128) {   // per-row scale and cache coordinates
      const int r = r0 + j;
      float rstd = 1.f;
      int pos = -1, page = 0;
      if (r < e.R_rows) {
        if (e.sumsq_in) {
          float ss = 0.f;
          for (int tt = 0; tt < e.sumsq_in_tiles; ++tt) ss += e.sumsq_in[size_t(tt) * e.sumsq_ld + r];
          rstd = rsqrtf(ss * e.inv_d + e.eps);
        }
        if (EPI == EPI_VERDICT) pos = r < e.R_store ? e.row_draft[r] : -1;   // the row's draft token, in the slot of the position
        if (EPI == EPI_QKV) {
          pos = e.row_pos[r];
          if (pos >= 0) page = e.page_table[size_t(e.row_seq[r]) * e.pages_per_seq + (pos >> 4)];
        }
      }
      s_rstd[j] = rstd; s_pos[j] = pos; s_page[j] = page;
    }
    // part 2: the first accumulator to shared memory
    acc_ok = mbar_wait(smem_u32(&acc_bar), 0, &abort_flag);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    drain(0);
  }
#pragma unroll
  for (int t = 0; t < MT; ++t) {   // the CTA's weight tiles, one after the other through the same staging buffer
  if (t > 0) {
    __syncthreads();               // the staged tile before this one has been finished
    if (warp >= 2) drain(t);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (splits > 1) cluster_sync_all();  // every partial tile of the cluster is staged
  const int wt = wtile * MT + t, n0t = wt * kBM;
  const int nfeat = n0t + 4 * lane;
  const LaneCtx lc = make_lane_ctx<EPI>(e, n0t, lane, N);
  uint2 gain4 = gain4_first;
  if (EPI == EPI_RESID && t > 0 && nfeat < N) gain4 = *reinterpret_cast<const uint2*>(e.gain_next + nfeat);
  auto fetch_operands = [&](int jj, float4& g0, float4& g1) {
    g0 = make_float4(0.f, 0.f, 0.f, 0.f); g1 = g0;
    const int r = r0 + krank * slice + jj;
    if (jj < own && r < e.R_rows && nfeat < N) {
      if (EPI == EPI_RESID) g0 = *reinterpret_cast<const float4*>(e.resid + size_t(r) * N + nfeat);
      if (EPI == EPI_QKV && lc.kind < 2) {
        const float* cs = e.rope + size_t(r) * e.dh + lc.rope_off;
        g0 = *reinterpret_cast<const float4*>(cs);       // c0 s0 c1 s1
        g1 = *reinterpret_cast<const float4*>(cs + 4);   // c2 s2 c3 s3
      }
    }
  };

  __syncwarp();
  // (an odd tile count leaves the last group's second tile beyond the matrix: nothing to finish)
  const bool tile_valid = EPI == EPI_SWIGLU ? wt * 64 < e.f : n0t < N;
  if (!tile_valid) {
  } else if (EPI == EPI_VERDICT && splits == 1) {
    // part 3, acceptance fused into the LM head: one lane per token row scans the row's 128 staged logits
    if (e.out) {   // on request the logits are stored as well (the plain epilogue's stores)
      for (int j = warp; j < NT; j += kTcThreads / 32) {
        float4 a;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w) : "r"(tiles + uint32_t((j * kRow + 4 * lane) * 4)));
        epi_plain(e, lc, r0 + j, r0 + j < e.R_rows && !abort_flag, a, s_rstd[j], N);
      }
    }
    const bool ok = !abort_flag;
    if (e.top_n <= 1) verdict_rows<1>(e, tiles, NT, r0, n0t, wt, N, warp, lane, s_rstd, s_pos, ok);
    else if (e.top_n == 2) verdict_rows<2>(e, tiles, NT, r0, n0t, wt, N, warp, lane, s_rstd, s_pos, ok);
    else verdict_rows<4>(e, tiles, NT, r0, n0t, wt, N, warp, lane, s_rstd, s_pos, ok);
  } else if ((EPI == EPI_SWIGLU || EPI == EPI_PLAIN) && splits == 1) {
    // part 3 without partial tiles to sum or operands to prefetch: all six warps finish rows,
    // in wide groups whose loads are issued first.
    constexpr int kWide = 12;
    for (int jb = warp * kWide; jb < NT; jb += (kTcThreads / 32) * kWide) {
      float4 acc[kWide];
#pragma unroll
      for (int b = 0; b < kWide; ++b) {
        const int j = min(jb + b, NT - 1);
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(acc[b].x), "=f"(acc[b].y), "=f"(acc[b].z), "=f"(acc[b].w) : "r"(tiles + uint32_t((j * kRow + 4 * lane) * 4)));
      }
#pragma unroll
      for (int b = 0; b < kWide; ++b) {
        const int j = min(jb + b, NT - 1), r = r0 + j;
        const bool live = jb + b < NT && r < e.R_rows && !(abort_flag);
        const float rstd = s_rstd[j];
        if (EPI == EPI_PLAIN) epi_plain(e, lc, r, live, acc[b], rstd, N);
        else epi_swiglu(e, r, live, wt * 64, lane, acc[b], rstd);
      }
    }
  } else {
    // part 3: sum the partial columns this CTA owns (ranks in order 0..splits-1) and finish them, all
    // six warps, group g by warp g % 6.  A group is as many columns as give about twelve loads in
    // flight per lane: every partial column of the group and its epilogue operands are requested
    // first (independent loads, one round trip through distributed shared memory), then summed in
    // rank order and finished.
    auto reduce_rows = [&](auto s_tag, auto rb_tag) {
      constexpr int S = decltype(s_tag)::value, RB = decltype(rb_tag)::value;
      uint32_t rank_base[S];
#pragma unroll
      for (int q = 0; q < S; ++q) rank_base[q] = S > 1 ? map_to_rank(tiles, uint32_t(q)) : tiles;
      for (int jb = warp * RB; jb < own; jb += (kTcThreads / 32) * RB) {
        float4 part[RB][S], g0[RB], g1[RB];
#pragma unroll
        for (int b = 0; b < RB; ++b) {
          const int jj = min(jb + b, own - 1);
#pragma unroll
          for (int q = 0; q < S; ++q)
            part[b][q] = ld_cluster_f4(rank_base[q] + uint32_t(((krank * slice + jj) * kRow + 4 * lane) * 4));
        }
#pragma unroll
        for (int b = 0; b < RB; ++b) fetch_operands(jb + b, g0[b], g1[b]);
#pragma unroll
        for (int b = 0; b < RB; ++b) {
          float4 acc = part[b][0];
#pragma unroll
          for (int q = 1; q < S; ++q) { acc.x += part[b][q].x; acc.y += part[b][q].y; acc.z += part[b][q].z; acc.w += part[b][q].w; }
          const int jj = jb + b;
          const int j = jj < own ? krank * slice + jj : 0, r = r0 + j;
          const bool live = jj < own && r < e.R_rows && !abort_flag;   // the last token tile may overhang the buffers
          const float rstd = s_rstd[j];
          if (EPI == EPI_PLAIN) epi_plain(e, lc, r, live, acc, rstd, N);
          else if (EPI == EPI_VERDICT) epi_verdict(e, lc, r, live, lane, acc, rstd, N, wt, s_pos[j]);
          else if (EPI == EPI_RESID) epi_resid(e, lc, r, live, lane, acc, N, wt, g0[b], gain4);
          else if (EPI == EPI_SWIGLU) epi_swiglu(e, r, live, wt * 64, lane, acc, rstd);
          else epi_qkv(e, lc, r, live, acc, rstd, s_pos[j], s_page[j], g0[b], g1[b]);
        }
      }
    };
    using std::integral_constant;
    switch (splits) {
      case 1: reduce_rows(integral_constant<int, 1>{}, integral_constant<int, 6>{}); break;
      case 2: reduce_rows(integral_constant<int, 2>{}, integral_constant<int, 6>{}); break;
      case 3: reduce_rows(integral_constant<int, 3>{}, integral_constant<int, 4>{}); break;
      case 4: reduce_rows(integral_constant<int, 4>{}, integral_constant<int, 3>{}); break;
      case 5: reduce_rows(integral_constant<int, 5>{}, integral_constant<int, 2>{}); break;
      case 6: reduce_rows(integral_constant<int, 6>{}, integral_constant<int, 2>{}); break;
      case 7: reduce_rows(integral_constant<int, 7>{}, integral_constant<int, 2>{}); break;
      default: reduce_rows(integral_constant<int, 8>{}, integral_constant<int, 1>{}); break;
    }
  }
  __syncwarp();
  }  // weight tiles of the CTA
  if (splits > 1) cluster_sync_all();  // peers may still be reading this CTA's staged tile or tensor memory
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(tmem_cols) : "memory");
  }
  if (threadIdx.x == 0 && abort_flag) atomicCAS(status, 0, LASER_ERR_TIMEOUT);
}

// ---- host side --------------------------------------------------------------------------
struct GemmState {
  // (pointer, rows, cols, box rows) -> tensor map
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> maps;
  bool ready = false;
};

GemmState* get_state(laser_model* m) {
  if (!m->gemm_state) m->gemm_state = new GemmState();
  return static_cast<GemmState*>(m->gemm_state);
}

laser_status tensor_map(GemmState* st, const void* ptr, int rows, int cols, int box_rows, const CUtensorMap** out) {
  auto key = std::make_tuple(ptr, rows, cols, box_rows);
  auto it = st->maps.find(key);
  if (it == st->maps.end()) {
    CUtensorMap tm;
    LASER_TRY(encode_bf16_2d(&tm, ptr, uint64_t(rows), uint64_t(cols), uint32_t(box_rows)));
    it = st->maps.emplace(key, tm).first;
  }
  *out = &it->second;
  return LASER_OK;
}

struct TcShape { int n_ttiles, NT, stages, tmem_cols; size_t smem; };

// mt = weight tiles per CTA (1 or 2); max_nt = most token rows per tile
TcShape tc_shape(int R_pad, int mt = 1, int max_nt = kMaxNT) {
  TcShape s;
  s.n_ttiles = ceil_div(R_pad, max_nt);
  s.NT = ceil_div(ceil_div(R_pad, s.n_ttiles), 16) * 16;
  const int stage_bytes = mt * kBM * 128 + s.NT * 128;
  s.stages = std::max(2, std::min(kMaxStages, (mt == 1 ? kSmemBudget : kSmemBudgetWide) / stage_bytes));
  s.tmem_cols = 32;
  while (s.tmem_cols < s.NT) s.tmem_cols <<= 1;
  if (mt == 2) s.tmem_cols = 2 * kAccCols;
  s.smem = std::max(size_t(s.stages) * stage_bytes, size_t(s.NT) * kVerdictRow * 4) + 1024;
  return s;
}

template <int EPI, int MT>
laser_status launch_epi(const CUtensorMap& tw, const CUtensorMap& ta, const GemmEpilogue& e, int N, const TcShape& sh,
                        int n_wtiles, int total_kb, int kbps, int splits, int32_t* status, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(sh.n_ttiles * splits), unsigned(n_wtiles), 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = sh.smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(splits);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // programmatic dependent launch: this kernel may begin while the previous one drains; it
  // orders itself with griddepcontrol.wait
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  LASER_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<EPI, MT>, tw, ta, e, N, sh.NT, total_kb, kbps, splits, sh.stages,
                                sh.tmem_cols, status));
  return LASER_OK;
}

laser_status prepare(GemmState* st) {
  if (st->ready) return LASER_OK;
  const int bytes = kSmemBudget + 2048, wide = kSmemBudgetWide + 2048;
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_PLAIN, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_PLAIN, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, wide));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, wide));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, wide));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, wide));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_VERDICT, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_VERDICT, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, wide));
  st->ready = true;
  return LASER_OK;
}

// Split count (cluster size along K).  Measured on the 7B shapes with 144 rows: a launch is
// fastest with roughly 200 CTAs (of the 296 resident slots), whatever the matrix: 1 for 172 or
// 250 weight tiles, 2 for 96, 6 for 32.  Fewer CTAs leave SMs idle, more add start-up and
// cluster-reduction cost faster than they shorten the K loop.
int pick_splits(int R_pad, int N, int K, int epi) {
  const int n_wtiles = epi == EPI_SWIGLU ? ceil_div(N / 2, 64) : ceil_div(N, kBM);
  const int tiles = n_wtiles * tc_shape(R_pad).n_ttiles, total_kb = ceil_div(K, kBK);
  int s = int(208.0 / tiles + 0.5);
  s = std::max(1, std::min(s, std::min(total_kb, 8)));   // portable cluster size
  while (s > 1 && ceil_div(total_kb, s) * (s - 1) >= total_kb) --s;   // no rank without K blocks
  return s;
}

}  // namespace

laser_status gemm_fused(laser_model* m, const __nv_bfloat16* A, const __nv_bfloat16* W, int R_pad, int N, int K, int epi,
                        const GemmEpilogue& e, cudaStream_t stream) {
  if (R_pad % 16 != 0 || K % 8 != 0 || N % 8 != 0 || (reinterpret_cast<uintptr_t>(A) & 15) || (reinterpret_cast<uintptr_t>(W) & 15)) {
    set_error("GEMM shape N=%d K=%d rows=%d unsupported (N, K multiples of 8, rows of 16, 16-byte aligned operands)", N, K, R_pad);
    return LASER_ERR_UNSUPPORTED;
  }
  GemmState* st = get_state(m);
  LASER_TRY(prepare(st));
  const int n_wtiles = epi == EPI_SWIGLU ? ceil_div(N / 2, 64) : ceil_div(N, kBM);
  const int splits = pick_splits(R_pad, N, K, epi);
  // several token tiles and no K split: two weight tiles per CTA share every staged activation tile
  // (where the halved CTA count still gives every SM one)
  const int n_tt = tc_shape(R_pad).n_ttiles;
  const int mt = (n_tt > 1 && splits == 1 && ceil_div(n_wtiles, 2) * n_tt >= 148) ? 2 : 1;
  TcShape sh = tc_shape(R_pad, mt);
  if (mt == 2) {
    // Token tiles of up to 256 rows (the largest MMA N) re-read the weights from L2 fewer times, but make fewer,
    // longer CTAs: taken where they do not cost more in whole waves of CTAs over the SMs (a CTA's time goes with
    // the bytes it stages per K block: 256 weight rows + NT token rows).
    const TcShape wide = tc_shape(R_pad, 2, kMaxNTWide);
    auto cost = [&](const TcShape& t) { return ceil_div(ceil_div(n_wtiles, 2) * t.n_ttiles, 148) * (256 + t.NT); };
    if (cost(wide) < cost(sh)) sh = wide;
  }
  const CUtensorMap *tw = nullptr, *ta = nullptr;
  LASER_TRY(tensor_map(st, W, N, K, epi == EPI_SWIGLU ? 64 : 128, &tw));
  LASER_TRY(tensor_map(st, A, m->R_pad, e.a_lo_off ? 2 * K : K, sh.NT, &ta));
  const int total_kb = ceil_div(K, kBK) * (e.a_lo_off ? 2 : 1), kbps = ceil_div(total_kb, splits);
  const int n_groups = ceil_div(n_wtiles, mt);     // grid rows: groups of mt weight tiles
#define LASER_GEMM_LAUNCH(E)                                                                                            \
  do {                                                                                                                  \
    if (mt == 1) LASER_TRY((launch_epi<E, 1>(*tw, *ta, e, N, sh, n_groups, total_kb, kbps, splits, m->status, stream))); \
    else LASER_TRY((launch_epi<E, 2>(*tw, *ta, e, N, sh, n_groups, total_kb, kbps, splits, m->status, stream)));         \
  } while (0);
  switch (epi) {
    case EPI_PLAIN: LASER_GEMM_LAUNCH(EPI_PLAIN) break;
    case EPI_RESID: LASER_GEMM_LAUNCH(EPI_RESID) break;
    case EPI_SWIGLU: LASER_GEMM_LAUNCH(EPI_SWIGLU) break;
    case EPI_VERDICT: LASER_GEMM_LAUNCH(EPI_VERDICT) break;
    default: LASER_GEMM_LAUNCH(EPI_QKV) break;
  }
#undef LASER_GEMM_LAUNCH
  count_launch();
  return LASER_OK;
}

void gemm_state_free(laser_model* m) {
  delete static_cast<GemmState*>(m->gemm_state);
  m->gemm_state = nullptr;
}

}  // namespace laser
