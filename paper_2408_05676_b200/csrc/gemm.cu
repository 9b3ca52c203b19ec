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
// Persistent kernel, one CTA per SM, CTAs grouped in thread-block clusters of `splits` along K.
// A cluster walks the output tiles assigned to it; each of its CTAs contracts its own K range
// of the tile.  Roles inside a CTA:
//   warp 0     TMA producer: weight and activation tiles (128-byte swizzle) into a ring of
//              shared-memory stages, running ahead across tile boundaries;
//   warp 1     MMA issuer: tcgen05.mma into one of two TMEM accumulators, tcgen05.commit frees
//              stages and publishes finished accumulators;
//   warps 2-5  epilogue: read the accumulator (tcgen05.ld), send every token column to the
//              CTA of the cluster that owns it (distributed shared memory), then sum the
//              `splits` partial columns they own in rank order (run-to-run identical, no
//              partial sums in global memory) and apply the fused epilogue.
// The epilogue of tile i overlaps the main loop of tile i+1 (double-buffered accumulator);
// cross-CTA hand-over uses cluster-scope mbarriers.  Every wait is bounded: on expiry the CTA
// records LASER_ERR_TIMEOUT, stops issuing work, still joins the final cluster barrier, frees
// its tensor memory and exits.
#include <map>
#include <tuple>

#include "model.cuh"
#include "tma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
constexpr int kTcThreads = 192;
constexpr int kBM = 128;          // weight rows per tile (MMA M)
constexpr int kBK = 64;           // K elements per stage = one 128-byte swizzle span of bf16
constexpr int kMaxStages = 6;
constexpr int kMaxNT = 192;       // token rows per tile: accumulator staging must fit shared memory
constexpr int kSmemLimit = 222 * 1024;   // dynamic shared memory one CTA may ask for
constexpr int kBatch = 3, kPre = 3;      // epilogue: columns per group, groups whose operands are prefetched

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows 128 B apart, groups
// of 8 rows 1024 B apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= uint64_t((smem_addr & 0x3FFFF) >> 4);        // start address
  d |= uint64_t(1024 >> 4) << 32;                   // stride byte offset between 8-row groups
  d |= uint64_t(1) << 46;                           // descriptor version of this architecture
  d |= uint64_t(2) << 61;                           // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  return remote;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v));
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait on a barrier that peers of the cluster arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_cluster(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) { *abort_flag = 1; return false; }
  }
}
// 16 consecutive fp32 columns of this thread's TMEM lane (no wait: pair with tmem_ld_wait)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float4 ld_shared_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
// AND of a flag over the 128 epilogue threads (named barrier 1), so that they leave a loop together.
__device__ __forceinline__ bool epilogue_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbar.red.and.pred p, 1, 128, q;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(r) : "r"(uint32_t(ok)) : "memory");
  return r != 0;
}
__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  return make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
}

// ---- fused epilogues: one warp finishes one token row r of a 128-feature tile; lane l holds
//      features n0 + 4l .. 4l+3 in v ----------------------------------------------------------
__device__ __forceinline__ void epi_plain(const GemmEpilogue& e, int r, int n0, int lane, float4 v, float rstd, int N) {
  if (r >= e.R_store) return;
  const int n = n0 + 4 * lane;
  float* o = e.out + size_t(r) * e.ldo + n;
  v.x *= rstd; v.y *= rstd; v.z *= rstd; v.w *= rstd;
  if (n + 3 < N && (e.ldo & 3) == 0) {
    *reinterpret_cast<float4*>(o) = v;
  } else {
    if (n < N) o[0] = v.x;
    if (n + 1 < N) o[1] = v.y;
    if (n + 2 < N) o[2] = v.z;
    if (n + 3 < N) o[3] = v.w;
  }
}

// resid += acc; xb = bf16(resid * gain of the next norm); per-tile sum of squares for that norm
__device__ __forceinline__ void epi_resid(const GemmEpilogue& e, int r, int n0, int lane, float4 v, int N, int tile,
                                          float4 x, uint2 g2) {
  const int n = n0 + 4 * lane;
  float ss = 0.f;
  if (n < N) {  // N is a multiple of 8 (checked on the host), so the four features are all valid
    x.x += v.x; x.y += v.y; x.z += v.z; x.w += v.w;
    *reinterpret_cast<float4*>(e.resid + size_t(r) * N + n) = x;
    const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&g2.x), g23 = *reinterpret_cast<const __nv_bfloat162*>(&g2.y);
    *reinterpret_cast<uint2*>(e.xb + size_t(r) * N + n) =
        pack4_bf16(x.x * __low2float(g01), x.y * __high2float(g01), x.z * __low2float(g23), x.w * __high2float(g23));
    ss = x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
  }
  for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if (lane == 0) e.sumsq_out[size_t(tile) * e.sumsq_ld + r] = ss;
}

// tile rows 0..63 = gate features f0.., rows 64..127 = up features f0..; act = silu(g) * u
__device__ __forceinline__ void epi_swiglu(const GemmEpilogue& e, int r, int f0, int lane, float4 v, float rstd) {
  float4 u;
  u.x = __shfl_xor_sync(0xffffffffu, v.x, 16); u.y = __shfl_xor_sync(0xffffffffu, v.y, 16);
  u.z = __shfl_xor_sync(0xffffffffu, v.z, 16); u.w = __shfl_xor_sync(0xffffffffu, v.w, 16);
  const int fidx = f0 + 4 * lane;
  if (lane < 16 && fidx < e.f) {  // f is a multiple of 8 (checked on the host)
    auto act = [rstd](float g, float up) { g *= rstd; up *= rstd; return __fdividef(g, 1.f + __expf(-g)) * up; };
    *reinterpret_cast<uint2*>(e.act + size_t(r) * e.f + fidx) =
        pack4_bf16(act(v.x, u.x), act(v.y, u.y), act(v.z, u.z), act(v.w, u.w));
  }
}

// rotary embedding of Q and K (pair i, i + dh/2), bf16 rounding, Q store, K/V page write
__device__ __forceinline__ void epi_qkv(const GemmEpilogue& e, int r, int n0, int lane, float4 v, float rstd, int N,
                                        int pos, int page, float4 cs01, float4 cs23) {
  v.x *= rstd; v.y *= rstd; v.z *= rstd; v.w *= rstd;
  const int dh = e.dh, half = dh >> 1, dq = e.H * dh, dkv = e.Hkv * dh;
  const int shift = dh >> 3;  // lanes between a feature and its rotation partner
  float4 pv;
  pv.x = __shfl_xor_sync(0xffffffffu, v.x, shift); pv.y = __shfl_xor_sync(0xffffffffu, v.y, shift);
  pv.z = __shfl_xor_sync(0xffffffffu, v.z, shift); pv.w = __shfl_xor_sync(0xffffffffu, v.w, shift);
  const int n = n0 + 4 * lane;
  if (n >= N) return;
  const int idx = n % dh;          // four consecutive features stay inside one half of one head
  float4 y = v;
  if (n < dq + dkv) {
    const float sg = idx < half ? -1.f : 1.f;
    y.x = v.x * cs01.x + sg * pv.x * cs01.y;
    y.y = v.y * cs01.z + sg * pv.y * cs01.w;
    y.z = v.z * cs23.x + sg * pv.z * cs23.y;
    y.w = v.w * cs23.z + sg * pv.w * cs23.w;
  }
  if (n < dq) {
    if (pos < 0) y = make_float4(0.f, 0.f, 0.f, 0.f);
    *reinterpret_cast<uint2*>(e.q + size_t(r) * dq + n) = pack4_bf16(y.x, y.y, y.z, y.w);
  } else if (pos >= 0) {
    const int is_v = n >= dq + dkv;
    const int h = (n - dq - is_v * dkv) / dh;
    bf16* dst = e.pages_layer + size_t(page) * e.page_elems + (size_t(is_v) * e.Hkv + h) * 16 * dh + size_t(pos & 15) * dh + idx;
    *reinterpret_cast<uint2*>(dst) = pack4_bf16(y.x, y.y, y.z, y.w);
  }
}


template <int EPI>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA, const GemmEpilogue e,
               int N, int NT, int n_ttiles, int n_wtiles, int total_kb, int kb_per_split, int splits, int stages,
               int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages];
  __shared__ uint64_t acc_full[2], acc_empty[2];   // TMEM accumulator hand-over MMA <-> epilogue
  __shared__ uint64_t red_full, red_free;          // reduction buffer hand-over between cluster peers
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ float s_rstd[kMaxNT];
  __shared__ int s_pos[kMaxNT], s_page[kMaxNT];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
  const uint32_t w_bytes = kBM * 128, a_bytes = uint32_t(NT) * 128, stage_bytes = w_bytes + a_bytes;
  const int slice = (NT + splits - 1) / splits;            // token columns owned by one CTA of the cluster
  const uint32_t red_addr = tiles + uint32_t(stages) * stage_bytes;   // [splits][slice][128] fp32
  const float* red = reinterpret_cast<const float*>(smem_raw + (red_addr - raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int krank = blockIdx.x % splits, cluster_id = blockIdx.x / splits, n_clusters = gridDim.x / splits;
  const int n_tiles = n_ttiles * n_wtiles;
  const int kb0 = krank * kb_per_split;
  const int nkb = max(0, min(kb_per_split, total_kb - kb0));
  constexpr int kAccCols = 256;                             // TMEM columns per accumulator buffer

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its prologue
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&acc_full[b]), 1); mbar_init(smem_u32(&acc_empty[b]), 1); }
    mbar_init(smem_u32(&red_full), uint32_t(splits));
    mbar_init(smem_u32(&red_free), uint32_t(splits));
    mbar_fence_init();
    tma_prefetch_map(&tmW);
    tma_prefetch_map(&tmA);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(2 * kAccCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (splits > 1) cluster_sync_all();   // peers' barriers exist before anyone arrives on them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    if (lane == 0) {  // ---- TMA producer ----
      // Flat iteration space: `it` walks the K blocks of this CTA's tiles in order.
      const int my_tiles = cluster_id < n_tiles ? (n_tiles - cluster_id + n_clusters - 1) / n_clusters : 0;
      const int total_it = my_tiles * nkb;
      auto load_w = [&](int it) {
        const int ti = it / nkb, kb = it - ti * nkb, wtile = (cluster_id + ti * n_clusters) / n_ttiles;
        const int s = it % stages, k = (kb0 + kb) * kBK;
        const uint32_t dst = tiles + uint32_t(s) * stage_bytes, bar = smem_u32(&full_bar[s]);
        tma_load_2d(dst, &tmW, k, EPI == EPI_SWIGLU ? wtile * 64 : wtile * kBM, bar);
        tma_load_2d(dst + w_bytes / 2, &tmW, k, EPI == EPI_SWIGLU ? e.f + wtile * 64 : wtile * kBM + 64, bar);
      };
      auto load_a = [&](int it) {
        const int ti = it / nkb, kb = it - ti * nkb, ttile = (cluster_id + ti * n_clusters) % n_ttiles;
        const int s = it % stages;
        tma_load_2d(tiles + uint32_t(s) * stage_bytes + w_bytes, &tmA, (kb0 + kb) * kBK, ttile * NT,
                    smem_u32(&full_bar[s]));
      };
      // The weights do not depend on the kernel before this one: fill the ring with weight
      // tiles first, and only then wait for the previous kernel's results (the activations).
      const int pre = min(stages, total_it);
      for (int it = 0; it < pre; ++it) { mbar_expect_tx(smem_u32(&full_bar[it % stages]), stage_bytes); load_w(it); }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int it = 0; it < pre; ++it) load_a(it);
      bool ok = true;
      int it = pre;
      for (; it < total_it; ++it) {
        const int s = it % stages;
        ok = mbar_wait(smem_u32(&empty_bar[s]), ((it / stages) - 1) & 1, &abort_flag);
        if (!ok) break;
        mbar_expect_tx(smem_u32(&full_bar[s]), stage_bytes);
        load_w(it);
        load_a(it);
      }
      if (!ok)  // drain copies still in flight before the CTA may exit
        for (int j = max(0, it - stages); j < it; ++j) mbar_drain(smem_u32(&full_bar[j % stages]), (j / stages) & 1);
      // Warm the L2 with the head of the next kernel's weights: HBM would otherwise idle while
      // the last epilogue, the exit and the next kernel's start-up run.
      if (ok) {
        prefetch_l2(e.next_w, e.next_bytes, blockIdx.x, gridDim.x);
        prefetch_l2(e.next_w2, e.next_bytes2, blockIdx.x, gridDim.x);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {  // ---- MMA issuer ----
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(NT >> 3) << 17) | (uint32_t(kBM >> 4) << 24);
      int it = 0, i = 0;
      bool ok = true;
      for (int t = cluster_id; t < n_tiles && ok; t += n_clusters, ++i) {
        const int buf = i & 1;
        if (i >= 2) ok = mbar_wait(smem_u32(&acc_empty[buf]), ((i >> 1) - 1) & 1, &abort_flag);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_acc = tmem_base + uint32_t(buf * kAccCols);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % stages;
          ok = mbar_wait(smem_u32(&full_bar[s]), (it / stages) & 1, &abort_flag);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t w_addr = tiles + uint32_t(s) * stage_bytes;
          const uint64_t wdesc = umma_desc(w_addr), adesc = umma_desc(w_addr + w_bytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)  // 16 bf16 = 32 bytes further along K inside the swizzle span
            umma_bf16(tmem_acc, wdesc + uint64_t(k * 2), adesc + uint64_t(k * 2), idesc, (kb | k) != 0);
          umma_commit(smem_u32(&empty_bar[s]));
        }
        if (ok) umma_commit(smem_u32(&acc_full[buf]));  // arrives when the tile's MMAs have finished
      }
    }
  } else {
    // ---- epilogue warps ----
    asm volatile("griddepcontrol.wait;" ::: "memory");   // everything below reads or overwrites earlier results
    const int et = threadIdx.x - 64, ew = warp - 2;
    const int quarter = warp & 3;  // a warp may only touch its own 32 TMEM lanes
    int i = 0, cur_ttile = -1;
    bool ok = true;
    for (int t = cluster_id; t < n_tiles && ok; t += n_clusters, ++i) {
      const int ttile = t % n_ttiles, wtile = t / n_ttiles, buf = i & 1;
      const int r0 = ttile * NT, n0 = wtile * kBM;
      // Global operands of the fused epilogue (residual, rotary table, gains) do not depend on
      // this kernel: ask for the first groups now, long before the accumulator is ready.
      const int own = min(slice, NT - krank * slice);
      const int nfeat = n0 + 4 * lane;
      auto fetch_operands = [&](int jj, float4& g0, float4& g1) {
        g0 = make_float4(0.f, 0.f, 0.f, 0.f); g1 = g0;
        const int r = r0 + krank * slice + jj;
        if (jj < own && r < e.R_rows && nfeat < N) {
          if (EPI == EPI_RESID) g0 = *reinterpret_cast<const float4*>(e.resid + size_t(r) * N + nfeat);
          if (EPI == EPI_QKV && nfeat < (e.H + e.Hkv) * e.dh) {
            const float* cs = e.rope + (size_t(r) * (e.dh >> 1) + (nfeat % e.dh) % (e.dh >> 1)) * 2;
            g0 = *reinterpret_cast<const float4*>(cs);       // c0 s0 c1 s1
            g1 = *reinterpret_cast<const float4*>(cs + 4);   // c2 s2 c3 s3
          }
        }
      };
      uint2 gain4 = make_uint2(0u, 0u);   // gains of this lane's four features (next norm)
      if (EPI == EPI_RESID && nfeat < N) gain4 = *reinterpret_cast<const uint2*>(e.gain_next + nfeat);
      float4 pg0[kPre][kBatch], pg1[kPre][kBatch];
#pragma unroll
      for (int k = 0; k < kPre; ++k)
#pragma unroll
        for (int b = 0; b < kBatch; ++b) fetch_operands((ew + 4 * k) * kBatch + b, pg0[k][b], pg1[k][b]);
      if (ttile != cur_ttile) {  // per-row scale and cache coordinates of this token tile
        cur_ttile = ttile;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        for (int j = et; j < NT; j += 128) {
          const int r = r0 + j;
          float rstd = 1.f;
          int pos = -1, page = 0;
          if (r < e.R_rows) {
            if (e.sumsq_in) {
              float ss = 0.f;
              for (int tt = 0; tt < e.sumsq_in_tiles; ++tt) ss += e.sumsq_in[size_t(tt) * e.sumsq_ld + r];
              rstd = rsqrtf(ss * e.inv_d + e.eps);
            }
            if (EPI == EPI_QKV) {
              pos = e.row_pos[r];
              if (pos >= 0) page = e.page_table[size_t(e.row_seq[r]) * e.pages_per_seq + (pos >> 4)];
            }
          }
          s_rstd[j] = rstd; s_pos[j] = pos; s_page[j] = page;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
      ok = mbar_wait(smem_u32(&acc_full[buf]), (i >> 1) & 1, &abort_flag);
      // the owners must have finished summing the previous tile before their buffers are overwritten
      if (ok && splits > 1 && i >= 1) ok = mbar_wait_cluster(smem_u32(&red_free), (i - 1) & 1, &abort_flag);
      ok = epilogue_all(ok);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // send every token column of this partial tile to its owner: [rank][column][128 features]
      const uint32_t tmem_acc = tmem_base + uint32_t(buf * kAccCols) + (uint32_t(quarter * 32) << 16);
      // columns are read 48 at a time (three loads in flight, one wait) and go to the owner of
      // their slice; an owner's base address is mapped once, columns are 512 B apart behind it
      for (int owner = 0; owner < splits; ++owner) {
        const int c_lo = owner * slice, c_hi = min(NT, c_lo + slice);
        const uint32_t local = red_addr + uint32_t(((krank * slice) * kBM + quarter * 32 + lane) * 4);
        const uint32_t base = splits > 1 ? map_to_rank(local, uint32_t(owner)) : local;
        for (int c = c_lo; c < c_hi; c += 48) {   // reads past c_hi stay inside the 256-column buffer
          uint32_t v0[16], v1[16], v2[16];
          tmem_ld16(tmem_acc + uint32_t(c), v0);
          if (c + 16 < c_hi) tmem_ld16(tmem_acc + uint32_t(c + 16), v1);
          if (c + 32 < c_hi) tmem_ld16(tmem_acc + uint32_t(c + 32), v2);
          tmem_ld_wait();
          const uint32_t dst = base + uint32_t(c - c_lo) * (kBM * 4);
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            if (c + x < c_hi) st_cluster_f32(dst + x * (kBM * 4), __uint_as_float(v0[x]));
            if (c + 16 + x < c_hi) st_cluster_f32(dst + (16 + x) * (kBM * 4), __uint_as_float(v1[x]));
            if (c + 32 + x < c_hi) st_cluster_f32(dst + (32 + x) * (kBM * 4), __uint_as_float(v2[x]));
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) {
        mbar_arrive(smem_u32(&acc_empty[buf]));   // the accumulator may be overwritten
        if (splits > 1) {
          asm volatile("fence.acq_rel.cluster;" ::: "memory");
          for (int rk = 0; rk < splits; ++rk) mbar_arrive_cluster(map_to_rank(smem_u32(&red_full), uint32_t(rk)));
        }
      }
      if (splits > 1) {
        ok = epilogue_all(mbar_wait_cluster(smem_u32(&red_full), i & 1, &abort_flag));
        if (!ok) break;
      }
      // sum the partial columns this CTA owns (ranks in order) and finish them
      // One group = kBatch columns: all partial columns of the group are read from shared
      // memory first (independent loads), then summed in rank order and finished.  Warp w takes
      // groups w, w+4, w+8, ...; the first kPre groups use the operands requested at the top
      // of the tile loop, later groups ask now.
      auto finish_group = [&](int jb, const float4 (&g0)[kBatch], const float4 (&g1)[kBatch]) {
        float4 part[kBatch][4];
#pragma unroll
        for (int b = 0; b < kBatch; ++b)
#pragma unroll
          for (int rk = 0; rk < 4; ++rk)
            if (rk < splits && jb + b < own) part[b][rk] = ld_shared_f4(red_addr + uint32_t(((rk * slice + jb + b) * kBM + 4 * lane) * 4));
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int jj = jb + b;
          if (jj >= own) break;
          float4 v = part[b][0];
#pragma unroll
          for (int rk = 1; rk < 4; ++rk)
            if (rk < splits) { v.x += part[b][rk].x; v.y += part[b][rk].y; v.z += part[b][rk].z; v.w += part[b][rk].w; }
          const int j = krank * slice + jj, r = r0 + j;
          if (r >= e.R_rows) continue;   // the last token tile may overhang the buffers
          const float rstd = s_rstd[j];
          if (EPI == EPI_PLAIN) epi_plain(e, r, n0, lane, v, rstd, N);
          else if (EPI == EPI_RESID) epi_resid(e, r, n0, lane, v, N, wtile, g0[b], gain4);
          else if (EPI == EPI_SWIGLU) epi_swiglu(e, r, wtile * 64, lane, v, rstd);
          else epi_qkv(e, r, n0, lane, v, rstd, N, s_pos[j], s_page[j], g0[b], g1[b]);
        }
      };
#pragma unroll
      for (int k = 0; k < kPre; ++k)
        if ((ew + 4 * k) * kBatch < own) finish_group((ew + 4 * k) * kBatch, pg0[k], pg1[k]);
      for (int jb = (ew + 4 * kPre) * kBatch; jb < own; jb += 4 * kBatch) {
        float4 g0[kBatch], g1[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) fetch_operands(jb + b, g0[b], g1[b]);
        finish_group(jb, g0, g1);
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");   // buffer fully read
      if (splits > 1 && et == 0)
        for (int rk = 0; rk < splits; ++rk) mbar_arrive_cluster(map_to_rank(smem_u32(&red_free), uint32_t(rk)));
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (splits > 1) cluster_sync_all();  // nobody leaves while a peer may still write to it
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * kAccCols) : "memory");
  }
  if (threadIdx.x == 0 && abort_flag) {
    atomicCAS(status, 0, LASER_ERR_TIMEOUT);
  }
}

// ---- host side --------------------------------------------------------------------------
struct GemmState {
  // (pointer, rows, cols, box rows) -> tensor map
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> maps;
  bool ready = false;
  int max_clusters[5] = {0, 0, 0, 0, 0};   // co-resident clusters of size 1, 2, 4 (index = size)
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

struct TcShape { int n_ttiles, NT, stages; size_t smem; };

TcShape tc_shape(int R_pad, int splits) {
  TcShape s;
  s.n_ttiles = ceil_div(R_pad, kMaxNT);
  s.NT = ceil_div(ceil_div(R_pad, s.n_ttiles), 16) * 16;
  const int stage_bytes = kBM * 128 + s.NT * 128;
  const int red_bytes = splits * ceil_div(s.NT, splits) * kBM * 4;
  s.stages = std::max(2, std::min(kMaxStages, (kSmemLimit - 1024 - red_bytes) / stage_bytes));
  s.smem = size_t(s.stages) * stage_bytes + red_bytes + 1024;
  return s;
}

template <int EPI>
void fill_launch(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int grid, int splits, size_t smem, cudaStream_t stream) {
  *cfg = cudaLaunchConfig_t{};
  cfg->gridDim = dim3(unsigned(grid), 1, 1);
  cfg->blockDim = dim3(kTcThreads, 1, 1);
  cfg->dynamicSmemBytes = smem;
  cfg->stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(splits);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // programmatic dependent launch: this kernel may begin while the previous one drains; it
  // orders itself with griddepcontrol.wait
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg->attrs = attr;
  cfg->numAttrs = 2;
}

template <int EPI>
laser_status launch_epi(const CUtensorMap& tw, const CUtensorMap& ta, const GemmEpilogue& e, int N, const TcShape& sh,
                        int n_wtiles, int total_kb, int kbps, int splits, int clusters, int32_t* status,
                        cudaStream_t stream) {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  fill_launch<EPI>(&cfg, attr, clusters * splits, splits, sh.smem, stream);
  LASER_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<EPI>, tw, ta, e, N, sh.NT, sh.n_ttiles, n_wtiles, total_kb, kbps,
                                splits, sh.stages, status));
  return LASER_OK;
}

// One-off per model: opt in to large shared memory and ask how many clusters of each size fit.
laser_status prepare(GemmState* st) {
  if (st->ready) return LASER_OK;
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
  LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_QKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit));
  int sms = 0, dev = 0;
  LASER_CUDA(cudaGetDevice(&dev));
  LASER_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  for (int s : {1, 2, 4}) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    fill_launch<EPI_RESID>(&cfg, attr, (sms / s) * s, s, size_t(kSmemLimit) - 8192, nullptr);
    int n = 0;
    cudaError_t err = cudaOccupancyMaxActiveClusters(&n, gemm_tc_kernel<EPI_RESID>, &cfg);
    if (err != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    st->max_clusters[s] = std::max(0, std::min(n, sms / s));
  }
  if (st->max_clusters[1] <= 0) { set_error("the GEMM kernel does not fit this device"); return LASER_ERR_UNSUPPORTED; }
  st->ready = true;
  return LASER_OK;
}

}  // namespace
// Tuning aid: a non-zero value overrides the modelled choice of the split count.
int g_force_splits = 0;
namespace {

// Split count (cluster size) with the least modelled time: clusters work in lock step on one
// tile each, a tile costs the K blocks of one rank plus a fixed share.
int pick_splits(const GemmState* st, int R_pad, int N, int K, int epi, int* clusters_out) {
  const int n_wtiles = epi == EPI_SWIGLU ? ceil_div(N / 2, 64) : ceil_div(N, kBM);
  const int total_kb = ceil_div(K, kBK);
  int best = 1, best_clusters = 1;
  double best_cost = 1e30;
  for (int s : {1, 2, 4}) {
    if (st->max_clusters[s] <= 0 || (g_force_splits && s != g_force_splits)) continue;
    const int kbps = ceil_div(total_kb, s);
    if (kbps * (s - 1) >= total_kb) continue;  // a rank would have no K blocks
    const int tiles = n_wtiles * tc_shape(R_pad, s).n_ttiles;
    const int clusters = std::min(st->max_clusters[s], tiles);
    const double cost = double(ceil_div(tiles, clusters)) * (kbps + 1.5) + 2.0 + 0.5 * s;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; best_clusters = clusters; }
  }
  *clusters_out = best_clusters;
  return best;
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
  int clusters = 1;
  const int splits = pick_splits(st, R_pad, N, K, epi, &clusters);
  const TcShape sh = tc_shape(R_pad, splits);
  const CUtensorMap *tw = nullptr, *ta = nullptr;
  LASER_TRY(tensor_map(st, W, N, K, 64, &tw));
  LASER_TRY(tensor_map(st, A, m->R_pad, K, sh.NT, &ta));
  const int total_kb = ceil_div(K, kBK), kbps = ceil_div(total_kb, splits);
  const int n_wtiles = epi == EPI_SWIGLU ? ceil_div(N / 2, 64) : ceil_div(N, kBM);
  switch (epi) {
    case EPI_PLAIN: LASER_TRY(launch_epi<EPI_PLAIN>(*tw, *ta, e, N, sh, n_wtiles, total_kb, kbps, splits, clusters, m->status, stream)); break;
    case EPI_RESID: LASER_TRY(launch_epi<EPI_RESID>(*tw, *ta, e, N, sh, n_wtiles, total_kb, kbps, splits, clusters, m->status, stream)); break;
    case EPI_SWIGLU: LASER_TRY(launch_epi<EPI_SWIGLU>(*tw, *ta, e, N, sh, n_wtiles, total_kb, kbps, splits, clusters, m->status, stream)); break;
    default: LASER_TRY(launch_epi<EPI_QKV>(*tw, *ta, e, N, sh, n_wtiles, total_kb, kbps, splits, clusters, m->status, stream)); break;
  }
  count_launch();
  return LASER_OK;
}

void gemm_state_free(laser_model* m) {
  delete static_cast<GemmState*>(m->gemm_state);
  m->gemm_state = nullptr;
}

}  // namespace laser
