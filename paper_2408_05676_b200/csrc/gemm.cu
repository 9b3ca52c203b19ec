// Dense contractions of the verify forward (QKV, O, gate/up, down, LM head):
// out[r][n] = sum_k A[r][k] * W[n][k], bf16 operands, fp32 accumulation.
//
// The token rows are few (batch x (K+1)) and the weight matrices are large, so the weight
// rows take the 128-wide M side of the MMA and the token rows the N side: a 128 x NT
// accumulator in tensor memory, NT <= 256 token rows, no padding of the rows to 128.
// Split-K partial sums go to separate planes that the consumer kernel adds in a fixed
// order, which keeps the result independent of scheduling.
//
// Tensor-memory kernel (tcgen05): one CTA per (token tile, weight tile, K range), two CTAs
// resident per SM.  Warp 0 streams 128x64 weight tiles and NTx64 activation tiles with TMA
// (128-byte swizzle) through a ring of shared-memory stages; warp 1 issues tcgen05.mma
// (M=128, N=NT, K=16) from shared-memory descriptors into a TMEM accumulator and releases
// stages with tcgen05.commit; warps 2-5 read the accumulator with tcgen05.ld and store it
// transposed (token-major).  Every wait is bounded: on expiry the CTA records
// LASER_ERR_TIMEOUT, drains its copies, frees its TMEM and exits.
#include <map>
#include <tuple>

#include "model.cuh"
#include "tma.cuh"

namespace laser {
namespace {

// ---------------------------------------------------------------------------------------
// Warp-level MMA kernel (mma.sync m16n8k16).  Serves shapes the tensor-memory kernel does
// not cover.  Each warp owns 8 weight rows and walks all token rows in groups of MT tiles
// of 16; operands are read straight from global memory / L1 in fragment layout.
// ---------------------------------------------------------------------------------------
constexpr int kMmaWarps = 4;

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int MT>
__global__ void __launch_bounds__(kMmaWarps * 32)
gemm_mma_kernel(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ W,
                float* __restrict__ out, int R_pad, int R_store, int N, int K, int k_per_split,
                size_t split_stride, int ldo) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = (blockIdx.x * kMmaWarps + warp) * 8;
  if (n0 >= N) return;
  const int g = lane >> 2, t2 = (lane & 3) * 2;
  const int kb = blockIdx.y * k_per_split, ke = min(K, kb + k_per_split);
  const __nv_bfloat16* wrow = W + size_t(n0 + g) * K + t2;
  float* o = out + size_t(blockIdx.y) * split_stride;
  for (int m0 = 0; m0 < R_pad; m0 += MT * 16) {
    float acc[MT][4];
#pragma unroll
    for (int t = 0; t < MT; ++t) acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f;
    for (int k = kb; k < ke; k += 16) {
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(wrow + k);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(wrow + k + 8);
#pragma unroll
      for (int t = 0; t < MT; ++t) {
        const int r = m0 + t * 16 + g;
        if (m0 + t * 16 < R_pad) {
          const __nv_bfloat16* a = A + size_t(r) * K + k + t2;
          const uint32_t a0 = *reinterpret_cast<const uint32_t*>(a);
          const uint32_t a1 = *reinterpret_cast<const uint32_t*>(a + size_t(8) * K);
          const uint32_t a2 = *reinterpret_cast<const uint32_t*>(a + 8);
          const uint32_t a3 = *reinterpret_cast<const uint32_t*>(a + size_t(8) * K + 8);
          mma_bf16_16816(acc[t], a0, a1, a2, a3, b0, b1);
        }
      }
    }
#pragma unroll
    for (int t = 0; t < MT; ++t) {
      const int r = m0 + t * 16 + g;
      if (m0 + t * 16 < R_pad) {
        if (r < R_store) *reinterpret_cast<float2*>(o + size_t(r) * ldo + n0 + t2) = make_float2(acc[t][0], acc[t][1]);
        if (r + 8 < R_store) *reinterpret_cast<float2*>(o + size_t(r + 8) * ldo + n0 + t2) = make_float2(acc[t][2], acc[t][3]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Tensor-memory kernel
// ---------------------------------------------------------------------------------------
constexpr int kTcThreads = 192;
constexpr int kBM = 128;          // weight rows per tile (MMA M)
constexpr int kBK = 64;           // K elements per stage = one 128-byte swizzle span of bf16
constexpr int kMaxStages = 6;
constexpr int kMaxNT = 256;
// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows 128 B apart, groups
// of 8 rows 1024 B apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= uint64_t((smem_addr & 0x3FFFF) >> 4);        // start address
  d |= uint64_t(0) << 16;                           // leading byte offset: unused for swizzled K-major
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

__global__ void __launch_bounds__(kTcThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA,
               float* __restrict__ out, int N, int R_store, int NT, int total_kb, int kb_per_split, int stages,
               size_t split_stride, int ldo, int tmem_cols, int32_t* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
  const uint32_t w_bytes = kBM * 128, a_bytes = uint32_t(NT) * 128, stage_bytes = w_bytes + a_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = blockIdx.x * NT, n0 = blockIdx.y * kBM;
  const int kb0 = blockIdx.z * kb_per_split;
  const int nkb = min(kb_per_split, total_kb - kb0);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
    mbar_init(smem_u32(&acc_bar), 1);
    mbar_fence_init();
    tma_prefetch_map(&tmW);
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

  if (warp == 0) {
    if (lane == 0) {  // TMA producer
      int issued = 0;
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const int s = kb % stages;
        if (kb >= stages) ok = mbar_wait(smem_u32(&empty_bar[s]), ((kb / stages) - 1) & 1, &abort_flag);
        if (!ok) break;
        const uint32_t bar = smem_u32(&full_bar[s]);
        const uint32_t dst = tiles + uint32_t(s) * stage_bytes;
        mbar_expect_tx(bar, stage_bytes);
        tma_load_2d(dst, &tmW, (kb0 + kb) * kBK, n0, bar);
        tma_load_2d(dst + w_bytes, &tmA, (kb0 + kb) * kBK, r0, bar);
        issued = kb + 1;
      }
      if (!ok) {  // drain copies still in flight before the CTA may exit
        for (int kb = max(0, issued - stages); kb < issued; ++kb)
          mbar_drain(smem_u32(&full_bar[kb % stages]), (kb / stages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {  // MMA issuer
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(NT >> 3) << 17) | (uint32_t(kBM >> 4) << 24);
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const int s = kb % stages;
        ok = mbar_wait(smem_u32(&full_bar[s]), (kb / stages) & 1, &abort_flag);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t w_addr = tiles + uint32_t(s) * stage_bytes;
        const uint64_t wdesc = umma_desc(w_addr), adesc = umma_desc(w_addr + w_bytes);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k)  // 16 bf16 = 32 bytes further along K inside the swizzle span
          umma_bf16(tmem_acc, wdesc + uint64_t(k * 2), adesc + uint64_t(k * 2), idesc, (kb | k) != 0);
        umma_commit(smem_u32(&empty_bar[s]));
      }
      umma_commit(smem_u32(&acc_bar));  // arrives when every MMA issued so far has finished
    }
  } else {  // epilogue warps: TMEM lane quarter = warp id modulo 4
    const int quarter = warp & 3;
    const bool ok = mbar_wait(smem_u32(&acc_bar), 0, &abort_flag);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok && nkb > 0) {
      const int n = n0 + quarter * 32 + lane;
      float* o = out + size_t(blockIdx.z) * split_stride + n;
      for (int c = 0; c < NT; c += 16) {
        uint32_t v[16];
        const uint32_t taddr = tmem_acc + (uint32_t(quarter * 32) << 16) + uint32_t(c);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(taddr) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (n < N) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int r = r0 + c + i;
            if (r < R_store) o[size_t(r) * ldo] = __uint_as_float(v[i]);
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
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
};

laser_status get_state(laser_model* m, GemmState** out) {
  if (!m->gemm_state) m->gemm_state = new GemmState();
  *out = static_cast<GemmState*>(m->gemm_state);
  return LASER_OK;
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

struct TcShape { int n_tiles, NT, stages, tmem_cols; size_t smem; };

TcShape tc_shape(int R_pad) {
  TcShape s;
  s.n_tiles = ceil_div(R_pad, kMaxNT);
  s.NT = ceil_div(ceil_div(R_pad, s.n_tiles), 16) * 16;
  const int stage_bytes = kBM * 128 + s.NT * 128;
  s.stages = std::max(2, std::min(kMaxStages, (110 * 1024) / stage_bytes));
  s.tmem_cols = 32;
  while (s.tmem_cols < s.NT) s.tmem_cols <<= 1;
  s.smem = size_t(s.stages) * stage_bytes + 1024;
  return s;
}

bool tc_ok(int N, int K) { return K % 8 == 0 && N >= 1 && K >= 8; }

}  // namespace

GemmPlan gemm_plan(int R_pad, int N, int K) {
  if (!tc_ok(N, K)) {
    const int blocks = ceil_div(N, 8 * kMmaWarps);
    int splits = std::max(1, std::min(8, ceil_div(296, blocks)));
    while (splits > 1 && ceil_div(ceil_div(K, splits), 16) * 16 * (splits - 1) >= K) --splits;
    return GemmPlan{splits};
  }
  // Pick the split count with the least modelled time: CTAs are spread over 148 SMs, each
  // costs its K blocks plus a fixed prologue/epilogue share, each extra plane costs a little.
  const TcShape sh = tc_shape(R_pad);
  const int tiles = ceil_div(N, kBM) * sh.n_tiles, total_kb = ceil_div(K, kBK);
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= std::min(total_kb, 16); ++s) {
    const int kbps = ceil_div(total_kb, s);
    if (kbps * (s - 1) >= total_kb) continue;  // a split would be empty
    const double cost = double(ceil_div(tiles * s, 148)) * (kbps + 3.0) + 0.4 * s;
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  return GemmPlan{best};
}

laser_status gemm_launch(laser_model* m, const __nv_bfloat16* A, const __nv_bfloat16* W, float* out,
                         int R_pad, int R_store, int N, int K, int splits, size_t split_stride, int ldo,
                         cudaStream_t stream) {
  if (R_pad % 16 != 0) { set_error("GEMM rows %d not a multiple of 16", R_pad); return LASER_ERR_UNSUPPORTED; }
  if (tc_ok(N, K) && (reinterpret_cast<uintptr_t>(A) & 15) == 0 && (reinterpret_cast<uintptr_t>(W) & 15) == 0) {
    GemmState* st = nullptr;
    LASER_TRY(get_state(m, &st));
    const TcShape sh = tc_shape(R_pad);
    const CUtensorMap *tw = nullptr, *ta = nullptr;
    LASER_TRY(tensor_map(st, W, N, K, kBM, &tw));
    LASER_TRY(tensor_map(st, A, m->R_pad, K, sh.NT, &ta));
    const int total_kb = ceil_div(K, kBK), kbps = ceil_div(total_kb, splits);
    LASER_CUDA(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024));
    dim3 grid(sh.n_tiles, ceil_div(N, kBM), splits);
    gemm_tc_kernel<<<grid, kTcThreads, sh.smem, stream>>>(*tw, *ta, out, N, R_store, sh.NT, total_kb, kbps, sh.stages,
                                                           split_stride, ldo, sh.tmem_cols, m->status);
    count_launch();
    LASER_CUDA(cudaGetLastError());
    return LASER_OK;
  }
  if (N % 8 != 0 || K % 16 != 0) {
    set_error("GEMM shape N=%d K=%d unsupported (need K%%8==0 and 16-byte aligned operands, or N%%8==0 and K%%16==0)", N, K);
    return LASER_ERR_UNSUPPORTED;
  }
  const int k_per_split = ceil_div(ceil_div(K, splits), 16) * 16;
  dim3 grid(ceil_div(N, 8 * kMmaWarps), splits);
  gemm_mma_kernel<9><<<grid, kMmaWarps * 32, 0, stream>>>(A, W, out, R_pad, R_store, N, K, k_per_split,
                                                           split_stride, ldo);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}

void gemm_state_free(laser_model* m) {
  delete static_cast<GemmState*>(m->gemm_state);
  m->gemm_state = nullptr;
}

}  // namespace laser
