// Dense contractions of the verify forward (QKV, O, gate/up, down, LM head):
// out[r][n] = sum_k A[r][k] * W[n][k], bf16 operands, fp32 accumulation.
//
// The token rows are few (batch x (K+1)) and the weight matrices are large, so the weight
// rows take the 128-wide M side of the MMA and the token rows the N side.  Split-K partial
// sums go to separate planes that the consumer kernel adds in a fixed order, which keeps
// the result independent of scheduling.
#include "model.cuh"

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

}  // namespace

GemmPlan gemm_plan(int R_pad, int N, int K) {
  (void)R_pad;
  const int blocks = ceil_div(N, 8 * kMmaWarps);
  int splits = std::max(1, std::min(8, ceil_div(296, blocks)));
  while (splits > 1 && ceil_div(ceil_div(K, splits), 16) * 16 * (splits - 1) >= K) --splits;
  return GemmPlan{splits};
}

laser_status gemm_launch(laser_model* m, const __nv_bfloat16* A, const __nv_bfloat16* W, float* out,
                         int R_pad, int R_store, int N, int K, int splits, size_t split_stride, int ldo,
                         cudaStream_t stream) {
  (void)m;
  if (N % 8 != 0 || K % 16 != 0 || R_pad % 16 != 0) {
    set_error("GEMM shape N=%d K=%d rows=%d unsupported (need N%%8==0, K%%16==0, rows%%16==0)", N, K, R_pad);
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

void gemm_state_free(laser_model* m) { (void)m; }

}  // namespace laser
