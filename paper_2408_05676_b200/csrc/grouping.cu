// Collaborative-based Grouping (Section 3.2): embeddings of users / items are clustered with K-means
// and every cluster gets its own retrieval pool.  This file holds the clustering itself - Lloyd's
// iteration over fp32 embeddings - so that group ids can be produced on the device next to the pools.
//
// Assignment: one warp per point; a lane keeps the point's coordinates d = lane, lane + 32, .. in
// registers, centroids are read from shared memory; the squared distance to each centroid is the
// lanes' partial sums combined by an xor-shuffle tree (a fixed order: run-to-run identical), ties go
// to the smaller cluster index.  Update: per-cluster sums with fp32 atomics (their order is not fixed,
// so centroids agree between runs to summation accuracy only), then a division; a cluster without
// points keeps its centroid.
#include "common.cuh"

namespace laser {
namespace {

constexpr int kMaxDim = 256;      // coordinates per lane: kMaxDim / 32
constexpr int kAssignWarps = 8;

__global__ void __launch_bounds__(kAssignWarps * 32)
kmeans_assign_kernel(const float* __restrict__ X, int64_t n, int dim, const float* __restrict__ C, int k,
                     int32_t* __restrict__ assign, float* __restrict__ sums, int32_t* __restrict__ counts) {
  extern __shared__ float s_c[];                 // [k][dim]
  for (int i = threadIdx.x; i < k * dim; i += blockDim.x) s_c[i] = C[i];
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t pt = int64_t(blockIdx.x) * kAssignWarps + warp; pt < n; pt += int64_t(gridDim.x) * kAssignWarps) {
    float x[kMaxDim / 32];
#pragma unroll
    for (int i = 0; i < kMaxDim / 32; ++i) x[i] = lane + 32 * i < dim ? X[pt * dim + lane + 32 * i] : 0.f;
    float best = INFINITY;
    int besti = 0;
    for (int j = 0; j < k; ++j) {
      float d = 0.f;
#pragma unroll
      for (int i = 0; i < kMaxDim / 32; ++i)
        if (lane + 32 * i < dim) { const float t = x[i] - s_c[j * dim + lane + 32 * i]; d = fmaf(t, t, d); }
      for (int o = 16; o; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      if (d < best) { best = d; besti = j; }     // strict: the first of equal distances stays
    }
    if (lane == 0) { assign[pt] = besti; atomicAdd(&counts[besti], 1); }
#pragma unroll
    for (int i = 0; i < kMaxDim / 32; ++i)
      if (lane + 32 * i < dim) atomicAdd(&sums[size_t(besti) * dim + lane + 32 * i], x[i]);
  }
}

__global__ void kmeans_update_kernel(float* __restrict__ C, const float* __restrict__ sums,
                                     const int32_t* __restrict__ counts, int k, int dim) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= k * dim) return;
  const int c = counts[i / dim];
  if (c > 0) C[i] = sums[i] / float(c);
}

}  // namespace
}  // namespace laser

using namespace laser;

LASER_API laser_status laser_group_kmeans(const float* x, int64_t n, int32_t dim, int32_t k, int32_t iters,
                                          float* centroids, int32_t* assign, int32_t* counts, void* stream_) {
  LASER_REQUIRE(x && centroids && assign && counts, "null argument");
  LASER_REQUIRE(n >= 1 && dim >= 1 && dim <= kMaxDim && k >= 1 && iters >= 1, "n = %lld, dim = %d (1..%d), k = %d, iters = %d",
                (long long)n, dim, kMaxDim, k, iters);
  const size_t smem = size_t(k) * dim * sizeof(float);
  LASER_REQUIRE(smem <= 200 * 1024, "k * dim = %d centroids' coordinates exceed shared memory", k * dim);
  cudaStream_t stream = as_stream(stream_);
  void* scratch = nullptr;
  LASER_TRY(scratch_get(SCRATCH_GROUPING, size_t(k) * dim * sizeof(float), &scratch));
  float* sums = static_cast<float*>(scratch);
  if (smem > 48 * 1024) LASER_CUDA(cudaFuncSetAttribute(kmeans_assign_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)));
  const unsigned blocks = unsigned(std::min<int64_t>((n + kAssignWarps - 1) / kAssignWarps, 148 * 8));
  for (int it = 0; it < iters; ++it) {
    LASER_CUDA(cudaMemsetAsync(sums, 0, size_t(k) * dim * sizeof(float), stream));
    LASER_CUDA(cudaMemsetAsync(counts, 0, size_t(k) * sizeof(int32_t), stream));
    kmeans_assign_kernel<<<blocks, kAssignWarps * 32, smem, stream>>>(x, n, dim, centroids, k, assign, sums, counts);
    kmeans_update_kernel<<<(k * dim + 255) / 256, 256, 0, stream>>>(centroids, sums, counts, k, dim);
    count_launch(2);
  }
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}
