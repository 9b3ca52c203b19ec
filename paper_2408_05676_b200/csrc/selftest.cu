// Self-test of the failure path every TMA-fed kernel of the library shares: a bounded mbarrier
// wait that runs out must end the wait, raise the CTA's abort flag, let the producer drain the
// copies it still has in flight, and surface LASER_ERR_TIMEOUT through the model's status word -
// leaving the context usable.  Nothing faults or hangs: the wait is on a barrier nobody arrives
// on, with a limit the caller passes (the production limit kWaitCycles is not touched).
#include "model.cuh"
#include "tma.cuh"

namespace laser {
namespace {

// report[0] = 1 when the starved wait returned false, report[1] = 1 when the abort flag was raised,
// report[2] = 1 when the drain saw the in-flight copy land, report[3] = cycles the wait took (clamped)
__global__ void __launch_bounds__(64)
selftest_wait_kernel(const float* __restrict__ src, long long limit_cycles, int32_t* __restrict__ status,
                     int32_t* __restrict__ report) {
  __shared__ __align__(128) float landing[64];
  __shared__ uint64_t starved_bar, copy_bar;
  __shared__ int abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&starved_bar), 1);
    mbar_init(smem_u32(&copy_bar), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == 0) {           // consumer role: waits for data that never comes
    if (lane == 0) {
      const long long t0 = clock64();
      const bool ok = mbar_wait(smem_u32(&starved_bar), 0, &abort_flag, limit_cycles);
      const long long dt = clock64() - t0;
      report[0] = ok ? 0 : 1;
      report[3] = int32_t(dt > 0x7fffffffLL ? 0x7fffffffLL : dt);
    }
  } else if (lane == 0) {    // producer role: one bulk copy in flight, then it learns of the abort
    mbar_expect_tx(smem_u32(&copy_bar), sizeof(landing));
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(landing)), "l"(src), "r"(uint32_t(sizeof(landing))), "r"(smem_u32(&copy_bar)) : "memory");
    const long long t0 = clock64();
    while (!*(volatile int*)&abort_flag && clock64() - t0 < 4 * limit_cycles + 1000000LL) {}
    report[1] = *(volatile int*)&abort_flag ? 1 : 0;
    report[2] = mbar_drain(smem_u32(&copy_bar), 0) ? 1 : 0;   // the copy must have landed before the CTA exits
  }
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) atomicCAS(status, 0, LASER_ERR_TIMEOUT);
}

}  // namespace
}  // namespace laser

LASER_API laser_status laser_selftest_wait(laser_model* m, int64_t limit_cycles, int32_t* report, void* stream) {
  using namespace laser;
  LASER_REQUIRE(m && report, "null argument");
  LASER_REQUIRE(limit_cycles >= 1000 && limit_cycles <= 2000000000LL, "limit_cycles = %lld outside [1e3, 2e9]", (long long)limit_cycles);
  selftest_wait_kernel<<<1, 64, 0, as_stream(stream)>>>(m->resid, (long long)limit_cycles, m->status, report);
  count_launch();
  LASER_CUDA(cudaGetLastError());
  return LASER_OK;
}
