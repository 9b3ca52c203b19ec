// Error reporting, version string and the per-device scratch buffers.
#include <cstdarg>
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace laser {

static thread_local char t_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(t_err, sizeof(t_err), fmt, ap);
  va_end(ap);
}

long long g_launches = 0;

namespace {
constexpr int kMaxDevices = 64;
struct Scratch { void* ptr = nullptr; size_t bytes = 0; };
Scratch g_scratch[kMaxDevices][SCRATCH_SLOTS];
std::mutex g_scratch_mu;
}  // namespace

laser_status scratch_get(int slot, size_t bytes, void** out) {
  int dev = 0;
  LASER_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) { set_error("device index %d out of range", dev); return LASER_ERR_UNSUPPORTED; }
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  Scratch& s = g_scratch[dev][slot];
  if (s.bytes < bytes) {
    LASER_CUDA(cudaDeviceSynchronize());
    if (s.ptr) LASER_CUDA(cudaFree(s.ptr));
    s.ptr = nullptr; s.bytes = 0;
    size_t want = (bytes + 255) & ~size_t(255);
    LASER_CUDA(cudaMalloc(&s.ptr, want));
    LASER_CUDA(cudaMemset(s.ptr, 0, want));
    s.bytes = want;
  }
  *out = s.ptr;
  return LASER_OK;
}

}  // namespace laser

LASER_API const char* laser_version(void) { return "laser-b200 0.1.0 (sm_100a)"; }
LASER_API const char* laser_last_error(void) { return laser::t_err; }
LASER_API int64_t laser_launch_count(void) { return laser::g_launches; }
