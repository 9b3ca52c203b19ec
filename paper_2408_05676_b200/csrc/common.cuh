// Shared host-side helpers of the library: error reporting, argument checks, the
// per-device scratch buffers and small utilities.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/laser.h"

#define LASER_API extern "C" __attribute__((visibility("default")))

namespace laser {

void set_error(const char* fmt, ...);

#define LASER_CUDA(expr)                                                                  \
  do {                                                                                    \
    cudaError_t e_ = (expr);                                                              \
    if (e_ != cudaSuccess) {                                                              \
      ::laser::set_error("%s: %s (%s:%d)", #expr, cudaGetErrorString(e_), __FILE__, __LINE__); \
      return e_ == cudaErrorMemoryAllocation ? LASER_ERR_OOM : LASER_ERR_CUDA;            \
    }                                                                                     \
  } while (0)

#define LASER_REQUIRE(cond, ...)                                                          \
  do {                                                                                    \
    if (!(cond)) {                                                                        \
      ::laser::set_error(__VA_ARGS__);                                                    \
      return LASER_ERR_INVALID_ARG;                                                       \
    }                                                                                     \
  } while (0)

#define LASER_TRY(expr)                                                                   \
  do {                                                                                    \
    laser_status s_ = (expr);                                                             \
    if (s_ != LASER_OK) return s_;                                                        \
  } while (0)

// Scratch of at least `bytes` on the current device for one subsystem (`slot`), 256-byte
// aligned, zero-filled when (re)allocated.  Grows by reallocation (synchronising the
// device), so a pointer is only valid until the next call that asks for more.  Contents
// persist between calls.
enum { SCRATCH_ACCEPT = 0, SCRATCH_DRAFT = 1, SCRATCH_ACCEPT_TREE = 2, SCRATCH_GROUPING = 3, SCRATCH_SLOTS = 4 };
laser_status scratch_get(int slot, size_t bytes, void** out);

// Kernel launch counter (per process) for the statistics.
extern long long g_launches;
inline void count_launch(int n = 1) { g_launches += n; }

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

template <typename T>
inline T ceil_div(T a, T b) { return (a + b - 1) / b; }

}  // namespace laser
