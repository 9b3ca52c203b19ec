// Error reporting, version string and the per-device scratch buffers.
#include <cstdarg>
#include <cstdio>
#include <mutex>

#include "tma.cuh"

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

laser_status tensor_map_encoder(EncodeTiledFn* out) {
  static EncodeTiledFn fn = nullptr;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !p) {
      set_error("cuTensorMapEncodeTiled is not available from the driver");
      return LASER_ERR_UNSUPPORTED;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  *out = fn;
  return LASER_OK;
}

laser_status encode_bf16_2d(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = nullptr;
  LASER_TRY(tensor_map_encoder(&enc));
  const cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
  const cuuint64_t strides[1] = {cuuint64_t(cols) * 2};
  const cuuint32_t box[2] = {64, cuuint32_t(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled failed (%d) for a %llu x %llu bf16 matrix, box %u x 64", int(r),
              (unsigned long long)rows, (unsigned long long)cols, box_rows);
    return LASER_ERR_CUDA;
  }
  return LASER_OK;
}

}  // namespace laser

LASER_API const char* laser_version(void) { return "laser-b200 0.1.0 (sm_100a)"; }
LASER_API const char* laser_last_error(void) { return laser::t_err; }
LASER_API int64_t laser_launch_count(void) { return laser::g_launches; }
