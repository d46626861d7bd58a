// Status strings and the device-architecture check of the NVFP4 library.
#include "common.cuh"

namespace nvfp4 {

int check_arch() {
  static int cached[64];  // 0 = unknown, 1 = ok, 2 = wrong arch
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return NVFP4_ERR_CUDA;
  if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev] == 1 ? NVFP4_OK : NVFP4_ERR_ARCH;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return NVFP4_ERR_CUDA;
  const int ok = (major == 10);
  if (dev >= 0 && dev < 64) cached[dev] = ok ? 1 : 2;
  return ok ? NVFP4_OK : NVFP4_ERR_ARCH;
}

int current_device() {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

int sm_count() {
  static DeviceInts table;
  const int dev = current_device();
  return cached_per_device(table, dev, 148, [&] {
    int n = 0;
    return (dev >= 0 && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) ? n : 0;
  });
}

}  // namespace nvfp4

extern "C" const char* nvfp4_status_string(int status) {
  switch (status) {
    case NVFP4_OK: return "ok";
    case NVFP4_ERR_NULL: return "a required pointer is NULL";
    case NVFP4_ERR_SHAPE: return "bad shape (non-positive size, contraction length not a multiple of 16, or ld too small)";
    case NVFP4_ERR_ALIGN: return "pointer or leading dimension not aligned as required";
    case NVFP4_ERR_ENUM: return "unknown dtype, rounding mode, layout or flag";
    case NVFP4_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case NVFP4_ERR_ARCH: return "the current device is not compute capability 10.x (sm_100a required)";
    case NVFP4_ERR_CUDA: return "a CUDA call or kernel launch failed";
    default: return "unknown status";
  }
}
