// Quantization-noise monitor (Section 4 of the paper): for a tensor x and its NVFP4 quantization,
//   sums[0] = sum (Q(x) - x)^2   (= d * sigma_q^2)        sums[1] = sum x^2   (= ||x||^2)
// The paper's gradient-to-noise ratio ||x|| / (sigma_q sqrt(d)) is sqrt(sums[1] / sums[0]); training
// should leave FP4 when it falls below sqrt(3).  One streaming pass over x and the codes.
#include <cuda_bf16.h>

#include "common.cuh"

namespace nvfp4 {
namespace {

constexpr int kNoiseThreads = 256;

struct NoiseParams {
  const void* x;
  int64_t rows, cols, ld;
  int transposed;            // quantized shape (Rq, Kq) = transposed ? (cols, rows) : (rows, cols)
  const float* gptr;
  const uint8_t* codes;      // [Rq, Kq/2]
  const uint8_t* scales;
  int64_t nkb, k_tiles;
  int swizzled;
  double* sums;
};

// value of a 4-bit E2M1 code: sign | exponent(2) | mantissa(1)
__device__ __forceinline__ float e2m1_value(uint32_t nib) {
  const uint32_t m = nib & 7u;
  const float mag = (m < 2u) ? 0.5f * (float)m : __uint_as_float(((126u + (m >> 1)) << 23) | ((m & 1u) << 22));
  return (nib & 8u) ? -mag : mag;
}

__device__ __forceinline__ float scale_at(const NoiseParams& p, int64_t qr, int64_t kb) {
  const int64_t off = p.swizzled ? sf_swizzled_offset(qr, kb, p.k_tiles) : qr * p.nkb + kb;
  return e4m3_decode(p.scales[off]);
}

template <typename T>
__global__ void __launch_bounds__(kNoiseThreads) noise_kernel(const NoiseParams p) {
  const float g = p.gptr ? __ldg(p.gptr) : 1.0f;
  const T* x = static_cast<const T*>(p.x);
  const int64_t groups_per_row = p.cols / 8;                 // eight consecutive source elements per step
  const int64_t total = p.rows * groups_per_row;
  float err2 = 0.0f, x2 = 0.0f;
  double derr2 = 0.0, dx2 = 0.0;
  int n_acc = 0;
  for (int64_t i = (int64_t)blockIdx.x * kNoiseThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kNoiseThreads) {
    const int64_t r = i / groups_per_row, c = (i % groups_per_row) * 8;
    float v[8];
    if constexpr (sizeof(T) == 2) {
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(x + r * p.ld + c));
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[2 * j] = __uint_as_float(w[j] << 16);
        v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
      }
    } else {
      const float4 a = __ldg(reinterpret_cast<const float4*>(x + r * p.ld + c));
      const float4 b = __ldg(reinterpret_cast<const float4*>(x + r * p.ld + c) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
    if (!p.transposed) {
      // quantized row r, elements c..c+7: four code bytes, one block scale
      const uint32_t packed = __ldg(reinterpret_cast<const uint32_t*>(p.codes + r * (p.cols / 2) + c / 2));
      const float d = __fmul_rn(scale_at(p, r, c / 16), g);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float e = __fsub_rn(__fmul_rn(e2m1_value((packed >> (4 * j)) & 15u), d), v[j]);
        err2 = __fmaf_rn(e, e, err2);
        x2 = __fmaf_rn(v[j], v[j], x2);
      }
    } else {
      // source element (r, c+j) is element r of quantized row c+j
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int64_t qr = c + j;
        const uint32_t byte = __ldg(p.codes + qr * (p.rows / 2) + r / 2);
        const float d = __fmul_rn(scale_at(p, qr, r / 16), g);
        const float e = __fsub_rn(__fmul_rn(e2m1_value((r & 1) ? (byte >> 4) : (byte & 15u)), d), v[j]);
        err2 = __fmaf_rn(e, e, err2);
        x2 = __fmaf_rn(v[j], v[j], x2);
      }
    }
    if (++n_acc == 16) {                                      // keep the fp32 partial sums short
      derr2 += (double)err2; dx2 += (double)x2;
      err2 = x2 = 0.0f; n_acc = 0;
    }
  }
  derr2 += (double)err2; dx2 += (double)x2;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    derr2 += __shfl_xor_sync(0xFFFFFFFFu, derr2, o);
    dx2 += __shfl_xor_sync(0xFFFFFFFFu, dx2, o);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(p.sums, derr2);
    atomicAdd(p.sums + 1, dx2);
  }
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

extern "C" int nvfp4_quantization_noise(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int transposed,
                                        const float* global_scale, const uint8_t* codes, const uint8_t* scales,
                                        int sf_layout, double* sums, void* cuda_stream) {
  if (!x || !codes || !scales || !sums) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (transposed != 0 && transposed != 1) return NVFP4_ERR_ENUM;
  if (sf_layout != NVFP4_SF_LINEAR && sf_layout != NVFP4_SF_SWIZZLED_128x4) return NVFP4_ERR_ENUM;
  if (rows <= 0 || cols <= 0 || ld < cols || cols % 8 != 0) return NVFP4_ERR_SHAPE;
  const int64_t Kq = transposed ? rows : cols;
  if (Kq % 16 != 0) return NVFP4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(codes) || (ld % 8) != 0 || (reinterpret_cast<uintptr_t>(sums) & 7u)) return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(sums, 0, 2 * sizeof(double), s) != cudaSuccess) return NVFP4_ERR_CUDA;
  NoiseParams p;
  p.x = x; p.rows = rows; p.cols = cols; p.ld = ld; p.transposed = transposed; p.gptr = global_scale;
  p.codes = codes; p.scales = scales; p.nkb = Kq / 16; p.k_tiles = ceil_div(p.nkb, 4);
  p.swizzled = sf_layout == NVFP4_SF_SWIZZLED_128x4; p.sums = sums;
  int64_t blocks = ceil_div(rows * (cols / 8), (int64_t)kNoiseThreads * 4);
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  if (blocks < 1) blocks = 1;
  if (dtype == NVFP4_BF16) noise_kernel<__nv_bfloat16><<<(unsigned)blocks, kNoiseThreads, 0, s>>>(p);
  else noise_kernel<float><<<(unsigned)blocks, kNoiseThreads, 0, s>>>(p);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}
