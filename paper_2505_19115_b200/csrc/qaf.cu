// The backward and update products of the paper's quantization-aware fine-tuning phase (Section 5:
// the forward pass stays in NVFP4, the backward and update GEMMs run in BF16):
//   dX[M,K] = dY[M,N] . W[N,K]          dW[N,K] = dY[M,N]^T . X[M,K]
// Both are computed by the bf16 variant of the CTA-pair GEMM.  The operands that are stored with the output
// axis contiguous (W and X for their own products, dY for the update) are read as they are, through MN-major
// shared-memory descriptors; nvfp4_transpose_bf16 remains as a utility.
#include <cuda_bf16.h>

#include "common.cuh"

namespace nvfp4 {
namespace {

constexpr int kTT = 64;            // tile edge (elements)
constexpr int kTPitch = kTT + 2;   // shared-memory row pitch: column reads hit distinct banks

// out[c, r] = x[r, c] for x[rows, cols] (leading dimension ld), out dense [cols, rows].
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                             int64_t ld, __nv_bfloat16* __restrict__ out) {
  __shared__ __nv_bfloat16 tile[kTT][kTPitch];
  const int64_t r0 = (int64_t)blockIdx.y * kTT, c0 = (int64_t)blockIdx.x * kTT;
  // load: 64 rows x 8 chunks of 8 elements (16 bytes), two chunks per thread
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int id = threadIdx.x + i * 256, row = id >> 3, ch = id & 7;
    const int64_t gr = r0 + row, gc = c0 + ch * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (gr < rows && gc < cols) v = __ldg(reinterpret_cast<const uint4*>(x + gr * ld + gc));   // cols % 8 == 0
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      *reinterpret_cast<uint32_t*>(&tile[row][ch * 8 + 2 * j]) = w[j];
  }
  __syncthreads();
  // store: output row = source column; 8 consecutive source rows make one 16-byte chunk
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int id = threadIdx.x + i * 256, col = id >> 3, ch = id & 7;
    const int64_t gc = c0 + col, gr = r0 + ch * 8;
    if (gc < cols && gr < rows) {                                                               // rows % 8 == 0
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t lo = *reinterpret_cast<const uint16_t*>(&tile[ch * 8 + 2 * j][col]);
        const uint32_t hi = *reinterpret_cast<const uint16_t*>(&tile[ch * 8 + 2 * j + 1][col]);
        w[j] = lo | (hi << 16);
      }
      *reinterpret_cast<uint4*>(out + gc * rows + gr) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

extern "C" int nvfp4_transpose_bf16(const void* x, int64_t rows, int64_t cols, int64_t ld, void* out, void* cuda_stream) {
  if (!x || !out) return NVFP4_ERR_NULL;
  if (rows <= 0 || cols <= 0 || ld < cols || rows % 8 != 0 || cols % 8 != 0) return NVFP4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(out) || (ld % 8) != 0) return NVFP4_ERR_ALIGN;
  if (ceil_div(rows, kTT) > 65535) return NVFP4_ERR_SHAPE;
  if (int st = check_arch()) return st;
  dim3 grid((unsigned)ceil_div(cols, kTT), (unsigned)ceil_div(rows, kTT));
  transpose_bf16_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const __nv_bfloat16*>(x), rows, cols, ld, static_cast<__nv_bfloat16*>(out));
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

extern "C" size_t nvfp4_linear_bwd_bf16_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  (void)M; (void)N; (void)K;
  return 0;                      // the products read W, X and dY as they are stored: nothing is staged
}

extern "C" int nvfp4_linear_bwd_bf16(const void* dY, const void* W, const void* X, int64_t M, int64_t N, int64_t K,
                                     void* dX, int dx_dtype, void* dW, int dw_dtype,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
  (void)workspace; (void)workspace_bytes;
  if (!dY || !W || !X || !dX || !dW) return NVFP4_ERR_NULL;
  if ((dx_dtype != NVFP4_BF16 && dx_dtype != NVFP4_FP32) || (dw_dtype != NVFP4_BF16 && dw_dtype != NVFP4_FP32)) return NVFP4_ERR_ENUM;
  if (M <= 0 || N <= 0 || K <= 0 || M % 16 != 0 || N % 16 != 0 || K % 16 != 0) return NVFP4_ERR_SHAPE;
  if (!aligned16(dY) || !aligned16(W) || !aligned16(X) || !aligned16(dX) || !aligned16(dW)) return NVFP4_ERR_ALIGN;
  // dX[M,K] = dY[M,N] . W[N,K]: contraction over N; dY has N contiguous (K-major operand), W is [contraction, output]
  // with the output axis contiguous (MN-major operand)
  if (int st = nvfp4_gemm_bf16_ex(dY, 0, W, 1, M, K, N, dX, dx_dtype, K, cuda_stream)) return st;
  // dW[N,K] = dY[M,N]^T . X[M,K]: contraction over the token axis M; both operands are [contraction, output]
  return nvfp4_gemm_bf16_ex(dY, 1, X, 1, N, K, M, dW, dw_dtype, K, cuda_stream);
}
