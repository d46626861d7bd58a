// Shared device/host helpers of the NVFP4 library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "nvfp4.h"

namespace nvfp4 {

// ---------------------------------------------------------------------------------------------
// Host-side argument helpers
// ---------------------------------------------------------------------------------------------
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Checks that the current device is a compute-capability 10.x part (cached per device).
int check_arch();

// ---------------------------------------------------------------------------------------------
// Scale-factor layout (128 rows x 4 blocks per 512-byte tile, k-tiles contiguous per row tile)
// ---------------------------------------------------------------------------------------------
__host__ __device__ inline int64_t sf_swizzled_offset(int64_t r, int64_t kb, int64_t k_tiles) {
  return ((r >> 7) * k_tiles + (kb >> 2)) * 512 + (r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3);
}

// ---------------------------------------------------------------------------------------------
// Number formats (Section 3 of the paper)
// ---------------------------------------------------------------------------------------------
// Unsigned E4M3 of a non-negative float: round to nearest even, saturate at 448.
__device__ __forceinline__ uint32_t e4m3_encode(float v) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(v));
  return r & 0xFFu;
}

// Exact value of an unsigned E4M3 code (0..0x7E).
__device__ __forceinline__ float e4m3_decode(uint32_t q) {
  return (q < 8u) ? __uint2float_rn(q) * 0x1p-9f : __uint_as_float((q << 20) + (120u << 23));
}

// Two floats -> one byte of E2M1 codes (lo in bits 0-3, hi in bits 4-7), nearest even, clamp at 6.
__device__ __forceinline__ uint32_t e2m1x2_rn(float lo, float hi) {
  uint32_t r;
  asm("{\n\t.reg .b8 t;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\t"
      "mov.b32 %0, {t, 0, 0, 0};\n\t}"
      : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al. 2011): key = seed, counter = (block index, offset)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                                               uint32_t c2, uint32_t c3) {
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c2 = hi0 ^ c3 ^ k1;
    c1 = lo1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// ---------------------------------------------------------------------------------------------
// Per-element rounding of a magnitude y in [0, 6] to a 3-bit E2M1 magnitude code
// ---------------------------------------------------------------------------------------------
// Stochastic rounding with one random byte u: round up iff (u + 0.5)/256 < frac(y / spacing).
// Below 1 the value is first moved to [1,2) by a round-up add (an order-preserving map onto the
// same 0.5 spacing); then adding (255-u)*2^14 + 0x1FFF to the float's bits carries into the kept
// mantissa bit exactly when the dropped 22 bits exceed (2u+1)*2^13.
__device__ __forceinline__ uint32_t e2m1_sr(float y, uint32_t u) {
  const bool small = y < 1.0f;
  const float w = small ? __fadd_ru(y, 1.0f) : y;
  const uint32_t z = __float_as_uint(w) + 0x3FDFFFu - (u << 14);
  return (z >> 22) - (small ? 254u : 252u);
}

}  // namespace nvfp4
