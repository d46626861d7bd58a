// Pieces shared by the NVFP4 quantizer kernels: launch constants, the parameter block, the
// per-block encoder (amax -> E4M3 scale -> E2M1 codes, Section 3 and Eq. 4-6) and source-block loads.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"

namespace nvfp4 {

constexpr int kThreads = 256;

struct QuantParams {
  const void* x;
  int64_t rows, cols, ld;
  const float* gptr;
  PhiloxStream rng;
  uint8_t* codes;
  uint8_t* scales;
  int64_t nkb;      // groups of 16 per quantized row (Kq / 16): NVFP4 blocks, and the unit of the random draws
  int64_t k_tiles;  // scale tiles per quantized row: ceil(scale blocks / 4)
  int64_t nsb;      // scale blocks per quantized row: Kq / 16 (NVFP4) or Kq / 32 (MXFP4)
};

// Reciprocal of every block scale a tensor can have: entry q = 1 / (decode(q) * g), one IEEE
// division each, 0 for the zero scale.  A block then costs one shared-memory read, not a division.
__device__ __forceinline__ void build_inv_table(float* inv_table, float g) {
  for (int q = threadIdx.x; q < 128; q += blockDim.x)
    inv_table[q] = (q == 0) ? 0.0f : __fdiv_rn(1.0f, __fmul_rn(e4m3_decode((uint32_t)q), g));
}

// MXFP4: the same table over the 255 E8M0 codes, entry q = 1 / (2^(q-127) * g), 0 for code 0.
__device__ __forceinline__ void build_inv_table_mx(float* inv_table, float g) {
  for (int q = threadIdx.x; q < 256; q += blockDim.x)
    inv_table[q] = (q == 0 || q == 255) ? 0.0f : __fdiv_rn(1.0f, __fmul_rn(__uint_as_float((uint32_t)q << 23), g));
}

// 16 values (signed, already widened to fp32) scaled by inv -> 8 bytes of codes (lo, hi words).
// `blk` is the linear index of this group of 16 (Philox counter).
template <bool SR>
__device__ __forceinline__ void encode_codes(const float (&v)[16], float inv, const PhiloxStream& rng, uint64_t blk,
                                             uint32_t& lo, uint32_t& hi);

// 16 values and their amax -> codes and one E4M3 scale byte.  c = (1/6)/g.
template <bool SR>
__device__ __forceinline__ void encode_block(const float (&v)[16], float amax, float c, const float* inv_table,
                                             const PhiloxStream& rng, uint64_t blk,
                                             uint32_t& lo, uint32_t& hi, uint32_t& sf) {
  const uint32_t q = e4m3_encode(__fmul_rn(amax, c));
  sf = q;
  encode_codes<SR>(v, inv_table[q], rng, blk, lo, hi);
}

template <bool SR>
__device__ __forceinline__ void encode_codes(const float (&v)[16], float inv, const PhiloxStream& rng, uint64_t blk,
                                             uint32_t& lo, uint32_t& hi) {
  float y[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) y[j] = __fmul_rn(v[j], inv);     // the sign rides along; the conversions clamp at 6
  if constexpr (!SR) {
    lo = e2m1x8_rn(y, 0);
    hi = e2m1x8_rn(y, 8);
  } else {
    const uint4 r4 = philox4x32_10(rng, (uint32_t)blk, (uint32_t)(blk >> 32));
    lo = e2m1x8_rs(y, 0, r4.x, r4.y);
    hi = e2m1x8_rs(y, 8, r4.z, r4.w);
  }
}

// max |.| of two packed bf16 pairs, per half (the sign bits of the result are meaningless)
__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// One block of 16 contiguous source values.
template <typename T>
struct Block16;

template <>
struct Block16<__nv_bfloat16> {
  uint32_t w[8];
  __device__ __forceinline__ void load(const __nv_bfloat16* src, bool aligned32) {
    if (aligned32) {
      asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                   : "l"(src));
    } else {
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(src));
      const uint4 b = __ldg(reinterpret_cast<const uint4*>(src) + 1);
      w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w; w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
    }
  }
  __device__ __forceinline__ float unpack(float (&v)[16]) const {
    uint32_t m = absmax_bf16x2(absmax_bf16x2(absmax_bf16x2(w[0], w[1]), absmax_bf16x2(w[2], w[3])),
                               absmax_bf16x2(absmax_bf16x2(w[4], w[5]), absmax_bf16x2(w[6], w[7])));
    m &= 0x7FFF7FFFu;
    const uint32_t top = max(m >> 16, m & 0xFFFFu);            // non-negative bf16 patterns order as integers
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
    return __uint_as_float(top << 16);
  }
};

template <>
struct Block16<float> {
  float4 f[4];
  __device__ __forceinline__ void load(const float* src, bool) {
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = __ldg(reinterpret_cast<const float4*>(src) + i);
  }
  __device__ __forceinline__ float unpack(float (&v)[16]) const {
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[4 * i] = f[i].x; v[4 * i + 1] = f[i].y; v[4 * i + 2] = f[i].z; v[4 * i + 3] = f[i].w;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) amax = fmaxf(amax, fabsf(v[j]));
    return amax;
  }
};

}  // namespace nvfp4
