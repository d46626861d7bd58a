// NVFP4 quantizer kernels (Section 3 and Eq. 4-6 of the paper): block amax -> E4M3 scale ->
// E2M1 codes with round-to-nearest or Philox stochastic rounding, along the contiguous axis
// (row kernel) or along the row axis with a transposed output (transposed kernel), plus the
// per-tensor amax scale.  All kernels are HBM-bound streaming kernels.
#include <cuda_bf16.h>

#include <type_traits>

#include "quantize_core.cuh"

namespace nvfp4 {

namespace {

// -------------------------------------------------------------------------------------------------
// Row quantizer: CTA tile = 128 rows x 32 blocks (512 columns); warp w takes rows w, w+8, ...;
// lane = block within the row segment, so a warp reads 1 KB (bf16) of one row per step (one
// 256-bit load per lane when rows are 32-byte aligned) and writes 256 contiguous code bytes.
// Several rows are in flight per thread, kept packed.  Swizzled scales are staged in shared
// memory and leave as eight contiguous 512-byte tiles.
// -------------------------------------------------------------------------------------------------
constexpr int kRowTileRows = 128;
constexpr int kSfChunkPitch = 528;  // 512 + 16: spreads the eight k-tiles over different banks

// MX = true is the MXFP4 variant (Section 3, Table 1): blocks of 32 with an E8M0 scale rounded up to a
// power of two.  A lane still encodes 16 values; the two lanes of a block share their amax by a shuffle
// and the even lane stores the scale.
template <typename T, bool SR, bool SWZ, bool MX = false>
__global__ void __launch_bounds__(kThreads, 3) quantize_row_kernel(const QuantParams p) {
  __shared__ __align__(16) uint8_t sf_s[SWZ ? 8 * kSfChunkPitch : 16];
  __shared__ float inv_table[MX ? 256 : 128];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t kb = (int64_t)blockIdx.x * 32 + lane;
  const int64_t row0 = (int64_t)blockIdx.y * kRowTileRows;
  const bool kb_ok = kb < p.nkb;
  const float g = p.gptr ? __ldg(p.gptr) : 1.0f;
  const float c = __fdiv_rn(__fdiv_rn(1.0f, 6.0f), g);
  const T* x = static_cast<const T*>(p.x);
  const bool aligned32 = ((reinterpret_cast<uintptr_t>(x) | (uintptr_t)(p.ld * (int64_t)sizeof(T))) & 31u) == 0;
  // scale position of this lane inside the CTA's 128-row x 32-group tile
  const int sf_chunk = MX ? (lane >> 3) : (lane >> 2);        // k-tile within the CTA tile
  const int sf_byte = MX ? ((lane >> 1) & 3) : (lane & 3);
  const bool sf_owner = MX ? ((lane & 1) == 0) : true;
  constexpr int kTilesPerCta = MX ? 4 : 8;

  if constexpr (MX) build_inv_table_mx(inv_table, g); else build_inv_table(inv_table, g);
  if constexpr (SWZ) {
    for (int i = threadIdx.x; i < 8 * kSfChunkPitch / 16; i += kThreads)
      reinterpret_cast<uint4*>(sf_s)[i] = make_uint4(0, 0, 0, 0);
  }
  __syncthreads();

  constexpr int U = (sizeof(T) == 2) ? 4 : 2;  // rows in flight per thread (32 packed registers)
  // A CTA whose 128 x 512 tile lies wholly inside the tensor (all of them but the last row and column of the grid)
  // runs the loop without any per-row or per-block predicate.
  const bool full_tile = row0 + kRowTileRows <= p.rows && ((int64_t)blockIdx.x + 1) * 32 <= p.nkb;
  auto sweep = [&](auto full_c) {
  constexpr bool FULL = decltype(full_c)::value;
#pragma unroll 1
  for (int it = 0; it < kRowTileRows / 8; it += U) {
    Block16<T> raw[U];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int64_t r = row0 + warp + 8 * (it + u);
      ok[u] = FULL || (kb_ok && r < p.rows);
      if (ok[u]) raw[u].load(x + r * p.ld + kb * 16, aligned32);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int rl = warp + 8 * (it + u);
      const int64_t r = row0 + rl;
      float v[16];
      float amax = 0.0f;
      if (ok[u]) amax = raw[u].unpack(v);
      if constexpr (MX) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));   // Kq % 32 == 0: both lanes valid or neither
      if (!ok[u]) continue;
      uint32_t lo, hi, sf;
      if constexpr (MX) {
        sf = e8m0_encode_up(__fmul_rn(amax, c));
        encode_codes<SR>(v, inv_table[sf], p.rng, (uint64_t)(r * p.nkb + kb), lo, hi);
      } else {
        encode_block<SR>(v, amax, c, inv_table, p.rng, (uint64_t)(r * p.nkb + kb), lo, hi, sf);
      }
      *reinterpret_cast<uint2*>(p.codes + (r * p.nkb + kb) * 8) = make_uint2(lo, hi);
      if (sf_owner) {
        if constexpr (SWZ) {
          sf_s[sf_chunk * kSfChunkPitch + (rl & 31) * 16 + (rl >> 5) * 4 + sf_byte] = (uint8_t)sf;
        } else {
          p.scales[r * p.nsb + (MX ? (kb >> 1) : kb)] = (uint8_t)sf;
        }
      }
    }
  }
  };
  if (full_tile) sweep(std::true_type{}); else sweep(std::false_type{});

  if constexpr (SWZ) {
    __syncthreads();
    const int q = threadIdx.x >> 5, i = threadIdx.x & 31;
    const int64_t kt = (int64_t)blockIdx.x * kTilesPerCta + q;
    if (q < kTilesPerCta && kt < p.k_tiles) {
      const uint4 val = *reinterpret_cast<const uint4*>(sf_s + q * kSfChunkPitch + i * 16);
      *reinterpret_cast<uint4*>(p.scales + ((int64_t)blockIdx.y * p.k_tiles + kt) * 512 + i * 16) = val;
    }
  }
}

// -------------------------------------------------------------------------------------------------
// Transposed quantizer: blocks run along the row axis of x[rows, cols]; the output is stored as
// [cols, rows/2] codes and [cols, rows/16] scales.  A CTA stages a (TILE_R rows x 64 cols) tile
// in shared memory with 16-byte async copies (zero-filled outside the tensor), every thread
// quantizes column pairs from it, and codes/scales leave through a second staging buffer so
// that global stores run along the output's contiguous axis.
// -------------------------------------------------------------------------------------------------
constexpr int kTCols = 64;

__device__ __forceinline__ void cp_async16_zfill(void* smem_dst, const void* gsrc, int src_bytes) {
  const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gsrc), "r"(src_bytes) : "memory");
}

template <typename T>
struct TTile {
  static constexpr int kRows = (sizeof(T) == 2) ? 256 : 128;          // 32 KB of input per tile
  static constexpr int kRowBlocks = kRows / 16;                        // 16 or 8
  static constexpr int kCodePitch = kRows / 2 + 8;                     // bytes per staged output row
  static constexpr int kChunksPerRow = kTCols * (int)sizeof(T) / 16;   // 8 or 16
};

template <typename T, bool SR, bool SWZ>
__global__ void __launch_bounds__(kThreads, 3) quantize_transposed_kernel(const QuantParams p) {
  using TT = TTile<T>;
  extern __shared__ __align__(16) uint8_t smem[];
  T* tile = reinterpret_cast<T*>(smem);                                        // [kRows][64]
  uint8_t* code_s = smem + TT::kRows * kTCols * sizeof(T);                     // [64][kCodePitch]
  uint8_t* sf_s = code_s + kTCols * TT::kCodePitch;                            // [64][kRowBlocks]

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t c0 = (int64_t)blockIdx.x * kTCols;
  const int64_t r0 = (int64_t)blockIdx.y * TT::kRows;
  const T* x = static_cast<const T*>(p.x);
  const float g = p.gptr ? __ldg(p.gptr) : 1.0f;
  const float c = __fdiv_rn(__fdiv_rn(1.0f, 6.0f), g);
  __shared__ float inv_table[128];
  build_inv_table(inv_table, g);                              // published by the barrier after the tile lands

  // ---- stage the input tile ----
  constexpr int kElemsPerChunk = 16 / (int)sizeof(T);
  constexpr int kChunks = TT::kRows * TT::kChunksPerRow;
#pragma unroll
  for (int i = 0; i < kChunks / kThreads; ++i) {
    const int id = threadIdx.x + i * kThreads;
    const int row = id / TT::kChunksPerRow, ch = id % TT::kChunksPerRow;
    const int64_t gr = r0 + row, gc = c0 + (int64_t)ch * kElemsPerChunk;
    int64_t valid = (gr < p.rows) ? (p.cols - gc) : 0;
    valid = valid < 0 ? 0 : (valid > kElemsPerChunk ? kElemsPerChunk : valid);
    const T* src = (valid > 0) ? (x + gr * p.ld + gc) : x;
    cp_async16_zfill(tile + row * kTCols + ch * kElemsPerChunk, src, (int)valid * (int)sizeof(T));
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- quantize: lane -> columns (2*lane, 2*lane+1), warp -> row blocks ----
  // Staging rows are ordered even columns first (column cl -> row (cl & 1) * 32 + cl / 2), so that a
  // warp's 8-byte code stores and its scale bytes fall into distinct banks.
#pragma unroll 1
  for (int rb = warp; rb < TT::kRowBlocks; rb += kThreads / 32) {
    float va[16], vb[16], amax_a, amax_b;
    if constexpr (sizeof(T) == 2) {
      uint32_t w[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) w[j] = *reinterpret_cast<const uint32_t*>(tile + (rb * 16 + j) * kTCols + 2 * lane);
      uint32_t m[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) m[j] = absmax_bf16x2(w[2 * j], w[2 * j + 1]);
#pragma unroll
      for (int j = 0; j < 4; ++j) m[j] = absmax_bf16x2(m[2 * j], m[2 * j + 1]);
      const uint32_t mm = absmax_bf16x2(absmax_bf16x2(m[0], m[1]), absmax_bf16x2(m[2], m[3])) & 0x7FFF7FFFu;
      amax_a = __uint_as_float(mm << 16);                     // low halves = column 2*lane
      amax_b = __uint_as_float(mm & 0xFFFF0000u);             // high halves = column 2*lane + 1
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        va[j] = __uint_as_float(w[j] << 16);
        vb[j] = __uint_as_float(w[j] & 0xFFFF0000u);
      }
    } else {
      amax_a = amax_b = 0.0f;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float2 f = *reinterpret_cast<const float2*>(tile + (rb * 16 + j) * kTCols + 2 * lane);
        va[j] = f.x;
        vb[j] = f.y;
        amax_a = fmaxf(amax_a, fabsf(f.x));
        amax_b = fmaxf(amax_b, fabsf(f.y));
      }
    }
    const int64_t kb = r0 / 16 + rb;
    const int64_t ca = c0 + 2 * lane;
    uint32_t lo, hi, sf;
    encode_block<SR>(va, amax_a, c, inv_table, p.rng, (uint64_t)(ca * p.nkb + kb), lo, hi, sf);
    *reinterpret_cast<uint2*>(code_s + lane * TT::kCodePitch + rb * 8) = make_uint2(lo, hi);
    sf_s[rb * kTCols + lane] = (uint8_t)sf;
    encode_block<SR>(vb, amax_b, c, inv_table, p.rng, (uint64_t)((ca + 1) * p.nkb + kb), lo, hi, sf);
    *reinterpret_cast<uint2*>(code_s + (32 + lane) * TT::kCodePitch + rb * 8) = make_uint2(lo, hi);
    sf_s[rb * kTCols + 32 + lane] = (uint8_t)sf;
  }
  __syncthreads();

  // ---- codes out: 8-byte units, contiguous along the quantized row ----
  const int64_t kb0 = r0 / 16;
#pragma unroll
  for (int i = 0; i < kTCols * TT::kRowBlocks / kThreads; ++i) {
    const int id = threadIdx.x + i * kThreads;
    const int cl = id / TT::kRowBlocks, u = id % TT::kRowBlocks;
    if (c0 + cl < p.cols && kb0 + u < p.nkb) {
      const int srow = (cl & 1) * 32 + (cl >> 1);
      const uint2 val = *reinterpret_cast<const uint2*>(code_s + srow * TT::kCodePitch + u * 8);
      *reinterpret_cast<uint2*>(p.codes + ((c0 + cl) * p.nkb + kb0 + u) * 8) = val;
    }
  }
  // ---- scales out ----
  if constexpr (SWZ) {
    constexpr int kKt = TT::kRowBlocks / 4;  // k-tiles per CTA tile
    const bool fill_upper = ((c0 & 127) == 0) && (c0 + kTCols >= p.cols);  // nobody else owns rows 64..127
    for (int id = threadIdx.x; id < kTCols * kKt; id += kThreads) {
      const int cl = id / kKt, t = id % kKt;
      const int64_t kt = kb0 / 4 + t;
      if (kt >= p.k_tiles) continue;
      const int srow = (cl & 1) * 32 + (cl >> 1);
      const uint8_t* s4 = sf_s + (t * 4) * kTCols + srow;
      const uint32_t val = (uint32_t)s4[0] | ((uint32_t)s4[kTCols] << 8) | ((uint32_t)s4[2 * kTCols] << 16) |
                           ((uint32_t)s4[3 * kTCols] << 24);
      *reinterpret_cast<uint32_t*>(p.scales + sf_swizzled_offset(c0 + cl, kt * 4, p.k_tiles)) = val;
      if (fill_upper)
        *reinterpret_cast<uint32_t*>(p.scales + sf_swizzled_offset(c0 + cl + 64, kt * 4, p.k_tiles)) = 0u;
    }
  } else {
    for (int id = threadIdx.x; id < kTCols * TT::kRowBlocks; id += kThreads) {
      const int cl = id / TT::kRowBlocks, u = id % TT::kRowBlocks;
      const int srow = (cl & 1) * 32 + (cl >> 1);
      if (c0 + cl < p.cols && kb0 + u < p.nkb) p.scales[(c0 + cl) * p.nkb + kb0 + u] = sf_s[u * kTCols + srow];
    }
  }
}

// -------------------------------------------------------------------------------------------------
// Per-tensor amax -> g = amax / (6*448)
//
// The running maximum is kept as the bit pattern of |x|: non-negative IEEE patterns order as unsigned
// integers, +Inf sits above every finite value and every NaN pattern above +Inf.  A tensor that
// holds a NaN therefore gets g = NaN, one that holds an infinity (and no NaN) g = +Inf, and every
// product computed with such a scale comes out as NaN (NaN * acc, or Inf * 0): a diverged step is
// visible in Y, dX and dW instead of being quantized into finite codes.
// -------------------------------------------------------------------------------------------------
// max |.| of two packed bf16 pairs, per half, NaN if either is (the sign bits of the result are meaningless)
__device__ __forceinline__ uint32_t absmax_nan_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

// Running maximum of one thread over words of source data (bf16 pairs or fp32 values).
template <typename T>
struct AmaxBits {
  uint32_t m = 0u;
  __device__ __forceinline__ void add8(const uint32_t (&w)[8]) {
    if constexpr (sizeof(T) == 2) {
      m = absmax_nan_bf16x2(absmax_nan_bf16x2(absmax_nan_bf16x2(absmax_nan_bf16x2(w[0], w[1]), absmax_nan_bf16x2(w[2], w[3])),
                                              absmax_nan_bf16x2(absmax_nan_bf16x2(w[4], w[5]), absmax_nan_bf16x2(w[6], w[7]))),
                            m);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) m = max(m, w[k] & 0x7FFFFFFFu);
    }
  }
  __device__ __forceinline__ void add4(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    if constexpr (sizeof(T) == 2) {
      m = absmax_nan_bf16x2(absmax_nan_bf16x2(absmax_nan_bf16x2(a, b), absmax_nan_bf16x2(c, d)), m);
    } else {
      m = max(max(m, a & 0x7FFFFFFFu), max(max(b & 0x7FFFFFFFu, c & 0x7FFFFFFFu), d & 0x7FFFFFFFu));
    }
  }
  // fp32 bit pattern of the maximum over the warp
  __device__ __forceinline__ uint32_t warp_bits() const {
    uint32_t bits = m;
    if constexpr (sizeof(T) == 2) {
      const uint32_t h = m & 0x7FFF7FFFu;                      // bf16 patterns widen to fp32 by a shift
      bits = max(h >> 16, h & 0xFFFFu) << 16;
    }
    return __reduce_max_sync(0xFFFFFFFFu, bits);
  }
};

// Strided tensors: 16-byte loads, grid-stride.
template <typename T>
__global__ void __launch_bounds__(kThreads) amax_kernel(const T* x, int64_t rows, int64_t cols, int64_t ld,
                                                        unsigned int* out_bits) {
  constexpr int kVec = 16 / (int)sizeof(T);
  const int64_t vec_per_row = cols / kVec;
  const int64_t total = rows * vec_per_row;
  AmaxBits<T> acc;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
    const int64_t r = i / vec_per_row, vcol = i % vec_per_row;
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(x + r * ld + vcol * kVec));
    acc.add4(q.x, q.y, q.z, q.w);
  }
  const uint32_t bits = acc.warp_bits();
  if ((threadIdx.x & 31) == 0 && bits != 0u) atomicMax(out_bits, bits);
}

// Dense tensors (ld == cols, 32-byte aligned): a flat sweep with four 256-bit loads in flight per thread.
// TICKET = false: the maximum is left in out[0] for amax_finalize_kernel.
// TICKET = true: one launch does it all.  out = {running max bits, ticket}, both zero on entry; the block that
// takes the last ticket turns the maximum into g = amax / 2688 (1 for an all-zero tensor), stores it in *g_out
// and leaves the two words zero again.
template <typename T, bool TICKET>
__global__ void __launch_bounds__(kThreads) amax_flat_kernel(const uint32_t* x, int64_t n_vec32, unsigned int* out, float* g_out) {
  __shared__ uint32_t warp_max[kThreads / 32];
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  AmaxBits<T> acc;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n_vec32; i += 4 * stride) {
    uint32_t w[4][8];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t j = i + u * stride;
      if (j < n_vec32) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(w[u][0]), "=r"(w[u][1]), "=r"(w[u][2]), "=r"(w[u][3]), "=r"(w[u][4]), "=r"(w[u][5]),
                       "=r"(w[u][6]), "=r"(w[u][7])
                     : "l"(x + j * 8));
      } else {
#pragma unroll
        for (int k = 0; k < 8; ++k) w[u][k] = 0u;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) acc.add8(w[u]);
  }
  const uint32_t bits = acc.warp_bits();
  if constexpr (!TICKET) {
    if ((threadIdx.x & 31) == 0 && bits != 0u) atomicMax(out, bits);
  } else {
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = bits;
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t block_bits = bits;
#pragma unroll
      for (int w8 = 1; w8 < kThreads / 32; ++w8) block_bits = max(block_bits, warp_max[w8]);
      if (block_bits != 0u) atomicMax(&out[0], block_bits);
      __threadfence();
      if (atomicAdd(&out[1], 1u) == gridDim.x - 1) {                      // every other block's maximum is in
        __threadfence();
        const float total = __uint_as_float(atomicExch(&out[0], 0u));
        *g_out = (total == 0.0f) ? 1.0f : __fdiv_rn(total, 2688.0f);
        out[1] = 0u;
      }
    }
  }
}

__global__ void amax_finalize_kernel(float* out) {
  const float amax = *out;
  *out = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 2688.0f);
}

template <typename T, bool SR, bool SWZ>
cudaError_t launch_row(const QuantParams& p, cudaStream_t s) {
  dim3 grid((unsigned)ceil_div(p.nkb, 32), (unsigned)ceil_div(p.rows, kRowTileRows));
  quantize_row_kernel<T, SR, SWZ><<<grid, kThreads, 0, s>>>(p);
  return cudaGetLastError();
}

template <typename T, bool SR, bool SWZ>
cudaError_t launch_transposed(const QuantParams& p, cudaStream_t s) {
  using TT = TTile<T>;
  const size_t smem = TT::kRows * kTCols * sizeof(T) + kTCols * TT::kCodePitch + kTCols * TT::kRowBlocks;
  static DeviceFlags smem_set;   // per instantiation, per device
  if (cudaError_t e = set_max_dynamic_smem(smem_set, quantize_transposed_kernel<T, SR, SWZ>, (int)smem)) return e;
  dim3 grid((unsigned)ceil_div(p.cols, kTCols), (unsigned)ceil_div(p.rows, TT::kRows));
  quantize_transposed_kernel<T, SR, SWZ><<<grid, kThreads, smem, s>>>(p);
  return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const QuantParams& p, bool transposed, bool sr, bool swz, cudaStream_t s) {
  if (!transposed) {
    if (sr) return swz ? launch_row<T, true, true>(p, s) : launch_row<T, true, false>(p, s);
    return swz ? launch_row<T, false, true>(p, s) : launch_row<T, false, false>(p, s);
  }
  if (sr) return swz ? launch_transposed<T, true, true>(p, s) : launch_transposed<T, true, false>(p, s);
  return swz ? launch_transposed<T, false, true>(p, s) : launch_transposed<T, false, false>(p, s);
}

}  // namespace

}  // namespace nvfp4

using namespace nvfp4;

extern "C" size_t nvfp4_sf_bytes(int64_t Rq, int64_t Kq, int sf_layout) {
  if (Rq <= 0 || Kq <= 0 || (Kq % 16) != 0) return 0;
  if (sf_layout == NVFP4_SF_LINEAR) return (size_t)(Rq * (Kq / 16));
  if (sf_layout == NVFP4_SF_SWIZZLED_128x4) return (size_t)(ceil_div(Rq, 128) * ceil_div(Kq, 64) * 512);
  return 0;
}

extern "C" int nvfp4_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                              int transposed, const float* global_scale, const nvfp4_rounding* rounding,
                              uint8_t* codes, uint8_t* scales, int sf_layout, void* cuda_stream) {
  if (!x || !rounding || !codes || !scales) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (transposed != 0 && transposed != 1) return NVFP4_ERR_ENUM;
  if (rounding->mode != NVFP4_RTN && rounding->mode != NVFP4_SR) return NVFP4_ERR_ENUM;
  if (rounding->reserved != 0) return NVFP4_ERR_ENUM;
  if (sf_layout != NVFP4_SF_LINEAR && sf_layout != NVFP4_SF_SWIZZLED_128x4) return NVFP4_ERR_ENUM;
  if (rows <= 0 || cols <= 0 || ld < cols) return NVFP4_ERR_SHAPE;
  const int64_t Kq = transposed ? rows : cols;
  if (Kq % 16 != 0 || cols % 8 != 0) return NVFP4_ERR_SHAPE;
  if (rows >= (int64_t)1 << 31 || cols >= (int64_t)1 << 31) return NVFP4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(scales) || (ld % 8) != 0) return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;

  QuantParams p;
  p.x = x; p.rows = rows; p.cols = cols; p.ld = ld; p.gptr = global_scale;
  philox_stream_init(&p.rng, rounding->seed, rounding->offset);
  p.codes = codes; p.scales = scales;
  p.nkb = Kq / 16; p.nsb = p.nkb; p.k_tiles = ceil_div(p.nsb, 4);
  if (ceil_div(rows, 128) > 65535) return NVFP4_ERR_SHAPE;  // grid.y limit
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (transposed && tile_quantizer_eligible(dtype, rows, cols, false))
    return tile_quantize(x, rows, cols, ld, global_scale, false, rounding, codes, scales, nullptr, nullptr, nullptr,
                         sf_layout, s);
  const bool sr = rounding->mode == NVFP4_SR, swz = sf_layout == NVFP4_SF_SWIZZLED_128x4;
  cudaError_t e = (dtype == NVFP4_BF16) ? dispatch<__nv_bfloat16>(p, transposed != 0, sr, swz, s)
                                        : dispatch<float>(p, transposed != 0, sr, swz, s);
  return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

namespace nvfp4 {
namespace {
template <typename T>
cudaError_t dispatch_row_mx(const QuantParams& p, bool sr, bool swz, cudaStream_t s) {
  dim3 grid((unsigned)ceil_div(p.nkb, 32), (unsigned)ceil_div(p.rows, kRowTileRows));
  if (sr) {
    if (swz) quantize_row_kernel<T, true, true, true><<<grid, kThreads, 0, s>>>(p);
    else quantize_row_kernel<T, true, false, true><<<grid, kThreads, 0, s>>>(p);
  } else {
    if (swz) quantize_row_kernel<T, false, true, true><<<grid, kThreads, 0, s>>>(p);
    else quantize_row_kernel<T, false, false, true><<<grid, kThreads, 0, s>>>(p);
  }
  return cudaGetLastError();
}
}  // namespace
}  // namespace nvfp4

extern "C" size_t nvfp4_sf_bytes_mx(int64_t Rq, int64_t Kq, int sf_layout) {
  if (Rq <= 0 || Kq <= 0 || (Kq % 32) != 0) return 0;
  if (sf_layout == NVFP4_SF_LINEAR) return (size_t)(Rq * (Kq / 32));
  if (sf_layout == NVFP4_SF_SWIZZLED_128x4) return (size_t)(ceil_div(Rq, 128) * ceil_div(Kq, 128) * 512);
  return 0;
}

extern "C" int nvfp4_quantize_mx(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int transposed,
                                 const float* global_scale, const nvfp4_rounding* rounding,
                                 uint8_t* codes, uint8_t* scales, int sf_layout,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!x || !rounding || !codes || !scales) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (transposed != 0 && transposed != 1) return NVFP4_ERR_ENUM;
  if (transposed && dtype != NVFP4_BF16) return NVFP4_ERR_ENUM;        // the transposed path goes through the bf16 transpose
  if ((rounding->mode != NVFP4_RTN && rounding->mode != NVFP4_SR) || rounding->reserved != 0) return NVFP4_ERR_ENUM;
  if (sf_layout != NVFP4_SF_LINEAR && sf_layout != NVFP4_SF_SWIZZLED_128x4) return NVFP4_ERR_ENUM;
  if (rows <= 0 || cols <= 0 || ld < cols || cols % 8 != 0) return NVFP4_ERR_SHAPE;
  const int64_t Rq = transposed ? cols : rows, Kq = transposed ? rows : cols;
  if (Kq % 32 != 0 || rows >= (int64_t)1 << 31 || cols >= (int64_t)1 << 31) return NVFP4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(scales) || (ld % 8) != 0) return NVFP4_ERR_ALIGN;
  if (ceil_div(Rq, 128) > 65535) return NVFP4_ERR_SHAPE;
  // bf16 tensors whose row count is a multiple of 32 (always true here: Kq = rows) go through the tile kernel, which
  // quantizes along the rows straight from the source; the transpose pass remains for what that kernel does not take
  const bool tile_path = transposed && rows % 32 == 0 && tile_quantizer_eligible(dtype, rows, cols, false);
  if (transposed && !tile_path &&
      (!workspace || workspace_bytes < (size_t)rows * cols * 2 || (reinterpret_cast<uintptr_t>(workspace) & 15u)))
    return NVFP4_ERR_WORKSPACE;
  if (int st = check_arch()) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (tile_path)
    return tile_quantize(x, rows, cols, ld, global_scale, false, rounding, codes, scales, nullptr, nullptr, nullptr, sf_layout, s,
                         /*mx_t=*/true);
  const void* src = x;
  int64_t src_ld = ld;
  if (transposed) {
    // Q(x^T) is by definition the row quantization of the materialised transpose
    if (int st = nvfp4_transpose_bf16(x, rows, cols, ld, workspace, cuda_stream)) return st;
    src = workspace;
    src_ld = rows;
  }
  QuantParams p;
  p.x = src; p.rows = Rq; p.cols = Kq; p.ld = src_ld; p.gptr = global_scale;
  philox_stream_init(&p.rng, rounding->seed, rounding->offset);
  p.codes = codes; p.scales = scales;
  p.nkb = Kq / 16; p.nsb = Kq / 32; p.k_tiles = ceil_div(p.nsb, 4);
  const bool sr = rounding->mode == NVFP4_SR, swz = sf_layout == NVFP4_SF_SWIZZLED_128x4;
  cudaError_t e = (dtype == NVFP4_BF16) ? dispatch_row_mx<__nv_bfloat16>(p, sr, swz, s) : dispatch_row_mx<float>(p, sr, swz, s);
  return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

extern "C" int nvfp4_quantize_dual(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                                   const float* global_scale,
                                   const nvfp4_rounding* rounding_row, uint8_t* codes_row, uint8_t* scales_row,
                                   const nvfp4_rounding* rounding_t, uint8_t* codes_t, uint8_t* scales_t,
                                   int sf_layout, void* cuda_stream) {
  if (!x || !rounding_row || !rounding_t || !codes_row || !scales_row || !codes_t || !scales_t) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  for (const nvfp4_rounding* r : {rounding_row, rounding_t})
    if ((r->mode != NVFP4_RTN && r->mode != NVFP4_SR) || r->reserved != 0) return NVFP4_ERR_ENUM;
  if (sf_layout != NVFP4_SF_LINEAR && sf_layout != NVFP4_SF_SWIZZLED_128x4) return NVFP4_ERR_ENUM;
  if (rows <= 0 || cols <= 0 || ld < cols || rows % 16 != 0 || cols % 16 != 0) return NVFP4_ERR_SHAPE;
  if (rows >= (int64_t)1 << 31 || cols >= (int64_t)1 << 31) return NVFP4_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(codes_row) || !aligned16(scales_row) || !aligned16(codes_t) || !aligned16(scales_t) ||
      (ld % 8) != 0)
    return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  if (tile_quantizer_eligible(dtype, rows, cols, true))
    return tile_quantize(x, rows, cols, ld, global_scale, true, rounding_t, codes_t, scales_t, rounding_row, codes_row,
                         scales_row, sf_layout, static_cast<cudaStream_t>(cuda_stream));
  // shapes or types the tile kernel does not take: the two single-output kernels, two reads
  if (int st = nvfp4_quantize(x, dtype, rows, cols, ld, 0, global_scale, rounding_row, codes_row, scales_row, sf_layout,
                              cuda_stream))
    return st;
  return nvfp4_quantize(x, dtype, rows, cols, ld, 1, global_scale, rounding_t, codes_t, scales_t, sf_layout, cuda_stream);
}

namespace nvfp4 {
// Per-tensor scale in one launch where the tensor allows it (dense, 32-byte aligned); `scratch_zeroed` is two
// zeroed 32-bit words in device memory that the kernel leaves zeroed.  Otherwise the three-step public path.
int tensor_amax_scale_ws(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* g_out,
                         unsigned int* scratch_zeroed, void* cuda_stream) {
  const int64_t total_bytes = rows * cols * (dtype == NVFP4_BF16 ? 2 : 4);
  if (!x || !g_out || !scratch_zeroed || rows <= 0 || cols <= 0 || ld != cols || (reinterpret_cast<uintptr_t>(x) & 31u) != 0 ||
      total_bytes % 32 != 0)
    return nvfp4_tensor_amax_scale(x, dtype, rows, cols, ld, g_out, cuda_stream);
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (int st = check_arch()) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int64_t n32 = total_bytes / 32;
  int64_t fb = ceil_div(n32, (int64_t)kThreads * 4);
  if (fb > sm_count() * 8) fb = sm_count() * 8;
  if (dtype == NVFP4_BF16)
    amax_flat_kernel<__nv_bfloat16, true><<<(unsigned)fb, kThreads, 0, s>>>(static_cast<const uint32_t*>(x), n32, scratch_zeroed, g_out);
  else
    amax_flat_kernel<float, true><<<(unsigned)fb, kThreads, 0, s>>>(static_cast<const uint32_t*>(x), n32, scratch_zeroed, g_out);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}
}  // namespace nvfp4

extern "C" int nvfp4_tensor_amax_scale(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                                       float* global_scale_out, void* cuda_stream) {
  if (!x || !global_scale_out) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (rows <= 0 || cols <= 0 || ld < cols || cols % 8 != 0) return NVFP4_ERR_SHAPE;
  if (!aligned16(x) || (ld % 8) != 0 || (reinterpret_cast<uintptr_t>(global_scale_out) & 3u)) return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(global_scale_out, 0, sizeof(float), s) != cudaSuccess) return NVFP4_ERR_CUDA;
  const int64_t vecs = rows * (cols / (dtype == NVFP4_BF16 ? 8 : 4));
  int64_t blocks = ceil_div(vecs, (int64_t)kThreads * 4);
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  if (blocks < 1) blocks = 1;
  unsigned int* bits = reinterpret_cast<unsigned int*>(global_scale_out);
  const int64_t total_bytes = rows * cols * (dtype == NVFP4_BF16 ? 2 : 4);
  if (ld == cols && (reinterpret_cast<uintptr_t>(x) & 31u) == 0 && total_bytes % 32 == 0) {
    const int64_t n32 = total_bytes / 32;
    int64_t fb = ceil_div(n32, (int64_t)kThreads * 4);
    if (fb > sm_count() * 8) fb = sm_count() * 8;
    if (dtype == NVFP4_BF16)
      amax_flat_kernel<__nv_bfloat16, false><<<(unsigned)fb, kThreads, 0, s>>>(static_cast<const uint32_t*>(x), n32, bits, nullptr);
    else
      amax_flat_kernel<float, false><<<(unsigned)fb, kThreads, 0, s>>>(static_cast<const uint32_t*>(x), n32, bits, nullptr);
  } else if (dtype == NVFP4_BF16)
    amax_kernel<__nv_bfloat16><<<(unsigned)blocks, kThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(x), rows, cols, ld, bits);
  else
    amax_kernel<float><<<(unsigned)blocks, kThreads, 0, s>>>(static_cast<const float*>(x), rows, cols, ld, bits);
  if (cudaGetLastError() != cudaSuccess) return NVFP4_ERR_CUDA;
  amax_finalize_kernel<<<1, 1, 0, s>>>(global_scale_out);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}
