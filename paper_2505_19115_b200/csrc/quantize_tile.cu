// Tile quantizer for bf16 tensors: one read of x[rows, cols] produces the transposed NVFP4
// quantization (blocks of 16 along the row axis, output stored [cols, rows/2]) and, optionally, the
// row quantization (blocks along the column axis) of the same tile.  This is the producer fusion
// for the operands that Eq. 4-6 need in both orientations: dY as Q(dY) for Eq. 5 and Q(dY^T) for
// Eq. 6, X as Q(X) for Eq. 4 and Q(X^T) for Eq. 6, W as Q(W) for Eq. 4 and Q(W^T) for Eq. 5.
//
// A CTA takes a tile of 256 rows x 64 columns (32 KB).  One thread fetches it with a tiled bulk
// copy (128-byte swizzle, zero fill outside the tensor); all threads quantize from shared memory;
// the packed codes are staged in shared memory and leave as tiled bulk stores (which clip at the
// tensor edge), the scales as plain stores.
#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "quantize_core.cuh"
#include "tensor_map.cuh"

namespace nvfp4 {
namespace {

constexpr int kTileRows = 256;
constexpr int kTileCols = 64;
constexpr int kTileBytes = kTileRows * kTileCols * 2;                 // 32 KB, rows of 128 bytes
constexpr int kCodesTBytes = kTileCols * (kTileRows / 2);             // 64 output rows x 128 bytes
constexpr int kCodesRBytes = kTileRows * (kTileCols / 2);             // 256 output rows x 32 bytes
constexpr int kSfTBytes = kTileCols * (kTileRows / 16);               // [16 row blocks][64 columns]
constexpr int kSfRBytes = 2 * 512;                                    // two scale tiles (128 rows x 4 blocks)
constexpr int kTileSmem = kTileBytes + kCodesTBytes + kCodesRBytes + kSfTBytes + kSfRBytes + 1024 /*align*/;
constexpr unsigned long long kTileWaitLimitNs = 2000000000ull;

struct TileParams {
  const float* gptr;
  int64_t rows, cols;
  // transposed output (always): quantized shape (cols, rows)
  PhiloxStream t_rng;
  uint8_t* t_scales;
  int64_t t_nkb, t_k_tiles;   // groups of 16 per quantized row (the unit of the random draws); scale tiles per quantized row
  int64_t t_nsb;              // scale blocks per quantized row: rows / 16 (NVFP4) or rows / 32 (MXFP4)
  // row output (DUAL only): quantized shape (rows, cols)
  PhiloxStream r_rng;
  uint8_t* r_scales;
  int64_t r_nkb, r_k_tiles;
};

__device__ unsigned int g_tile_error_word = 0;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of (row, byte) inside a tile of 128-byte rows stored with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz128(uint32_t row, uint32_t byte) {
  return row * 128u + ((((byte >> 4) ^ (row & 7u)) << 4) | (byte & 15u));
}

// MX_T: the transposed output is MXFP4 (Section 3, Table 1): blocks of 32 rows with an E8M0 scale rounded up to a
// power of two; a warp then takes 32 rows at a time, and the two groups of 16 inside a block keep their own
// random draws (group index as for NVFP4).
// Shared-memory accesses with the address split into a register part and a compile-time byte offset, so that
// the unrolled loops below spend no instructions on addresses.  The loads are plain (not volatile) statements, so
// that the compiler may schedule them ahead of the arithmetic of the previous block; the tile they read is written
// once, by the bulk copy, and their base address is taken only after the wait for that copy (tile_base_after_wait).
template <int IMM>
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm("ld.shared.b32 %0, [%1 + %2];" : "=r"(v) : "r"(addr), "n"(IMM));
  return v;
}
template <int IMM>
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4 + %5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr), "n"(IMM));
  return v;
}
// The tile's shared-memory address as a value the compiler must consider produced here: every load whose address
// derives from it stays behind the point of the call.
__device__ __forceinline__ uint32_t tile_base_after_wait(const void* tile) {
  uint32_t a = smem_addr(tile);
  asm volatile("" : "+r"(a) :: "memory");
  return a;
}
template <int IMM>
__device__ __forceinline__ void sts64(uint32_t addr, uint32_t lo, uint32_t hi) {
  asm volatile("st.shared.v2.b32 [%0 + %3], {%1, %2};" ::"r"(addr), "r"(lo), "r"(hi), "n"(IMM) : "memory");
}

template <bool SR_T, bool DUAL, bool SR_R, bool SWZ, bool MX_T = false>
__global__ void __launch_bounds__(kThreads, 4)
quantize_tile_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_ct,
                     const __grid_constant__ CUtensorMap map_cr, const TileParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
  uint8_t* tile = smem;                                   // [256][128 B], swizzled
  uint8_t* codes_t = tile + kTileBytes;                   // [64][128 B], swizzled
  uint8_t* codes_r = codes_t + kCodesTBytes;              // [256][32 B]
  uint8_t* sf_t = codes_r + kCodesRBytes;                 // [16][64]
  uint8_t* sf_r = sf_t + kSfTBytes;                       // [2][512]
  static_assert(!(MX_T && DUAL), "the MXFP4 variant writes the transposed output only");
  __shared__ __align__(8) uint64_t bar;
  __shared__ float inv_table[MX_T ? 256 : 128];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t c0 = (int64_t)blockIdx.x * kTileCols;
  const int64_t r0 = (int64_t)blockIdx.y * kTileRows;
  const float g = p.gptr ? __ldg(p.gptr) : 1.0f;
  const float c = __fdiv_rn(__fdiv_rn(1.0f, 6.0f), g);

  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bar)));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&bar)), "r"(kTileBytes) : "memory");
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_addr(tile)), "l"(&map_x), "r"(smem_addr(&bar)), "r"((int)c0), "r"((int)r0) : "memory");
  }
  if constexpr (MX_T) build_inv_table_mx(inv_table, g); else build_inv_table(inv_table, g);
  __syncthreads();                                        // barrier initialised, table published
  {
    // bounded wait for the tile; on a timeout every thread leaves without storing anything
    const uint32_t b = smem_addr(&bar);
    uint32_t done = 0;
    unsigned long long t0 = 0;
    for (uint32_t spin = 0; !done; ++spin) {
      asm volatile("{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                   : "=r"(done) : "r"(b) : "memory");
      if (!done && (spin & 255u) == 255u) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (t0 == 0) t0 = now;
        if (now - t0 > kTileWaitLimitNs) {
          if (threadIdx.x == 0) atomicOr(&g_tile_error_word, 0x200u);
          return;
        }
      }
    }
  }

  // ---- transposed output: lane -> columns (2*lane, 2*lane+1), warp -> row blocks ----
  // Codes are staged as [column][128 bytes] with the 128-byte swizzle the tiled store expects.
  if constexpr (MX_T) {
    const int rb = warp;                                      // 8 warps, 8 blocks of 32 rows
    uint32_t w[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) w[j] = *reinterpret_cast<const uint32_t*>(tile + swz128(rb * 32 + j, 4 * lane));
    uint32_t m[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) m[j] = absmax_bf16x2(w[2 * j], w[2 * j + 1]);
#pragma unroll
    for (int j = 0; j < 8; ++j) m[j] = absmax_bf16x2(m[2 * j], m[2 * j + 1]);
#pragma unroll
    for (int j = 0; j < 4; ++j) m[j] = absmax_bf16x2(m[2 * j], m[2 * j + 1]);
    const uint32_t mm = absmax_bf16x2(absmax_bf16x2(m[0], m[1]), absmax_bf16x2(m[2], m[3])) & 0x7FFF7FFFu;
    const uint32_t sfa = e8m0_encode_up(__fmul_rn(__uint_as_float(mm << 16), c));
    const uint32_t sfb = e8m0_encode_up(__fmul_rn(__uint_as_float(mm & 0xFFFF0000u), c));
    const float inv_a = inv_table[sfa], inv_b = inv_table[sfb];
    const int64_t ca = c0 + 2 * lane;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float va[16], vb[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        va[j] = __uint_as_float(w[16 * h + j] << 16);
        vb[j] = __uint_as_float(w[16 * h + j] & 0xFFFF0000u);
      }
      const int64_t kb = r0 / 16 + rb * 2 + h;                // group of 16 along the quantized row
      uint32_t lo, hi;
      encode_codes<SR_T>(va, inv_a, p.t_rng, (uint64_t)(ca * p.t_nkb + kb), lo, hi);
      *reinterpret_cast<uint2*>(codes_t + swz128(2 * lane, (rb * 2 + h) * 8)) = make_uint2(lo, hi);
      encode_codes<SR_T>(vb, inv_b, p.t_rng, (uint64_t)((ca + 1) * p.t_nkb + kb), lo, hi);
      *reinterpret_cast<uint2*>(codes_t + swz128(2 * lane + 1, (rb * 2 + h) * 8)) = make_uint2(lo, hi);
    }
    sf_t[rb * kTileCols + 2 * lane] = (uint8_t)sfa;
    sf_t[rb * kTileCols + 2 * lane + 1] = (uint8_t)sfb;
  } else {
  // Two forms of the same arithmetic.  With stochastic rounding in both outputs the kernel sits at its register limit
  // (64, for four CTAs per SM) and runs fastest with addresses precomputed and the two columns' Philox calls
  // interleaved; every other instantiation has registers to spare and runs fastest with the plain loop, which lets
  // the compiler overlap the two row blocks (same-process A/B: 4.43 against 4.17 TB/s for SR/SR, 5.50 against
  // 5.08-5.16 for the single SR output, 5.31 against 4.93-5.12 for RtN rows + SR transposed).
  if constexpr (DUAL && SR_T && SR_R) {
  {
    // Row rb*16 + j of the tile, bytes 4*lane..4*lane+3: (row & 7) = j & 7, so the swizzled position inside a
    // row depends on j & 7 only; eight base addresses serve all loads, the rest is a compile-time offset.
    const uint32_t tile_s = tile_base_after_wait(tile) + (uint32_t)warp * 2048u;
    uint32_t rowbase[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) rowbase[q] = tile_s + q * 128 + ((((uint32_t)(lane >> 2) ^ q) << 4) | ((uint32_t)(lane & 3) << 2));
    // staging position of this lane's two output rows (columns 2*lane, 2*lane+1) for row block `warp`; the second
    // row block of this warp (warp + 8) sits four 16-byte chunks further, which the swizzle turns into an XOR with 64
    const uint32_t ct_s = smem_addr(codes_t);
    const uint32_t ra = 2 * lane, rbw = 2 * lane + 1;
    const uint32_t st_a = ct_s + ra * 128 + ((((uint32_t)(warp >> 1) ^ (ra & 7)) << 4) | ((uint32_t)(warp & 1) << 3));
    const uint32_t st_b = ct_s + rbw * 128 + ((((uint32_t)(warp >> 1) ^ (rbw & 7)) << 4) | ((uint32_t)(warp & 1) << 3));
    const uint64_t blk_a0 = (uint64_t)((c0 + 2 * lane) * p.t_nkb + r0 / 16 + warp);
    uint8_t* sf_lane = sf_t + warp * kTileCols + 2 * lane;
#pragma unroll
    for (int it = 0; it < 2; ++it) {                          // row blocks warp and warp + 8
      uint32_t w[16];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        w[j] = it ? lds32<16384 + 0>(rowbase[j]) : lds32<0>(rowbase[j]);
        w[j + 8] = it ? lds32<16384 + 1024>(rowbase[j]) : lds32<1024>(rowbase[j]);
      }
      uint32_t m[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) m[j] = absmax_bf16x2(w[2 * j], w[2 * j + 1]);
#pragma unroll
      for (int j = 0; j < 4; ++j) m[j] = absmax_bf16x2(m[2 * j], m[2 * j + 1]);
      const uint32_t mm = absmax_bf16x2(absmax_bf16x2(m[0], m[1]), absmax_bf16x2(m[2], m[3])) & 0x7FFF7FFFu;
      const uint64_t blk_a = blk_a0 + 8u * it, blk_b = blk_a + (uint64_t)p.t_nkb;
      const uint32_t sfa = e4m3_encode(__fmul_rn(__uint_as_float(mm << 16), c));
      const uint32_t sfb = e4m3_encode(__fmul_rn(__uint_as_float(mm & 0xFFFF0000u), c));
      const float inv_a = inv_table[sfa], inv_b = inv_table[sfb];
      uint4 ra = make_uint4(0, 0, 0, 0), rb = ra;
      if constexpr (SR_T) philox4x32_10_x2(p.t_rng, blk_a, blk_b, ra, rb);
      uint32_t lo, hi;
      {
        float y[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) y[j] = __fmul_rn(__uint_as_float(w[j] << 16), inv_a);          // column 2*lane
        if constexpr (SR_T) { lo = e2m1x8_rs(y, 0, ra.x, ra.y); hi = e2m1x8_rs(y, 8, ra.z, ra.w); }
        else { lo = e2m1x8_rn(y, 0); hi = e2m1x8_rn(y, 8); }
        if (it) sts64<0>(st_a ^ 64u, lo, hi); else sts64<0>(st_a, lo, hi);
      }
      {
        float y[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) y[j] = __fmul_rn(__uint_as_float(w[j] & 0xFFFF0000u), inv_b);  // column 2*lane + 1
        if constexpr (SR_T) { lo = e2m1x8_rs(y, 0, rb.x, rb.y); hi = e2m1x8_rs(y, 8, rb.z, rb.w); }
        else { lo = e2m1x8_rn(y, 0); hi = e2m1x8_rn(y, 8); }
        if (it) sts64<0>(st_b ^ 64u, lo, hi); else sts64<0>(st_b, lo, hi);
      }
      *reinterpret_cast<uint16_t*>(sf_lane + it * 8 * kTileCols) = (uint16_t)(sfa | (sfb << 8));
    }
  }
  } else {
#pragma unroll
  for (int rb = warp; rb < kTileRows / 16; rb += kThreads / 32) {
    uint32_t w[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) w[j] = *reinterpret_cast<const uint32_t*>(tile + swz128(rb * 16 + j, 4 * lane));
    uint32_t m[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) m[j] = absmax_bf16x2(w[2 * j], w[2 * j + 1]);
#pragma unroll
    for (int j = 0; j < 4; ++j) m[j] = absmax_bf16x2(m[2 * j], m[2 * j + 1]);
    const uint32_t mm = absmax_bf16x2(absmax_bf16x2(m[0], m[1]), absmax_bf16x2(m[2], m[3])) & 0x7FFF7FFFu;
    float va[16], vb[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      va[j] = __uint_as_float(w[j] << 16);                    // column 2*lane
      vb[j] = __uint_as_float(w[j] & 0xFFFF0000u);            // column 2*lane + 1
    }
    const int64_t kb = r0 / 16 + rb;
    const int64_t ca = c0 + 2 * lane;
    uint32_t lo, hi, sf;
    encode_block<SR_T>(va, __uint_as_float(mm << 16), c, inv_table, p.t_rng, (uint64_t)(ca * p.t_nkb + kb), lo, hi, sf);
    *reinterpret_cast<uint2*>(codes_t + swz128(2 * lane, rb * 8)) = make_uint2(lo, hi);
    sf_t[rb * kTileCols + 2 * lane] = (uint8_t)sf;
    encode_block<SR_T>(vb, __uint_as_float(mm & 0xFFFF0000u), c, inv_table, p.t_rng, (uint64_t)((ca + 1) * p.t_nkb + kb), lo, hi, sf);
    *reinterpret_cast<uint2*>(codes_t + swz128(2 * lane + 1, rb * 8)) = make_uint2(lo, hi);
    sf_t[rb * kTileCols + 2 * lane + 1] = (uint8_t)sf;
  }
  }
  }

  // ---- row output: thread -> (row, block of 16 columns); four rows per thread ----
  if constexpr (DUAL) {
    const int kbl = threadIdx.x & 3;                          // block within the tile's 64 columns
    const int t = threadIdx.x >> 2;                           // row within a group of 64; (row & 7) = t & 7 for all four groups
    const uint32_t ld_a = tile_base_after_wait(tile) + (uint32_t)t * 128u + (((uint32_t)(2 * kbl) ^ (uint32_t)(t & 7)) << 4);
    const uint32_t ld_b = ld_a ^ 16u;                         // the neighbouring 16-byte chunk
    const uint32_t st_r = smem_addr(codes_r) + (uint32_t)t * 32u + (uint32_t)kbl * 8u;
    uint8_t* sf_thread = sf_r + (t & 31) * 16 + (t >> 5) * 4 + kbl;
    const uint64_t blk_r0 = (uint64_t)((r0 + t) * p.r_nkb + c0 / 16 + kbl);
    const uint64_t blk_step = (uint64_t)(64 * p.r_nkb);
    auto row_block = [&](auto I) {
      constexpr int i = decltype(I)::value;
      const uint4 a = lds128<i * 8192>(ld_a);
      const uint4 b = lds128<i * 8192>(ld_b);
      Block16<__nv_bfloat16> blk;
      blk.w[0] = a.x; blk.w[1] = a.y; blk.w[2] = a.z; blk.w[3] = a.w;
      blk.w[4] = b.x; blk.w[5] = b.y; blk.w[6] = b.z; blk.w[7] = b.w;
      float v[16];
      const float amax = blk.unpack(v);
      uint32_t lo, hi, sf;
      encode_block<SR_R>(v, amax, c, inv_table, p.r_rng, blk_r0 + (uint64_t)i * blk_step, lo, hi, sf);
      sts64<i * 2048>(st_r, lo, hi);
      if constexpr (SWZ) {
        sf_thread[(i >> 1) * 512 + (i & 1) * 8] = (uint8_t)sf;
      } else {
        const int rl = i * 64 + t;
        if (r0 + rl < p.rows && c0 / 16 + kbl < p.r_nkb) p.r_scales[(r0 + rl) * p.r_nkb + c0 / 16 + kbl] = (uint8_t)sf;
      }
    };
    row_block(std::integral_constant<int, 0>{});
    row_block(std::integral_constant<int, 1>{});
    row_block(std::integral_constant<int, 2>{});
    row_block(std::integral_constant<int, 3>{});
  }

  // ---- codes out: tiled bulk stores from the staging buffers (clipped at the tensor edge) ----
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (threadIdx.x == 0) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(&map_ct), "r"(smem_addr(codes_t)), "r"((int)(r0 / 2)), "r"((int)c0) : "memory");
    if constexpr (DUAL)
      asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                   ::"l"(&map_cr), "r"(smem_addr(codes_r)), "r"((int)(c0 / 2)), "r"((int)r0) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }

  // ---- scales out ----
  constexpr int kSbRows = MX_T ? 32 : 16;                     // rows per scale block of the transposed output
  constexpr int kSbPerTile = kTileRows / kSbRows;             // 16 or 8 scale blocks per column
  constexpr int kKtPerTile = kSbPerTile / 4;                  // 4 or 2 scale tiles per column
  const int64_t kb0 = r0 / kSbRows;
  if constexpr (SWZ) {
    // transposed scales: one 32-bit word = four row blocks of one column
    const bool fill_upper = ((c0 & 127) == 0) && (c0 + kTileCols >= p.cols);   // nobody else owns rows 64..127
    for (int id = threadIdx.x; id < kTileCols * kKtPerTile; id += kThreads) {
      const int cl = id / kKtPerTile, t = id % kKtPerTile;
      const int64_t kt = kb0 / 4 + t;
      if (kt >= p.t_k_tiles) continue;
      const uint8_t* s4 = sf_t + (t * 4) * kTileCols + cl;
      const uint32_t val = (uint32_t)s4[0] | ((uint32_t)s4[kTileCols] << 8) | ((uint32_t)s4[2 * kTileCols] << 16) |
                           ((uint32_t)s4[3 * kTileCols] << 24);
      *reinterpret_cast<uint32_t*>(p.t_scales + sf_swizzled_offset(c0 + cl, kt * 4, p.t_k_tiles)) = val;
      if (fill_upper)
        *reinterpret_cast<uint32_t*>(p.t_scales + sf_swizzled_offset(c0 + cl + 64, kt * 4, p.t_k_tiles)) = 0u;
    }
    if constexpr (DUAL) {
      // row scales: the tile owns two whole 512-byte scale tiles (128 rows x this k-tile)
      if (threadIdx.x < 64) {
        const int h = threadIdx.x >> 5, i = threadIdx.x & 31;
        if (r0 + h * 128 < p.rows) {
          const uint4 val = *reinterpret_cast<const uint4*>(sf_r + h * 512 + i * 16);
          *reinterpret_cast<uint4*>(p.r_scales + ((r0 / 128 + h) * p.r_k_tiles + c0 / 64) * 512 + i * 16) = val;
        }
      }
    }
  } else {
    for (int id = threadIdx.x; id < kTileCols * kSbPerTile; id += kThreads) {
      const int cl = id / kSbPerTile, u = id % kSbPerTile;
      if (c0 + cl < p.cols && kb0 + u < p.t_nsb) p.t_scales[(c0 + cl) * p.t_nsb + kb0 + u] = sf_t[u * kTileCols + cl];
    }
  }
  if (threadIdx.x == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // staging must outlive the stores' reads
}

bool make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t inner, uint64_t outer,
                 uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool SR_T, bool DUAL, bool SR_R, bool SWZ, bool MX_T = false>
cudaError_t launch_tile(const CUtensorMap& mx, const CUtensorMap& mct, const CUtensorMap& mcr, const TileParams& p,
                        cudaStream_t s) {
  static DeviceFlags smem_set;   // per instantiation, per device
  if (cudaError_t e = set_max_dynamic_smem(smem_set, quantize_tile_kernel<SR_T, DUAL, SR_R, SWZ, MX_T>, kTileSmem)) return e;
  dim3 grid((unsigned)ceil_div(p.cols, kTileCols), (unsigned)ceil_div(p.rows, kTileRows));
  quantize_tile_kernel<SR_T, DUAL, SR_R, SWZ, MX_T><<<grid, kThreads, kTileSmem, s>>>(mx, mct, mcr, p);
  return cudaGetLastError();
}

template <bool DUAL, bool SWZ>
cudaError_t dispatch_tile(bool sr_t, bool sr_r, const CUtensorMap& mx, const CUtensorMap& mct, const CUtensorMap& mcr,
                          const TileParams& p, cudaStream_t s) {
  if constexpr (DUAL) {
    if (sr_t) return sr_r ? launch_tile<true, true, true, SWZ>(mx, mct, mcr, p, s) : launch_tile<true, true, false, SWZ>(mx, mct, mcr, p, s);
    return sr_r ? launch_tile<false, true, true, SWZ>(mx, mct, mcr, p, s) : launch_tile<false, true, false, SWZ>(mx, mct, mcr, p, s);
  } else {
    return sr_t ? launch_tile<true, false, false, SWZ>(mx, mct, mcr, p, s) : launch_tile<false, false, false, SWZ>(mx, mct, mcr, p, s);
  }
}

}  // namespace

// True when the tile kernel can take the tensor: bf16, rows a multiple of 32 (16-byte pitch of the
// transposed codes) and, for the row output, columns a multiple of 32 as well.
bool tile_quantizer_eligible(int dtype, int64_t rows, int64_t cols, bool dual) {
  if (dtype != NVFP4_BF16 || rows % 32 != 0) return false;
  if (dual && cols % 32 != 0) return false;
  if (ceil_div(rows, kTileRows) > 65535) return false;      // grid.y limit
  return true;
}

// Launches the tile kernel.  r_* arguments are ignored unless `dual`.  Arguments are validated by the callers.
int tile_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, const float* g, bool dual,
                  const nvfp4_rounding* rt, uint8_t* codes_t, uint8_t* scales_t,
                  const nvfp4_rounding* rr, uint8_t* codes_r, uint8_t* scales_r, int sf_layout, cudaStream_t s, bool mx_t) {
  CUtensorMap mx, mct, mcr;
  if (!make_map_2d(&mx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, x, (uint64_t)cols, (uint64_t)rows, (uint64_t)ld * 2, kTileCols,
                   kTileRows, CU_TENSOR_MAP_SWIZZLE_128B))
    return NVFP4_ERR_CUDA;
  if (!make_map_2d(&mct, CU_TENSOR_MAP_DATA_TYPE_UINT8, codes_t, (uint64_t)rows / 2, (uint64_t)cols, (uint64_t)rows / 2,
                   kTileRows / 2, kTileCols, CU_TENSOR_MAP_SWIZZLE_128B))
    return NVFP4_ERR_CUDA;
  mcr = mct;
  if (dual && !make_map_2d(&mcr, CU_TENSOR_MAP_DATA_TYPE_UINT8, codes_r, (uint64_t)cols / 2, (uint64_t)rows,
                           (uint64_t)cols / 2, kTileCols / 2, kTileRows, CU_TENSOR_MAP_SWIZZLE_NONE))
    return NVFP4_ERR_CUDA;
  TileParams p;
  p.gptr = g; p.rows = rows; p.cols = cols;
  philox_stream_init(&p.t_rng, rt->seed, rt->offset);
  p.t_scales = scales_t; p.t_nkb = rows / 16;
  p.t_nsb = mx_t ? rows / 32 : rows / 16;
  p.t_k_tiles = ceil_div(p.t_nsb, 4);
  const nvfp4_rounding* r2 = dual ? rr : rt;
  philox_stream_init(&p.r_rng, r2->seed, r2->offset);
  p.r_scales = scales_r; p.r_nkb = cols / 16; p.r_k_tiles = ceil_div(p.r_nkb, 4);
  const bool swz = sf_layout == NVFP4_SF_SWIZZLED_128x4;
  const bool sr_t = rt->mode == NVFP4_SR, sr_r = dual && rr->mode == NVFP4_SR;
  cudaError_t e;
  if (mx_t) {                                                 // MXFP4, transposed output only
    if (dual) return NVFP4_ERR_ENUM;
    if (sr_t) e = swz ? launch_tile<true, false, false, true, true>(mx, mct, mcr, p, s) : launch_tile<true, false, false, false, true>(mx, mct, mcr, p, s);
    else e = swz ? launch_tile<false, false, false, true, true>(mx, mct, mcr, p, s) : launch_tile<false, false, false, false, true>(mx, mct, mcr, p, s);
    return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
  }
  if (dual) e = swz ? dispatch_tile<true, true>(sr_t, sr_r, mx, mct, mcr, p, s) : dispatch_tile<true, false>(sr_t, sr_r, mx, mct, mcr, p, s);
  else e = swz ? dispatch_tile<false, true>(sr_t, sr_r, mx, mct, mcr, p, s) : dispatch_tile<false, false>(sr_t, sr_r, mx, mct, mcr, p, s);
  return e == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

// Reads and clears this file's device error word (set when a tile wait ran out).
int tile_error_word(unsigned int* out) {
  unsigned int w = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&w, g_tile_error_word, sizeof(w)) != cudaSuccess) return NVFP4_ERR_CUDA;
  if (w != 0 && cudaMemcpyToSymbol(g_tile_error_word, &zero, sizeof(zero)) != cudaSuccess) return NVFP4_ERR_CUDA;
  *out = w;
  return NVFP4_OK;
}

}  // namespace nvfp4
