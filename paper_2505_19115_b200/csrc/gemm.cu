// Block-scaled NVFP4 GEMM on the 5th-generation tensor cores (the contraction of Eq. 1-3):
//   D[m,n] = (gA*gB) * sum_kb sA[m,kb]*sB[n,kb] * sum_{k in kb} a[m,k]*b[n,k]
//
// Two kernels, both persistent and warp-specialised, both with every mbarrier wait bounded in time (on a timeout the
// CTA records the site in a device error word, gives its outstanding copies time to land, frees its tensor memory
// and returns):
//
//   gemm2_nvfp4_kernel   the product kernel: a cluster of two CTAs computes a 256 x 256 tile with
//                        tcgen05.mma.cta_group::2 (described above its definition); variants for bf16 / fp32 /
//                        quantized output, MXFP4 operands, bf16 operands (K-major or read in place MN-major)
//   gemm_nvfp4_kernel    the first design, one CTA per tile (128 x BN): warp 0 stages packed codes by tiled bulk
//                        copies and scale tiles by plain bulk copies, warp 1 copies the stage's scales to tensor
//                        memory with tcgen05.cp and issues 128 x BN x 64 MMAs into double-buffered accumulators,
//                        warps 2-5 read the accumulator out.  Kept as an independent second implementation that the
//                        tests compare the product kernel with, bit for bit.
#include <cuda.h>
#include <cuda_bf16.h>

#include "quantize_core.cuh"
#include "tc_ptx.cuh"
#include "tensor_map.cuh"

namespace nvfp4 {
namespace {

__device__ unsigned int g_error_word = 0;

// Cycle account of the CTA-pair kernel (debug builds only: -DNVFP4_GEMM_ACCOUNT, see microbench.py gemm_account).
// Each role of pair 0 adds up the clock64() cycles it spends in each of its waits and in its work; the product
// build compiles all of it away.
#ifdef NVFP4_GEMM_ACCOUNT
__device__ long long g_account[32];
#define ACCOUNT_VARS(...) long long __VA_ARGS__
#define ACCOUNT(var, ...) { const long long acc_t0_ = clock64(); __VA_ARGS__; var += clock64() - acc_t0_; }
#define ACCOUNT_STORE(cond, slot, value) { if (cond) g_account[slot] = (value); }
#define ACCOUNT_NOW() clock64()
#else
#define ACCOUNT_VARS(...)
#define ACCOUNT(var, ...) { __VA_ARGS__; }
#define ACCOUNT_STORE(cond, slot, value)
#define ACCOUNT_NOW() 0ll
#endif

constexpr int BM = 128;           // rows of A per tile (= UMMA M)
constexpr int BK_BYTES = 128;     // packed bytes per row per stage = 256 E2M1 values
constexpr int BK = 256;
constexpr int MMA_K = 64;         // values per tcgen05.mma (32 bytes)
constexpr int kGemmThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

template <int BN>
struct Cfg {
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr int kAccStages = (BN == 256) ? 1 : 2;
  static constexpr int kABytes = BM * BK_BYTES;                   // 16 KB
  static constexpr int kBBytes = BN * BK_BYTES;                   // 16 / 32 KB
  static constexpr int kSfaBytes = 4 * 512;                       // 128 rows x 16 blocks
  static constexpr int kSfbBytes = (BN / 128) * 4 * 512;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
  // tensor-memory columns: accumulators first, then two scale buffers (A: 16, B: BN/32*4 columns)
  static constexpr uint32_t kAccCols = BN;
  static constexpr uint32_t kSfaCol = kAccStages * BN;
  static constexpr uint32_t kSfCols = 16 + (BN / 32) * 4;         // one stage of scales
  static constexpr int kSfBufs = (kSfaCol + 2 * kSfCols <= kTmemCols) ? 2 : 1;
  static_assert(kSfaCol + kSfBufs * kSfCols <= kTmemCols, "tensor memory overflow");
};

struct GemmParams {
  const uint8_t* a_sf;
  const uint8_t* b_sf;
  const float* a_g;
  const float* b_g;
  void* d;
  int64_t ldd;
  int M, N, K;
  int tiles_m, tiles_n, k_stages;   // k_stages = ceil(K / 256)
  int k_tiles;                      // 512-byte scale tiles per row tile: ceil(K / 64) (NVFP4), ceil(K / 128) (MXFP4)
  int k_mmas;                       // instructions along K
  int a_row_tiles, b_row_tiles;     // ceil(M / 128), ceil(N / 128)
  int d_is_bf16;
};

// ------------------------------------------------------------------------------------------------
// Bounded waits (the PTX wrappers are in tc_ptx.cuh)
// ------------------------------------------------------------------------------------------------
// Bounded waits.  They return false (and record `site`) if the barrier did not flip within the time
// limit or another role of this CTA already gave up.
//
// mbar_wait spins without pause: for the MMA issuer, whose latency is the kernel's critical path.
// mbar_wait_relaxed sleeps between polls: every other role waits most of the time, and a dozen
// warps polling shared memory back to back slow the issuer's own barrier reads several times over.
__device__ __forceinline__ bool mbar_wait_timeout(uint32_t site, volatile uint32_t* abort_flag, unsigned long long t0) {
  if (*abort_flag) return true;
  if (global_timer_ns() - t0 > kWaitLimitNs) {
    *abort_flag = 1u;
    atomicOr(&g_error_word, 0x100u | site);
    return true;
  }
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t site) {
  for (int i = 0; i < 4096; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (mbar_wait_timeout(site, abort_flag, t0)) return false;
  }
}
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t site) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  while (true) {
    for (int i = 0; i < 256; ++i) {
      __nanosleep(32);
      if (mbar_try_wait(bar, parity)) return true;
    }
    if (mbar_wait_timeout(site, abort_flag, t0)) return false;
  }
}
// Wait of the MMA-issuing warp.  The poll is a relaxed one: with MMAs in flight an acquiring
// try_wait stalls its thread for ~170 cycles even when the phase is already complete, a relaxed one
// for ~40, and the issuer has only 512 cycles per stage.  Nothing the issuer does afterwards reads
// memory through the generic proxy: it issues tcgen05.mma, whose shared-memory operands were written
// by the bulk copies that completed the phase, and whose tensor-memory scales are ordered by
// tcgen05.fence::after_thread_sync.
__device__ __forceinline__ bool mbar_wait_issuer(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t site) {
  for (int i = 0; i < 4096; ++i)
    if (mbar_try_wait_relaxed(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  while (true) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_relaxed(bar, parity)) return true;
    if (mbar_wait_timeout(site, abort_flag, t0)) return false;
  }
}
// Whole-warp wait of the scale movers, relaxed polls by every lane: these warps issue tcgen05.st, and
// next to such operations an acquiring poll costs ~180 cycles even when the phase is complete (see
// mbar_wait_issuer), which with two waits per stage made the movers the slowest role.  What they read
// afterwards is shared memory written by the bulk copies that completed the phase, so the successful poll is
// followed by one acquire fence at CTA scope: relaxed observation + fence is the acquire pattern of the PTX
// memory model, paid once per wait instead of once per poll (0.3 % of the kernel in a same-process A/B).
__device__ __forceinline__ bool mbar_wait_warp_relaxed(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t site) {
  const bool ok = mbar_wait_issuer(bar, parity, abort_flag, site);
  asm volatile("fence.acq_rel.cta;" ::: "memory");
  return ok;
}
// Whole-warp wait: lane 0 polls, then every lane observes the completed phase once itself.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t site) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait_relaxed(bar, parity, abort_flag, site);
  ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
  if (ok) (void)mbar_try_wait(bar, parity);
  return ok;
}

// Tile order: panels of kPanel row tiles, column-major inside a panel, so that the CTAs running at
// the same time share both their A row tiles and their B row tiles (each operand tile is then read
// by ~8 CTAs instead of one B tile by all of them, and the wave's working set stays small in L2).
constexpr int kPanel = 8;
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int per_panel = kPanel * tiles_n;
  const int panel = tile / per_panel, in_panel = tile - panel * per_panel;
  const int height = min(kPanel, tiles_m - panel * kPanel);
  tn = in_panel / height;
  tm = panel * kPanel + in_panel - tn * height;
}

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_nvfp4_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const GemmParams p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte aligned base for the swizzled operand tiles
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  // stage layout: [A 16K][B][SFA 2K][SFB]
  const uint32_t bar_base = smem_base + C::kStages * C::kStageBytes;
  uint8_t* bar_gen = smem_gen + C::kStages * C::kStageBytes;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * C::kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * C::kStages + C::kAccStages + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * C::kStages + 2 * C::kAccStages));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.tiles_m * p.tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < C::kAccStages; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      uint32_t armed = 0, armed_ph = 0;  // per stage: armed at least once / phase of the last arming
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        int tm, tn;
        tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
        for (int ks = 0; ks < p.k_stages; ++ks) {
          if (!(ok = mbar_wait_relaxed(empty_bar(s), ph ^ 1u, abort_flag, 1))) break;
          const int kt0 = ks * 4;
          const int nkt = min(4, p.k_tiles - kt0);                        // scale tiles in this stage
          const uint32_t sf_bytes = (uint32_t)nkt * 512u;
          const uint32_t st = smem_base + s * C::kStageBytes;
          mbar_arrive_expect_tx(full_bar(s), C::kABytes + C::kBBytes + sf_bytes * (1 + BN / 128));
          armed |= 1u << s;
          armed_ph = (armed_ph & ~(1u << s)) | (ph << s);
          tma_load_2d(st, &map_a, full_bar(s), ks * BK_BYTES, tm * BM);
          tma_load_2d(st + C::kABytes, &map_b, full_bar(s), ks * BK_BYTES, tn * BN);
          bulk_load(st + C::kABytes + C::kBBytes, p.a_sf + ((int64_t)tm * p.k_tiles + kt0) * 512, sf_bytes, full_bar(s));
#pragma unroll
          for (int h = 0; h < BN / 128; ++h) {
            const int rt = min(tn * (BN / 128) + h, p.b_row_tiles - 1);   // clamp: rows past N are never stored
            bulk_load(st + C::kABytes + C::kBBytes + C::kSfaBytes + h * 2048,
                      p.b_sf + ((int64_t)rt * p.k_tiles + kt0) * 512, sf_bytes, full_bar(s));
          }
          if (++s == C::kStages) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {
        // drain: give every armed stage a bounded chance to land before the CTA exits
        for (int q = 0; q < C::kStages; ++q) {
          if (!(armed & (1u << q))) continue;
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar(q), (armed_ph >> q) & 1u) && global_timer_ns() - t0 < 1000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(BM, BN);
      int s = 0;
      uint32_t ph = 0;
      int acc = 0;
      uint32_t acc_ph = 0;
      uint32_t sfbuf = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (!(ok = mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, 2))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * C::kAccCols;
        for (int ks = 0; ks < p.k_stages; ++ks) {
          if (!(ok = mbar_wait(full_bar(s), ph, abort_flag, 3))) break;
          tc_fence_after();
          const uint32_t st = smem_base + s * C::kStageBytes;
          const int nkt = min(4, p.k_tiles - ks * 4);
          const uint32_t sfa_t = tmem_base + C::kSfaCol + sfbuf * C::kSfCols;
          const uint32_t sfb_t = sfa_t + 16;
          for (int j = 0; j < nkt; ++j) {
            tc_cp_sf(sfa_t + 4 * j, sf_desc(st + C::kABytes + C::kBBytes + 512 * j));
#pragma unroll
            for (int h = 0; h < BN / 128; ++h)
              tc_cp_sf(sfb_t + (BN / 32) * j + 4 * h, sf_desc(st + C::kABytes + C::kBBytes + C::kSfaBytes + h * 2048 + 512 * j));
          }
          const uint64_t adesc = operand_desc(st), bdesc = operand_desc(st + C::kABytes);
          for (int j = 0; j < nkt; ++j) {
            tc_mma_nvf4(d_tmem, adesc + 2u * j, bdesc + 2u * j, idesc, sfa_t + 4 * j, sfb_t + (BN / 32) * j,
                        (ks | j) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));           // frees the stage once the MMAs above have read it
          if (C::kSfBufs == 2) sfbuf ^= 1u;
          if (++s == C::kStages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar(acc));           // accumulator complete
        if (++acc == C::kAccStages) { acc = 0; acc_ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------- epilogue -------------------------------
    const int quarter = warp & 3;            // tensor-memory lanes this warp may read
    const float alpha = (p.a_g ? __ldg(p.a_g) : 1.0f) * (p.b_g ? __ldg(p.b_g) : 1.0f);
    int acc = 0;
    uint32_t acc_ph = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
      int tm, tn;
        tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
      if (!(ok = mbar_wait_warp(tfull_bar(acc), acc_ph, abort_flag, 4))) break;
      tc_fence_after();
      const int row = tm * BM + quarter * 32 + lane;
      const uint32_t t_row = tmem_base + acc * C::kAccCols + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(t_row + c0, r);
        tmem_ld_wait();
        tmem_ld_pin(r);
        const int col = tn * BN + c0;
        if (row < p.M && col < p.N) {
          if (p.d_is_bf16) {
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.d) + (int64_t)row * p.ldd + col;
            if (col + 32 <= p.N) {
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * e]) * alpha,
                                                                 __uint_as_float(r[8 * v + 2 * e + 1]) * alpha);
                  w[e] = *reinterpret_cast<const uint32_t*>(&h);
                }
                reinterpret_cast<uint4*>(dst)[v] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            } else {
              for (int e = 0; e < 32 && col + e < p.N; ++e) dst[e] = __float2bfloat16_rn(__uint_as_float(r[e]) * alpha);
            }
          } else {
            float* dst = static_cast<float*>(p.d) + (int64_t)row * p.ldd + col;
            if (col + 32 <= p.N) {
#pragma unroll
              for (int v = 0; v < 8; ++v)
                reinterpret_cast<float4*>(dst)[v] =
                    make_float4(__uint_as_float(r[4 * v]) * alpha, __uint_as_float(r[4 * v + 1]) * alpha,
                                __uint_as_float(r[4 * v + 2]) * alpha, __uint_as_float(r[4 * v + 3]) * alpha);
            } else {
              for (int e = 0; e < 32 && col + e < p.N; ++e) dst[e] = __uint_as_float(r[e]) * alpha;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == C::kAccStages) { acc = 0; acc_ph ^= 1u; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}


// ------------------------------------------------------------------------------------------------
// CTA-pair kernel (cta_group::2): a cluster of two CTAs computes a 256 x BN tile.  Each CTA stages
// its own 128 rows of A, half of the B tile and the scale tiles it needs (its A rows, all BN B
// rows); the leader CTA issues the MMAs for both, every CTA drains its own 128 accumulator rows.
// All loads are plain tiled copies (no multicast); the peer's operand copies signal the leader's
// barrier.
//
// Scales reach tensor memory through registers: four warps per CTA read the stage's scale tiles
// from shared memory and write them with tcgen05.st into one of several scale buffers, ahead of
// the MMA issuer.  (A tcgen05.cp per 512-byte scale tile costs 75-120 cycles and an NVFP4 stage
// needs 12 of them for 512 cycles of MMA work, which caps the kernel near a third of the MMA rate;
// the register path keeps up with the tensor cores.)
//
// The epilogue goes through shared memory (128-byte swizzle) and leaves as tiled bulk stores.
// Warps: 0 operand producer, 1 MMA issuer, 2-5 epilogue, 6-9 scale movers, 10 scale producer.
// ------------------------------------------------------------------------------------------------
constexpr int kGemm2Threads = 352;

template <int BN>
struct Cfg2 {
  static constexpr int kSfbTiles = (BN % 128 == 0) ? BN / 128 : BN / 128 + 1;
  static constexpr int kStages = (BN == 128) ? 6 : 5;
  static constexpr int kAccStages = (BN == 256) ? 1 : 2;
  static constexpr int kABytes = 128 * BK_BYTES;
  static constexpr int kBBytes = (BN / 2) * BK_BYTES;
  static constexpr int kSfaBytes = 2048;
  static constexpr int kSfbBytes = kSfbTiles * 2048;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;
  static constexpr int kEpiWarpBytes = 2 * 4096;                   // two 32-row x 128-byte buffers per warp
  static constexpr int kEpiBytes = 4 * kEpiWarpBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + kEpiBytes + 1024 /*align*/ + 512 /*barriers*/ + 512 /*reciprocal table*/;
  // tensor memory: accumulators, then kSfBufs scale buffers of (16 columns for A, 16 per B tile)
  static constexpr uint32_t kSfaCol = kAccStages * BN;
  static constexpr uint32_t kSfCols = 16 + kSfbTiles * 16;
  static constexpr int kSfBufsFit = (int)((kTmemCols - kSfaCol) / kSfCols);
  static constexpr int kSfBufs = kSfBufsFit > kStages ? kStages : kSfBufsFit;
  // with as many scale buffers as stages, buffer b is stage s and needs no barrier of its own
  static constexpr bool kSfFollowsStage = (kSfBufs == kStages);
  static constexpr int kNumBarriers = 4 * kStages + 2 * kSfBufs + 2 * kAccStages;
  static_assert(kStageBytes % 1024 == 0, "stage must keep the 1024-byte swizzle alignment");
  static_assert(kSfBufs >= 2, "need at least two scale buffers in tensor memory");
  static_assert(kSmemBytes <= 232448, "shared memory overflow");
  static_assert(8 * kNumBarriers + 8 <= 512, "barrier area overflow");
};

struct Gemm2Params {
  const float* a_g;
  const float* b_g;
  int M, N, K;
  int tiles_m, tiles_n, k_stages, k_tiles;
  int k_mmas;                       // instructions along K (64 values each; 16 for bf16 operands)
  int a_row_tiles, b_row_tiles;
  // quantized output (OUT == 2): per-tensor scale of the output, rounding, scales destination
  const float* out_g;
  PhiloxStream out_rng;
  uint8_t* out_scales;
  int out_sr, out_swizzled;
  int64_t out_nkb, out_k_tiles;
};

// OUT: 0 = fp32, 1 = bf16, 2 = the NVFP4 row quantization of the product (codes + scales), for a
// consumer that would quantize D along N anyway (the next layer's Q(X) of Eq. 4): no high-precision
// round trip through memory.
// BF16_IN: operands are plain bf16 [rows, K] (K-major) instead of packed codes with scales; the scale
// producer and the scale movers then have nothing to do and a k-stage is 64 values (128 bytes per row).
// MX: MXFP4 operands (blocks of 32, E8M0 scales): a 512-byte scale tile then covers 128 values, a
// stage holds two tiles per 128 rows instead of four, and two consecutive instructions share a
// scale column, each using one half of it.
// MN (bf16 operands only): bit 0 / bit 1 = operand A / B is stored with its OUTPUT axis contiguous, [K, M] or [K, N]
// row-major, instead of [M, K] / [N, K] (the backward and update products of Eq. 2-3 read W, X and dY that way): a
// stage then holds, per operand, two boxes of 64 contraction rows x 64 output rows (128 bytes), and the MMA reads
// them through MN-major descriptors, so no transposed copy of the tensor is ever made.
template <int BN, int OUT, bool BF16_IN = false, bool MX = false, int MN = 0>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemm2Threads, 1)
gemm2_nvfp4_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   const __grid_constant__ CUtensorMap map_sfa, const __grid_constant__ CUtensorMap map_sfb,
                   const __grid_constant__ CUtensorMap map_d, const Gemm2Params p) {
  using C = Cfg2<BN>;
  constexpr bool BF16_OUT = (OUT == 1), Q_OUT = (OUT == 2);
  constexpr bool MN_A = (MN & 1) != 0, MN_B = (MN & 2) != 0;
  static_assert(MN == 0 || (BF16_IN && BN == 256), "MN-major operands exist for the bf16 variant with the 256-wide tile");
  static_assert(!Q_OUT || BN == 256, "the quantized epilogue stores one 128-byte row of codes per tile row");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t epi_base = smem_base + C::kStages * C::kStageBytes;
  const uint32_t bar_base = epi_base + C::kEpiBytes;
  uint8_t* bar_gen = smem_gen + C::kStages * C::kStageBytes + C::kEpiBytes;
  // full: operands of both CTAs landed (leader's copy is the one waited on)
  // sfl:  this CTA's scale tiles landed        empty: the stage's MMAs are done (both CTAs)
  // sfr:  scale buffer written in both CTAs (leader's copy)   sfe: scale buffer free again (both CTAs)
  // sfx:  this CTA's scale tiles of the stage have been read out of shared memory: the slot is refilled then,
  //       a ring round before the stage's operands, so that scales are in tensor memory before operands land
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto sfl_bar = [&](int s) { return bar_base + 8u * (C::kStages + s); };
  auto empty_bar = [&](int s) { return bar_base + 8u * (2 * C::kStages + s); };
  auto sfr_bar = [&](int b) { return bar_base + 8u * (3 * C::kStages + b); };
  auto sfe_bar = [&](int b) { return bar_base + 8u * (3 * C::kStages + C::kSfBufs + b); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (3 * C::kStages + 2 * C::kSfBufs + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (3 * C::kStages + 2 * C::kSfBufs + C::kAccStages + a); };
  auto sfx_bar = [&](int s) { return bar_base + 8u * (3 * C::kStages + 2 * C::kSfBufs + 2 * C::kAccStages + s); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * C::kNumBarriers);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* inv_table = reinterpret_cast<float*>(bar_gen + 512);   // OUT == 2 only: 1 / (decode(q) * out_g) per scale code
  if constexpr (Q_OUT) build_inv_table(inv_table, p.out_g ? __ldg(p.out_g) : 1.0f);

  const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(sfl_bar(s), 1); mbar_init(empty_bar(s), 1); mbar_init(sfx_bar(s), 4); }
    for (int b = 0; b < C::kSfBufs; ++b) { mbar_init(sfr_bar(b), 8); mbar_init(sfe_bar(b), 1); }
    for (int a = 0; a < C::kAccStages; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc_pair(smem_u32((const void*)tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // both CTAs' barriers exist before any remote signal
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The producer and issuer warps run their loops with all 32 lanes (so that loop state, addresses and
  // descriptors stay warp-uniform) and predicate only the asynchronous instructions on one lane.
  if (warp == 0) {
    // ------------------------------- operand producer (both CTAs) -------------------------------
    // One warp can issue a tiled copy every ~75 cycles, so operands and scales have a producer each.
    const bool issuer = elect_one();
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    constexpr uint32_t kOperandTx = C::kABytes + C::kBBytes;       // per CTA, signalled on the leader's barrier
    ACCOUNT_VARS(a_wait = 0, a_total = -ACCOUNT_NOW());
    for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
      int tm, tn;
      tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
      const int m0 = tm * 256 + (int)rank * 128, n0 = tn * BN + (int)rank * (BN / 2);
      for (int ks = 0; ks < p.k_stages; ++ks) {
        // polled without sleeping: the refill of a freed stage is on the main loop's critical path (the ring is
        // five stages deep for a copy latency of three to four stage times), and a sleeping poll adds its period to it
        ACCOUNT(a_wait, ok = mbar_wait_issuer(empty_bar(s), ph ^ 1u, abort_flag, 0x11));
        if (!ok) break;
        const uint32_t st = smem_base + s * C::kStageBytes;
        const uint32_t lead_full = map_to_cta(full_bar(s), 0);
        if (issuer) {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(s), 2u * kOperandTx);
          if constexpr (MN_A) {                     // [K, M]: x = byte offset of the output row, y = contraction index
            tma_load_2d_pair(st, &map_a, lead_full, m0 * 2, ks * 64);
            tma_load_2d_pair(st + C::kABytes / 2, &map_a, lead_full, (m0 + 64) * 2, ks * 64);
          } else {
            tma_load_2d_pair(st, &map_a, lead_full, ks * BK_BYTES, m0);
          }
          if constexpr (MN_B) {
            tma_load_2d_pair(st + C::kABytes, &map_b, lead_full, n0 * 2, ks * 64);
            tma_load_2d_pair(st + C::kABytes + C::kBBytes / 2, &map_b, lead_full, (n0 + 64) * 2, ks * 64);
          } else {
            tma_load_2d_pair(st + C::kABytes, &map_b, lead_full, ks * BK_BYTES, n0);
          }
        }
        if (++s == C::kStages) { s = 0; ph ^= 1u; }
      }
    }
    ACCOUNT_STORE(pair == 0 && rank == 0 && issuer, 0, a_wait);
    ACCOUNT_STORE(pair == 0 && rank == 0 && issuer, 1, a_total + ACCOUNT_NOW());
    if (!ok && issuer) {                            // give copies in flight a bounded time to land
      const unsigned long long t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 200000ull) {}
    }
  } else if (warp == 10) {
    // ------------------------------- scale producer (both CTAs) -------------------------------
    const bool issuer = elect_one() && !BF16_IN;
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    constexpr int kSfTiles = MX ? 2 : 4;                           // 512-byte scale tiles per stage and 128 rows
    constexpr uint32_t kScaleTx = (C::kSfaBytes + C::kSfbBytes) / 4 * kSfTiles;   // signalled on this CTA's own barrier
    for (int tile = pair; !BF16_IN && ok && tile < num_tiles; tile += num_pairs) {
      int tm, tn;
      tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
      const int a_row = min(tm * 2 + (int)rank, p.a_row_tiles - 1) * p.k_tiles;
      int b_row[C::kSfbTiles];
#pragma unroll
      for (int h = 0; h < C::kSfbTiles; ++h)                       // rows past N are never stored
        b_row[h] = min((tn * BN) / 128 + h, p.b_row_tiles - 1) * p.k_tiles;
      for (int ks = 0; ks < p.k_stages; ++ks) {
        if (!(ok = mbar_wait_relaxed(sfx_bar(s), ph ^ 1u, abort_flag, 0x18))) break;
        const uint32_t sf = smem_base + s * C::kStageBytes + C::kABytes + C::kBBytes;
        if (issuer) {
          mbar_arrive_expect_tx(sfl_bar(s), kScaleTx);
          tma_load_2d(sf, &map_sfa, sfl_bar(s), 0, a_row + ks * kSfTiles);
#pragma unroll
          for (int h = 0; h < C::kSfbTiles; ++h)
            tma_load_2d(sf + C::kSfaBytes + h * 2048, &map_sfb, sfl_bar(s), 0, b_row[h] + ks * kSfTiles);
        }
        if (++s == C::kStages) { s = 0; ph ^= 1u; }
      }
    }
    if (!ok && issuer) {
      const unsigned long long t0 = global_timer_ns();
      while (global_timer_ns() - t0 < 200000ull) {}
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (leader CTA only) -------------------------------
    if (rank == 0) {
      const bool issuer = elect_one();
      constexpr uint32_t idesc = BF16_IN ? instr_desc_bf16(256, BN, MN_A, MN_B) : instr_desc(256, BN);
      int s = 0, b = 0, acc = 0;
      uint32_t ph = 0, bph = 0, acc_ph = 0;
      bool ok = true;
      ACCOUNT_VARS(a_acc = 0, a_ops = 0, a_sf = 0, a_total = -ACCOUNT_NOW());
      for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
        int tm_unused, tn;
        tile_coords(tile, p.tiles_m, p.tiles_n, tm_unused, tn);
        const uint32_t sfb_off = (uint32_t)((tn * BN) % 128) / 32;         // first scale column of this N tile
        ACCOUNT(a_acc, ok = mbar_wait_issuer(tempty_bar(acc), acc_ph ^ 1u, abort_flag, 0x12));
        if (!ok) break;
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int ks = 0; ks < p.k_stages; ++ks) {
          ACCOUNT(a_ops, ok = mbar_wait_issuer(full_bar(s), ph, abort_flag, 0x13));
          if (!ok) break;
          if constexpr (!BF16_IN) {
            ACCOUNT(a_sf, ok = mbar_wait_issuer(sfr_bar(b), bph, abort_flag, 0x15));
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t st = smem_base + s * C::kStageBytes;
          const int nkt = min(4, p.k_mmas - ks * 4);
          const uint32_t sfa_t = tmem_base + C::kSfaCol + b * C::kSfCols;
          const uint32_t sfb_t = sfa_t + 16 + sfb_off;
          const uint64_t adesc = MN_A ? operand_desc_mn(st, C::kABytes / 2) : operand_desc(st);
          const uint64_t bdesc = MN_B ? operand_desc_mn(st + C::kABytes, C::kBBytes / 2) : operand_desc(st + C::kABytes);
          if (issuer && BF16_IN) {
            // one instruction = 16 contraction indices: 32 bytes along a K-major row, 16 rows (2048 bytes) of an MN-major box
            constexpr uint32_t a_step = MN_A ? (2048u >> 4) : 2u, b_step = MN_B ? (2048u >> 4) : 2u;
            for (int j = 0; j < nkt; ++j) tc_mma_bf16_pair(d_tmem, adesc + a_step * j, bdesc + b_step * j, idesc, (ks | j) ? 1u : 0u);
            tc_commit_pair(empty_bar(s));
          } else if (issuer && MX) {
            for (int j = 0; j < nkt; ++j)
              tc_mma_mxf4_pair(d_tmem, adesc + 2u * j, bdesc + 2u * j, (j & 1) ? instr_desc_mx(256, BN, 1) : instr_desc_mx(256, BN, 0),
                               sfa_t + 4 * (j >> 1), sfb_t + 4 * C::kSfbTiles * (j >> 1), (ks | j) ? 1u : 0u);
            tc_commit_pair(empty_bar(s));
            if constexpr (!C::kSfFollowsStage) tc_commit_pair(sfe_bar(b));
          } else if (issuer) {
            if (nkt == 4) {
#pragma unroll
              for (int j = 0; j < 4; ++j)
                tc_mma_nvf4_pair(d_tmem, adesc + 2u * j, bdesc + 2u * j, idesc, sfa_t + 4 * j,
                                 sfb_t + 4 * C::kSfbTiles * j, (ks | j) ? 1u : 0u);
            } else {
              for (int j = 0; j < nkt; ++j)
                tc_mma_nvf4_pair(d_tmem, adesc + 2u * j, bdesc + 2u * j, idesc, sfa_t + 4 * j,
                                 sfb_t + 4 * C::kSfbTiles * j, (ks | j) ? 1u : 0u);
            }
            tc_commit_pair(empty_bar(s));           // shared-memory stage free in both CTAs
            if constexpr (!C::kSfFollowsStage) tc_commit_pair(sfe_bar(b));   // scale buffer free in both CTAs
          }
          if (++s == C::kStages) { s = 0; ph ^= 1u; }
          if (++b == C::kSfBufs) { b = 0; bph ^= 1u; }
        }
        if (!ok) break;
        if (issuer) tc_commit_pair(tfull_bar(acc));
        if (++acc == C::kAccStages) { acc = 0; acc_ph ^= 1u; }
      }
      ACCOUNT_STORE(pair == 0 && issuer, 4, a_acc);
      ACCOUNT_STORE(pair == 0 && issuer, 5, a_ops);
      ACCOUNT_STORE(pair == 0 && issuer, 6, a_sf);
      ACCOUNT_STORE(pair == 0 && issuer, 7, a_total + ACCOUNT_NOW());
    }
  } else if (warp >= 6) {                           // warps 6-9 (warp 10 was taken above)
    // ------------------------------- scale movers (both CTAs) -------------------------------
    // Shared-memory scale tile: row l (16 bytes) = four 32-row groups x four k-blocks.  Tensor
    // memory wants exactly that word in lane l of every 32-lane quarter, one column per group.
    const int quarter = warp & 3;
    const uint32_t lane_field = (uint32_t)(quarter * 32) << 16;
    const uint32_t lead_sfr0 = map_to_cta(sfr_bar(0), 0);
    int s = 0, b = 0;
    uint32_t ph = 0, bph = 0;
    bool ok = true;
    ACCOUNT_VARS(a_land = 0, a_free = 0, a_total = -ACCOUNT_NOW());
    for (int tile = pair; !BF16_IN && ok && tile < num_tiles; tile += num_pairs) {
      for (int ks = 0; ks < p.k_stages; ++ks) {
        ACCOUNT(a_land, ok = mbar_wait_warp_relaxed(sfl_bar(s), ph, abort_flag, 0x16));
        if (!ok) break;
        if constexpr (!C::kSfFollowsStage) {
          ACCOUNT(a_free, ok = mbar_wait_warp_relaxed(sfe_bar(b), bph ^ 1u, abort_flag, 0x17));
        } else {                                    // buffer b == stage s: free once that stage's previous MMAs are done
          ACCOUNT(a_free, ok = mbar_wait_warp_relaxed(empty_bar(s), ph ^ 1u, abort_flag, 0x17));
        }
        if (!ok) break;
        tc_fence_after();
        const uint8_t* sf = smem_gen + s * C::kStageBytes + C::kABytes + C::kBBytes + lane * 16;
        const uint32_t t_sf = tmem_base + C::kSfaCol + b * C::kSfCols + lane_field;
        {
          uint32_t r[16];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint4 v = *reinterpret_cast<const uint4*>(sf + j * 512);
            r[4 * j] = v.x; r[4 * j + 1] = v.y; r[4 * j + 2] = v.z; r[4 * j + 3] = v.w;
          }
          tmem_st16(t_sf, r);
        }
#pragma unroll
        for (int c = 0; c < C::kSfbTiles; ++c) {    // 16 columns at a time: column x = 4*T*j + 4*h + w
          uint32_t r[16];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int x = 16 * c + 4 * q, j = x / (4 * C::kSfbTiles), h = (x / 4) % C::kSfbTiles;
            const uint4 v = *reinterpret_cast<const uint4*>(sf + C::kSfaBytes + h * 2048 + j * 512);
            r[4 * q] = v.x; r[4 * q + 1] = v.y; r[4 * q + 2] = v.z; r[4 * q + 3] = v.w;
          }
          tmem_st16(t_sf + 16 + 16 * c, r);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(sfx_bar(s));     // the tiles are in registers: the slot may be refilled
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lead_sfr0 + 8u * b);
        if (++s == C::kStages) { s = 0; ph ^= 1u; }
        if (++b == C::kSfBufs) { b = 0; bph ^= 1u; }
      }
    }
    ACCOUNT_STORE(pair == 0 && rank == 0 && warp == 6 && lane == 0, 8, a_land);
    ACCOUNT_STORE(pair == 0 && rank == 0 && warp == 6 && lane == 0, 9, a_free);
    ACCOUNT_STORE(pair == 0 && rank == 0 && warp == 6 && lane == 0, 10, a_total + ACCOUNT_NOW());
  } else {
    // ------------------------------- epilogue (both CTAs, warps 2-5) -------------------------------
    const int quarter = warp & 3;
    const float alpha = (p.a_g ? __ldg(p.a_g) : 1.0f) * (p.b_g ? __ldg(p.b_g) : 1.0f);
    const uint32_t my_buf = epi_base + quarter * C::kEpiWarpBytes;
    constexpr int kChunkCols = BF16_OUT ? 64 : 32;
    constexpr int kLoads = kChunkCols / 32;
    const uint32_t lead_tempty0 = map_to_cta(tempty_bar(0), 0);
    int acc = 0;
    uint32_t acc_ph = 0, chunk_no = 0;
    bool ok = true;
    ACCOUNT_VARS(a_tile = 0, a_read = 0, a_total = -ACCOUNT_NOW(), a_read_t0 = 0);
    for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
      int tm, tn;
      tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
      ACCOUNT(a_tile, ok = mbar_wait_warp(tfull_bar(acc), acc_ph, abort_flag, 0x14));
      if (!ok) break;
#ifdef NVFP4_GEMM_ACCOUNT
      a_read_t0 = clock64();
#endif
      tc_fence_after();
      const int row0 = tm * 256 + (int)rank * 128 + quarter * 32;
      const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(quarter * 32) << 16);
      if constexpr (Q_OUT) {
        // ---- quantized output: this lane's row, the tile's 256 columns = 16 blocks of 16 ----
        const float cq = __fdiv_rn(__fdiv_rn(1.0f, 6.0f), p.out_g ? __ldg(p.out_g) : 1.0f);
        const int64_t row = (int64_t)row0 + lane;
        uint32_t codes[32];                          // 128 bytes of codes
        uint32_t sfw[4] = {0u, 0u, 0u, 0u};          // 16 scale bytes, four per k-tile
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint32_t r[32];
          tmem_ld32(t_row + 32 * c, r);
          tmem_ld_wait();
          tmem_ld_pin(r);
          if (c == 7) {                              // accumulator fully read: hand it back to the leader
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_tempty0 + 8u * acc);
          }
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float v[16], amax = 0.0f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              v[j] = __uint_as_float(r[16 * h + j]) * alpha;     // the value the fp32 epilogue would store
              amax = fmaxf(amax, fabsf(v[j]));
            }
            const int kbl = 2 * c + h;
            const uint64_t blk = (uint64_t)(row * p.out_nkb + (int64_t)tn * (BN / 16) + kbl);
            uint32_t lo, hi, sf;
            if (p.out_sr) encode_block<true>(v, amax, cq, inv_table, p.out_rng, blk, lo, hi, sf);
            else encode_block<false>(v, amax, cq, inv_table, p.out_rng, blk, lo, hi, sf);
            codes[2 * kbl] = lo;
            codes[2 * kbl + 1] = hi;
            sfw[kbl >> 2] |= sf << (8 * (kbl & 3));
          }
        }
        // codes: stage 32 rows x 128 bytes (128-byte swizzle) and store them as one box
        const uint32_t buf = my_buf + (chunk_no & 1u) * 4096u;
        if (chunk_no >= 2) {
          if (lane == 0) tma_store_wait_read<1>();
          __syncwarp();
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t dst = buf + lane * 128 + ((c ^ (lane & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(codes[4 * c]), "r"(codes[4 * c + 1]),
                       "r"(codes[4 * c + 2]), "r"(codes[4 * c + 3]) : "memory");
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&map_d, buf, tn * (BN / 2), row0);
          tma_store_commit();
        }
        ++chunk_no;
        // scales
        if (p.out_swizzled) {
          if ((row >> 7) < (((int64_t)p.M + 127) >> 7)) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              const int64_t kt = (int64_t)tn * (BN / 64) + t;
              if (kt < p.out_k_tiles)
                *reinterpret_cast<uint32_t*>(p.out_scales + sf_swizzled_offset(row, kt * 4, p.out_k_tiles)) = sfw[t];
            }
          }
        } else if (row < p.M) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int64_t kb = (int64_t)tn * (BN / 16) + i;
            if (kb < p.out_nkb) p.out_scales[row * p.out_nkb + kb] = (uint8_t)(sfw[i >> 2] >> (8 * (i & 3)));
          }
        }
        if (++acc == C::kAccStages) { acc = 0; acc_ph ^= 1u; }
        continue;
      }
      // The MMA issuer cannot start the next tile before this accumulator is read out, so the read-out is
      // what must finish early, not the stores: the first kHeld chunks are converted and parked in
      // registers, the others stream through the staging buffers, the accumulator is handed back
      // as soon as the last of them is read, and the parked chunks are stored after that.
      constexpr int kChunks = BN / kChunkCols;
      constexpr int kHeld = (kChunks > 3) ? 3 : kChunks - 1;

      // one chunk: accumulator columns [c0, c0 + kChunkCols) -> 32 output words (scaled, converted)
      auto read_chunk = [&](int c0, uint32_t (&w)[32]) {
        uint32_t r[kLoads][32];
#pragma unroll
        for (int l = 0; l < kLoads; ++l) tmem_ld32(t_row + c0 + 32 * l, r[l]);
        tmem_ld_wait();
#pragma unroll
        for (int l = 0; l < kLoads; ++l) tmem_ld_pin(r[l]);
        if constexpr (BF16_OUT) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(r[0][2 * e]) * alpha, __uint_as_float(r[0][2 * e + 1]) * alpha);
            const __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(r[kLoads - 1][2 * e]) * alpha, __uint_as_float(r[kLoads - 1][2 * e + 1]) * alpha);
            w[e] = *reinterpret_cast<const uint32_t*>(&h0);
            w[16 + e] = *reinterpret_cast<const uint32_t*>(&h1);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) w[e] = __float_as_uint(__uint_as_float(r[0][e]) * alpha);
        }
      };
      // stage 32 rows x 128 bytes (row = lane, eight 16-byte pieces, piece index XOR (row & 7): the
      // 128-byte swizzle) and send them off as one tiled store
      auto store_chunk = [&](int c0, const uint32_t (&w)[32]) {
        const uint32_t buf = my_buf + (chunk_no & 1u) * 4096u;
        if (chunk_no >= 2) {                        // the store issued two chunks ago has read this buffer
          if (lane == 0) tma_store_wait_read<1>();
          __syncwarp();
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t dst = buf + lane * 128 + ((c ^ (lane & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w[4 * c]), "r"(w[4 * c + 1]),
                       "r"(w[4 * c + 2]), "r"(w[4 * c + 3]) : "memory");
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&map_d, buf, tn * BN + c0, row0);
          tma_store_commit();
        }
        ++chunk_no;
      };

      uint32_t held[kHeld][32];
#pragma unroll
      for (int h = 0; h < kHeld; ++h) read_chunk(h * kChunkCols, held[h]);
#pragma unroll 1
      for (int c = kHeld; c < kChunks; ++c) {
        uint32_t w[32];
        read_chunk(c * kChunkCols, w);
        if (c == kChunks - 1) {                     // accumulator fully read: hand it back to the leader
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(lead_tempty0 + 8u * acc);
#ifdef NVFP4_GEMM_ACCOUNT
          a_read += clock64() - a_read_t0;
#endif
        }
        store_chunk(c * kChunkCols, w);
      }
#pragma unroll
      for (int h = 0; h < kHeld; ++h) store_chunk(h * kChunkCols, held[h]);
      if (++acc == C::kAccStages) { acc = 0; acc_ph ^= 1u; }
    }
    if (lane == 0) tma_store_wait_all();
    ACCOUNT_STORE(pair == 0 && rank == 0 && warp == 2 && lane == 0, 12, a_tile);
    ACCOUNT_STORE(pair == 0 && rank == 0 && warp == 2 && lane == 0, 13, a_read);
    ACCOUNT_STORE(pair == 0 && rank == 0 && warp == 2 && lane == 0, 14, a_total + ACCOUNT_NOW());
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // the peer's MMAs and loads are done before anyone frees or exits
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
// Packed codes [rows, row_bytes] -> box of (128 bytes x box_rows), 128-byte swizzle, zero fill.
bool make_codes_map(CUtensorMap* map, const uint8_t* base, int64_t rows, int64_t row_bytes, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)BK_BYTES, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Scale tiles as a 2-D tensor of 32-bit words: one 512-byte tile per row, boxes of four tiles.
bool make_sf_map(CUtensorMap* map, const uint8_t* base, int64_t n_tiles, int box_tiles = 4) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {128, (cuuint64_t)n_tiles};
  const cuuint64_t strides[1] = {512};
  const cuuint32_t box[2] = {128, (cuuint32_t)box_tiles};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint8_t*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output D[M, N] (row pitch ldd elements) -> boxes of 32 rows x 128 bytes, 128-byte swizzle.
bool make_out_map(CUtensorMap* map, void* base, int64_t M, int64_t N, int64_t ldd, bool bf16) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t esz = bf16 ? 2 : 4;
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)ldd * esz};
  const cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides,
            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
int launch_gemm(const uint8_t* a_codes, const uint8_t* b_codes, GemmParams p, cudaStream_t s) {
  using C = Cfg<BN>;
  CUtensorMap map_a, map_b;
  if (!make_codes_map(&map_a, a_codes, p.M, p.K / 2, BM)) return NVFP4_ERR_CUDA;
  if (!make_codes_map(&map_b, b_codes, p.N, p.K / 2, BN)) return NVFP4_ERR_CUDA;
  p.tiles_m = (p.M + BM - 1) / BM;
  p.tiles_n = (p.N + BN - 1) / BN;
  static DeviceFlags smem_set;                         // per instantiation, per device
  if (set_max_dynamic_smem(smem_set, gemm_nvfp4_kernel<BN>, C::kSmemBytes) != cudaSuccess) return NVFP4_ERR_CUDA;
  const int tiles = p.tiles_m * p.tiles_n;
  const int grid = tiles < sm_count() ? tiles : sm_count();
  gemm_nvfp4_kernel<BN><<<grid, kGemmThreads, C::kSmemBytes, s>>>(map_a, map_b, p);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

// Output of the quantized epilogue (OUT == 2); unused otherwise.
struct QuantOut {
  const float* g = nullptr;
  const nvfp4_rounding* rounding = nullptr;
  uint8_t* codes = nullptr;
  uint8_t* scales = nullptr;
  int sf_layout = NVFP4_SF_LINEAR;
};

// Packed codes of the quantized output [M, N/2 bytes] -> boxes of 32 rows x 128 bytes, 128-byte swizzle.
bool make_qout_map(CUtensorMap* map, uint8_t* base, int64_t M, int64_t N) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)(N / 2), (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)(N / 2)};
  const cuuint32_t box[2] = {128, 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int OUT, bool BF16_IN = false, bool MX = false, int MN = 0>
int launch_gemm2(const uint8_t* a_codes, const uint8_t* b_codes, const GemmParams& g, cudaStream_t s,
                 const QuantOut& q = QuantOut()) {
  using C = Cfg2<BN>;
  CUtensorMap map_a, map_b, map_sfa, map_sfb, map_d;
  const int64_t row_bytes = BF16_IN ? (int64_t)g.K * 2 : g.K / 2;       // operand rows as bytes
  // MN-major bf16 operand: the tensor is [K, rows] with the output axis contiguous; boxes of 64 contraction rows x 128 bytes
  if (!((MN & 1) ? make_codes_map(&map_a, a_codes, g.K, (int64_t)g.M * 2, 64) : make_codes_map(&map_a, a_codes, g.M, row_bytes, 128)))
    return NVFP4_ERR_CUDA;
  if (!((MN & 2) ? make_codes_map(&map_b, b_codes, g.K, (int64_t)g.N * 2, 64) : make_codes_map(&map_b, b_codes, g.N, row_bytes, BN / 2)))
    return NVFP4_ERR_CUDA;
  if constexpr (BF16_IN) {
    map_sfa = map_a;                                                     // never used by the kernel
    map_sfb = map_b;
  } else {
    if (!make_sf_map(&map_sfa, g.a_sf, (int64_t)g.a_row_tiles * g.k_tiles, MX ? 2 : 4)) return NVFP4_ERR_CUDA;
    if (!make_sf_map(&map_sfb, g.b_sf, (int64_t)g.b_row_tiles * g.k_tiles, MX ? 2 : 4)) return NVFP4_ERR_CUDA;
  }
  if constexpr (OUT == 2) {
    if (!make_qout_map(&map_d, q.codes, g.M, g.N)) return NVFP4_ERR_CUDA;
  } else {
    if (!make_out_map(&map_d, g.d, g.M, g.N, g.ldd, OUT == 1)) return NVFP4_ERR_CUDA;
  }
  Gemm2Params p;
  p.a_g = g.a_g; p.b_g = g.b_g; p.M = g.M; p.N = g.N; p.K = g.K;
  p.tiles_m = (g.M + 255) / 256;
  p.tiles_n = (g.N + BN - 1) / BN;
  p.k_stages = g.k_stages; p.k_tiles = g.k_tiles;
  p.k_mmas = g.k_mmas;
  p.a_row_tiles = g.a_row_tiles; p.b_row_tiles = g.b_row_tiles;
  p.out_g = q.g; p.out_scales = q.scales; p.out_sr = 0; p.out_swizzled = q.sf_layout == NVFP4_SF_SWIZZLED_128x4;
  p.out_nkb = g.N / 16; p.out_k_tiles = ceil_div(p.out_nkb, 4);
  philox_stream_init(&p.out_rng, q.rounding ? q.rounding->seed : 0, q.rounding ? q.rounding->offset : 0);
  if (q.rounding) p.out_sr = q.rounding->mode == NVFP4_SR;
  static DeviceFlags smem_set;                         // per instantiation, per device
  if (set_max_dynamic_smem(smem_set, gemm2_nvfp4_kernel<BN, OUT, BF16_IN, MX, MN>, C::kSmemBytes) != cudaSuccess)
    return NVFP4_ERR_CUDA;
  const int tiles = p.tiles_m * p.tiles_n;
  const int max_pairs = sm_count() / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  gemm2_nvfp4_kernel<BN, OUT, BF16_IN, MX, MN><<<2 * pairs, kGemm2Threads, C::kSmemBytes, s>>>(map_a, map_b, map_sfa, map_sfb, map_d, p);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

template <int BN>
int launch_gemm2_dt(const uint8_t* a_codes, const uint8_t* b_codes, const GemmParams& g, cudaStream_t s) {
  return g.d_is_bf16 ? launch_gemm2<BN, 1>(a_codes, b_codes, g, s) : launch_gemm2<BN, 0>(a_codes, b_codes, g, s);
}

}  // namespace

// 0 = automatic.  128 / 256: single-CTA kernel with that tile width.  2128 / 2192 / 2256: CTA-pair
// kernel with a 256 x {128,192,256} tile.
int gemm_tile_n_override = 0;

}  // namespace nvfp4

using namespace nvfp4;

extern "C" int nvfp4_gemm_set_tile_n(int bn) {
  if (bn != 0 && bn != 128 && bn != 256 && bn != 2128 && bn != 2192 && bn != 2256) return NVFP4_ERR_ENUM;
  gemm_tile_n_override = bn;
  return NVFP4_OK;
}

extern "C" int nvfp4_gemm(const uint8_t* a_codes, const uint8_t* a_sf, const float* a_g,
                          const uint8_t* b_codes, const uint8_t* b_sf, const float* b_g,
                          int64_t M, int64_t N, int64_t K, void* d, int d_dtype, int64_t ldd, void* cuda_stream) {
  if (!a_codes || !a_sf || !b_codes || !b_sf || !d) return NVFP4_ERR_NULL;
  if (d_dtype != NVFP4_BF16 && d_dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (M <= 0 || N <= 0 || K <= 0 || (K % 32) != 0 || ldd < N) return NVFP4_ERR_SHAPE;
  if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256 || K >= (1ll << 31) - 256) return NVFP4_ERR_SHAPE;
  const int64_t esz = (d_dtype == NVFP4_BF16) ? 2 : 4;
  if (!aligned16(a_codes) || !aligned16(a_sf) || !aligned16(b_codes) || !aligned16(b_sf) || !aligned16(d) ||
      ((ldd * esz) % 16) != 0)
    return NVFP4_ERR_ALIGN;
  if ((a_g && (reinterpret_cast<uintptr_t>(a_g) & 3u)) || (b_g && (reinterpret_cast<uintptr_t>(b_g) & 3u)))
    return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;

  GemmParams p;
  p.a_sf = a_sf; p.b_sf = b_sf; p.a_g = a_g; p.b_g = b_g; p.d = d; p.ldd = ldd;
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.k_stages = (int)ceil_div(K, BK);
  p.k_tiles = (int)ceil_div(K, MMA_K);
  p.k_mmas = p.k_tiles;
  p.a_row_tiles = (int)ceil_div(M, 128);
  p.b_row_tiles = (int)ceil_div(N, 128);
  p.d_is_bf16 = (d_dtype == NVFP4_BF16);
  p.tiles_m = p.tiles_n = 0;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int bn = gemm_tile_n_override ? gemm_tile_n_override : 2256;
  switch (bn) {
    case 128: return launch_gemm<128>(a_codes, b_codes, p, s);
    case 256: return launch_gemm<256>(a_codes, b_codes, p, s);
    case 2128: return launch_gemm2_dt<128>(a_codes, b_codes, p, s);
    case 2192: return launch_gemm2_dt<192>(a_codes, b_codes, p, s);
    default: return launch_gemm2_dt<256>(a_codes, b_codes, p, s);
  }
}

extern "C" int nvfp4_gemm_quantized(const uint8_t* a_codes, const uint8_t* a_sf, const float* a_g,
                                    const uint8_t* b_codes, const uint8_t* b_sf, const float* b_g,
                                    int64_t M, int64_t N, int64_t K,
                                    const float* out_global_scale, const nvfp4_rounding* rounding,
                                    uint8_t* out_codes, uint8_t* out_scales, int sf_layout, void* cuda_stream) {
  if (!a_codes || !a_sf || !b_codes || !b_sf || !rounding || !out_codes || !out_scales) return NVFP4_ERR_NULL;
  if ((rounding->mode != NVFP4_RTN && rounding->mode != NVFP4_SR) || rounding->reserved != 0) return NVFP4_ERR_ENUM;
  if (sf_layout != NVFP4_SF_LINEAR && sf_layout != NVFP4_SF_SWIZZLED_128x4) return NVFP4_ERR_ENUM;
  if (M <= 0 || N <= 0 || K <= 0 || (K % 32) != 0 || (N % 32) != 0) return NVFP4_ERR_SHAPE;
  if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256 || K >= (1ll << 31) - 256) return NVFP4_ERR_SHAPE;
  if (!aligned16(a_codes) || !aligned16(a_sf) || !aligned16(b_codes) || !aligned16(b_sf) || !aligned16(out_codes) ||
      !aligned16(out_scales))
    return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  GemmParams p;
  p.a_sf = a_sf; p.b_sf = b_sf; p.a_g = a_g; p.b_g = b_g; p.d = nullptr; p.ldd = N;
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.k_stages = (int)ceil_div(K, BK);
  p.k_tiles = (int)ceil_div(K, MMA_K);
  p.k_mmas = p.k_tiles;
  p.a_row_tiles = (int)ceil_div(M, 128);
  p.b_row_tiles = (int)ceil_div(N, 128);
  p.d_is_bf16 = 0;
  p.tiles_m = p.tiles_n = 0;
  QuantOut q;
  q.g = out_global_scale; q.rounding = rounding; q.codes = out_codes; q.scales = out_scales; q.sf_layout = sf_layout;
  return launch_gemm2<256, 2>(a_codes, b_codes, p, static_cast<cudaStream_t>(cuda_stream), q);
}

extern "C" int nvfp4_gemm_mx(const uint8_t* a_codes, const uint8_t* a_sf, const float* a_g,
                             const uint8_t* b_codes, const uint8_t* b_sf, const float* b_g,
                             int64_t M, int64_t N, int64_t K, void* d, int d_dtype, int64_t ldd, void* cuda_stream) {
  if (!a_codes || !a_sf || !b_codes || !b_sf || !d) return NVFP4_ERR_NULL;
  if (d_dtype != NVFP4_BF16 && d_dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (M <= 0 || N <= 0 || K <= 0 || (K % 32) != 0 || ldd < N) return NVFP4_ERR_SHAPE;
  if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256 || K >= (1ll << 31) - 256) return NVFP4_ERR_SHAPE;
  const int64_t esz = (d_dtype == NVFP4_BF16) ? 2 : 4;
  if (!aligned16(a_codes) || !aligned16(a_sf) || !aligned16(b_codes) || !aligned16(b_sf) || !aligned16(d) ||
      ((ldd * esz) % 16) != 0)
    return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  GemmParams p;
  p.a_sf = a_sf; p.b_sf = b_sf; p.a_g = a_g; p.b_g = b_g; p.d = d; p.ldd = ldd;
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.k_stages = (int)ceil_div(K, BK);
  p.k_tiles = (int)ceil_div(K, 128);                 // one 512-byte scale tile covers four blocks of 32
  p.k_mmas = (int)ceil_div(K, MMA_K);
  p.a_row_tiles = (int)ceil_div(M, 128);
  p.b_row_tiles = (int)ceil_div(N, 128);
  p.d_is_bf16 = (d_dtype == NVFP4_BF16);
  p.tiles_m = p.tiles_n = 0;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  return p.d_is_bf16 ? launch_gemm2<256, 1, false, true>(a_codes, b_codes, p, s)
                     : launch_gemm2<256, 0, false, true>(a_codes, b_codes, p, s);
}

namespace {
int gemm_bf16_any(const void* a, int a_mn, const void* b, int b_mn, int64_t M, int64_t N, int64_t K,
                  void* d, int d_dtype, int64_t ldd, void* cuda_stream);
}

extern "C" int nvfp4_gemm_bf16(const void* a, const void* b, int64_t M, int64_t N, int64_t K,
                               void* d, int d_dtype, int64_t ldd, void* cuda_stream) {
  return gemm_bf16_any(a, 0, b, 0, M, N, K, d, d_dtype, ldd, cuda_stream);
}

extern "C" int nvfp4_gemm_bf16_ex(const void* a, int a_mn_major, const void* b, int b_mn_major, int64_t M, int64_t N, int64_t K,
                                  void* d, int d_dtype, int64_t ldd, void* cuda_stream) {
  if ((a_mn_major != 0 && a_mn_major != 1) || (b_mn_major != 0 && b_mn_major != 1)) return NVFP4_ERR_ENUM;
  if (a_mn_major && !b_mn_major) return NVFP4_ERR_ENUM;      // no product of Eq. 1-3 has that shape; not instantiated
  return gemm_bf16_any(a, a_mn_major, b, b_mn_major, M, N, K, d, d_dtype, ldd, cuda_stream);
}

namespace {
int gemm_bf16_any(const void* a, int a_mn, const void* b, int b_mn, int64_t M, int64_t N, int64_t K,
                  void* d, int d_dtype, int64_t ldd, void* cuda_stream) {
  if (!a || !b || !d) return NVFP4_ERR_NULL;
  if ((a_mn && M % 8 != 0) || (b_mn && N % 8 != 0)) return NVFP4_ERR_SHAPE;   // 16-byte row pitch of an MN-major operand
  if (d_dtype != NVFP4_BF16 && d_dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (M <= 0 || N <= 0 || K <= 0 || (K % 16) != 0 || ldd < N) return NVFP4_ERR_SHAPE;
  if (M >= (1ll << 31) - 256 || N >= (1ll << 31) - 256 || K >= (1ll << 30)) return NVFP4_ERR_SHAPE;
  const int64_t esz = (d_dtype == NVFP4_BF16) ? 2 : 4;
  if (!aligned16(a) || !aligned16(b) || !aligned16(d) || ((ldd * esz) % 16) != 0) return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  GemmParams p;
  p.a_sf = p.b_sf = nullptr; p.a_g = p.b_g = nullptr; p.d = d; p.ldd = ldd;
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.k_stages = (int)ceil_div(K * 2, BK_BYTES);       // 64 bf16 values per stage
  p.k_tiles = (int)(K / 16);                         // 32-byte steps = one MMA each
  p.k_mmas = p.k_tiles;
  p.a_row_tiles = (int)ceil_div(M, 128);
  p.b_row_tiles = (int)ceil_div(N, 128);
  p.d_is_bf16 = (d_dtype == NVFP4_BF16);
  p.tiles_m = p.tiles_n = 0;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const uint8_t* ab = static_cast<const uint8_t*>(a);
  const uint8_t* bb = static_cast<const uint8_t*>(b);
  const int mn = (a_mn ? 1 : 0) | (b_mn ? 2 : 0);
  switch (mn) {
    case 0: return p.d_is_bf16 ? launch_gemm2<256, 1, true>(ab, bb, p, s) : launch_gemm2<256, 0, true>(ab, bb, p, s);
    case 2: return p.d_is_bf16 ? launch_gemm2<256, 1, true, false, 2>(ab, bb, p, s) : launch_gemm2<256, 0, true, false, 2>(ab, bb, p, s);
    case 3: return p.d_is_bf16 ? launch_gemm2<256, 1, true, false, 3>(ab, bb, p, s) : launch_gemm2<256, 0, true, false, 3>(ab, bb, p, s);
    default: return NVFP4_ERR_ENUM;
  }
}
}  // namespace

extern "C" int nvfp4_device_error_word(uint32_t* host_out) {
  if (!host_out) return NVFP4_ERR_NULL;
  unsigned int w = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&w, g_error_word, sizeof(w)) != cudaSuccess) return NVFP4_ERR_CUDA;
  if (w != 0 && cudaMemcpyToSymbol(g_error_word, &zero, sizeof(zero)) != cudaSuccess) return NVFP4_ERR_CUDA;
  unsigned int tile_w = 0;
  if (int st = tile_error_word(&tile_w)) return st;
  w |= tile_w;
  *host_out = w;
  return NVFP4_OK;
}

#ifdef NVFP4_GEMM_ACCOUNT
// Debug builds only: the cycle account of the last CTA-pair launch (32 values, host pointer).
//   [0] operand producer: waiting for a free stage   [1] its total
//   [4] issuer: waiting for the accumulator          [5] waiting for operands   [6] waiting for scales   [7] its total
//   [8] scale mover: waiting for scale tiles to land [9] waiting for a free scale buffer   [10] its total
//   [12] epilogue warp: waiting for a finished tile  [13] reading the accumulator out      [14] its total
extern "C" NVFP4_API int nvfp4_debug_gemm_account(long long* host_out) {
  if (!host_out) return NVFP4_ERR_NULL;
  return cudaMemcpyFromSymbol(host_out, g_account, sizeof(long long) * 32) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}
#endif
