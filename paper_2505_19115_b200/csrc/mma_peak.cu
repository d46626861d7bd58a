// Issue-rate measurement of the block-scaled FP4 tensor-core instruction the GEMM is built on:
// tcgen05.mma.cta_group::2.kind::mxf4nvf4 (256 x 256 x 64 per instruction) issued back to back on
// operands that stay resident in shared memory and scales that stay resident in tensor memory: no loads,
// no epilogue.  What it reports is the ceiling the tensor pipe itself sets at the clock the run held, the
// denominator for "how much of the issue rate does the GEMM reach" (the contraction of Eq. 1-3).
#include "common.cuh"
#include "tc_ptx.cuh"

namespace nvfp4 {
namespace {

constexpr int kPeakThreads = 128;
constexpr int kPeakOperandBytes = 32768;     // per CTA: 128 rows of A and 128 rows of B, 128 bytes (256 values) each
constexpr unsigned long long kPeakWaitLimitNs = 2000000000ull;

// out[3 * pair + 0] = cycles from the first issue to the completion of the last instruction (leader CTA's clock),
// out[3 * pair + 1] = instructions issued, out[3 * pair + 2] = 1 if the wait for completion ran out.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPeakThreads, 1)
mma_peak_kernel(int stages, int instr_n, int64_t* out) {
  __shared__ __align__(1024) uint8_t operands[kPeakOperandBytes];
  __shared__ __align__(8) uint64_t done_bar_storage;
  __shared__ uint32_t tmem_slot;
  const int warp = threadIdx.x >> 5;
  const uint32_t rank = cluster_ctarank();
  const uint32_t done_bar = smem_u32(&done_bar_storage);

  if (threadIdx.x == 0) {
    mbar_init(done_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc_pair(smem_u32(&tmem_slot), 512);
  // operand bytes: any nibble is a valid E2M1 code; a multiplicative hash keeps the data lines toggling
  for (int i = threadIdx.x; i < kPeakOperandBytes / 4; i += kPeakThreads)
    reinterpret_cast<uint32_t*>(operands)[i] = (uint32_t)(i + 1 + (int)blockIdx.x * 8191) * 2654435761u;
  fence_async_smem();                          // generic-proxy writes -> visible to the tensor core's reads
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);

  // scales: 1.0 (UE4M3 0x38) in every byte of 48 columns (16 for A, 32 for the 256 rows of B), all 128 lanes
  {
    uint32_t ones[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) ones[i] = 0x38383838u;
    const uint32_t t_sf = tmem_base + 256u + ((uint32_t)(warp * 32) << 16);
    tmem_st16(t_sf, ones);
    tmem_st16(t_sf + 16, ones);
    tmem_st16(t_sf + 32, ones);
    tmem_st_wait();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                          // both CTAs' operands, scales and barriers are in place
  tc_fence_after();

  long long cycles = 0;
  if (rank == 0 && warp == 0) {
    const bool issuer = elect_one();
    const uint32_t idesc = instr_desc(256, instr_n);
    const uint64_t adesc = operand_desc(smem_u32(operands)), bdesc = operand_desc(smem_u32(operands) + 16384u);
    const uint32_t sfa_t = tmem_base + 256u, sfb_t = sfa_t + 16u;
    const long long t0 = clock64();
    for (int s = 0; s < stages; ++s) {
      if (issuer) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          tc_mma_nvf4_pair(tmem_base, adesc + 2u * j, bdesc + 2u * j, idesc, sfa_t + 4 * j, sfb_t + 8 * j, (s | j) ? 1u : 0u);
      }
      __syncwarp();
    }
    if (issuer) tc_commit_pair(done_bar);      // arrives on both CTAs' barriers once every instruction above is done
    cycles = -t0;
  }
  // every thread of both CTAs waits (bounded) for the completion before tensor memory is freed
  bool timed_out = false;
  {
    const unsigned long long w0 = global_timer_ns();
    while (!mbar_try_wait(done_bar, 0)) {
      if (global_timer_ns() - w0 > kPeakWaitLimitNs) { timed_out = true; break; }
    }
  }
  if (rank == 0 && threadIdx.x == 0) {
    cycles += clock64();
    out[3 * (blockIdx.x >> 1) + 0] = cycles;
    out[3 * (blockIdx.x >> 1) + 1] = 4ll * stages;
    out[3 * (blockIdx.x >> 1) + 2] = timed_out ? 1 : 0;
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

// Runs the measurement on the current device: `stages` groups of four 256 x instr_n x 64 instructions per CTA pair
// (1 <= stages <= 2^20; instr_n a multiple of 32 up to 256), one pair per two multiprocessors.  out (device): 3 x (sm_count / 2) 64-bit integers per
// pair: cycles, instructions, timed-out flag.  *pairs_out (host) receives the number of pairs launched.
extern "C" int nvfp4_microbench_mma_peak(int stages, int instr_n, int64_t* out, size_t out_bytes, int* pairs_out,
                                         void* cuda_stream) {
  if (!out || !pairs_out) return NVFP4_ERR_NULL;
  if (stages < 1 || stages > (1 << 20)) return NVFP4_ERR_SHAPE;
  if (instr_n < 32 || instr_n > 256 || instr_n % 32 != 0) return NVFP4_ERR_SHAPE;   // the resident B tile has 256 rows
  if (reinterpret_cast<uintptr_t>(out) & 7u) return NVFP4_ERR_ALIGN;
  if (int st = check_arch()) return st;
  const int pairs = sm_count() / 2;
  if (out_bytes < (size_t)pairs * 3 * sizeof(int64_t)) return NVFP4_ERR_WORKSPACE;
  *pairs_out = pairs;
  mma_peak_kernel<<<2 * pairs, kPeakThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(stages, instr_n, out);
  return cudaGetLastError() == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}
