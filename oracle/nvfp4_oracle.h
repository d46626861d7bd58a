/*
 * NVFP4 CPU oracle -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow, obviously-correct restatement of the paper's quantizer
 * (Section 3: E2M1 elements, blocks of 16, one E4M3 scale per block; Section 1
 * and Eq. 4-6: round-to-nearest and stochastic rounding) and of the three
 * linear-layer products (Eq. 1-3) as dequantize-then-matmul.  It shares no code
 * with the CUDA library and must never be linked, imported or called by it.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything is host memory.  All functions are single IEEE-754 binary32
 * operations exactly as written (compile with -ffp-contract=off, no fast-math).
 *
 * Parity status: every function below is pinned by tests that do not call it
 * to produce their own expectations (format definitions, enumeration, closed
 * forms, published known-answer vectors, a library cast).  The paper prints no
 * worked numeric example, so none of the pins is a value printed by the paper.
 */
#ifndef NVFP4_ORACLE_H
#define NVFP4_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Section 3: E2M1 = 1 sign, 2 exponent (bias 1), 1 mantissa bit.  `code` is the
 * 4-bit pattern s|ee|m in the low nibble. */
float nvfp4o_e2m1_decode(uint8_t code);

/* Section 3 (block scales are stored in E4M3), sign bit unused: unsigned E4M3,
 * bias 7, 3 mantissa bits, subnormals, largest finite 448 (0x7E), no infinity.
 * Encode rounds to nearest, ties to the even mantissa, and saturates at 448. */
uint8_t nvfp4o_e4m3_encode(float v);
float nvfp4o_e4m3_decode(uint8_t code);

/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw 2011). */
void nvfp4o_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4]);

/* The four 16-bit random integers that one Philox output word gives to four
 * consecutive elements: elements 0,1 share bytes 0 (low half) and 2 (high half) of
 * the word, elements 2,3 share bytes 1 and 3; the odd element of each pair reads
 * its 16 bits in reversed order. */
void nvfp4o_word_random_u16(uint32_t w, uint16_t out[4]);

/* The 16 random integers of block B: counter (B_lo, B_hi, offset_lo, offset_hi),
 * key (seed_lo, seed_hi); output word q serves elements 4q..4q+3. */
void nvfp4o_block_random_u16(uint64_t seed, uint64_t offset, uint64_t block, uint16_t out[16]);

/* Section 1: RtN maps y in [0,6] to the closest grid magnitude (ties to the
 * code with an even mantissa bit); SR picks one of the two neighbours with
 * probability given by the distance, using a 16-bit random integer r: with f the
 * position of y inside its grid step, it rounds up iff floor(f*2^16) + r >= 2^16.
 * Both return the 3-bit magnitude code. */
uint8_t nvfp4o_round_rtn(float y);
uint8_t nvfp4o_round_sr(float y, uint16_t r16);
/* nvfp4o_round_sr of one value for n random integers (a loop over the call above). */
void nvfp4o_round_sr_many(float y, const uint16_t* r16, int64_t n, uint8_t* out);

/* Quantize a logical [Rq, Kq] fp32 tensor (row stride Kq) in blocks of 16 along
 * Kq.  mode 0 = RtN, 1 = SR.  codes: Rq*Kq/2 bytes (element 2i in the low
 * nibble of byte i); scales: Rq*Kq/16 bytes, linear [Rq, Kq/16].  Kq % 16 == 0.
 * g is the per-tensor scale (1.0f = none). */
void nvfp4o_quantize(const float* x, int64_t Rq, int64_t Kq, float g, int mode,
                     uint64_t seed, uint64_t offset,
                     uint8_t* codes, uint8_t* scales, int nthreads);

/* The same for rows first_row .. first_row+Rq-1 of a taller tensor: x points at the slice, and
 * the block of slice row r, block kb draws its random integers as block (first_row + r)*(Kq/16) + kb.
 * Lets a test check a slice of a tensor too large to quantize whole on the host. */
void nvfp4o_quantize_rows(const float* x, int64_t Rq, int64_t Kq, float g, int mode,
                          uint64_t seed, uint64_t offset, int64_t first_row,
                          uint8_t* codes, uint8_t* scales, int nthreads);

/* MXFP4 (Section 3, Table 1): E2M1 elements in blocks of 32 along Kq with an E8M0 scale.
 * e8m0 code c means 2^(c-127); encode_up gives the smallest power of two >= v (0 for v <= 0, which
 * flushes the block).  Scale = encode_up(amax * ((1/6)/g)); elements as for NVFP4; the random
 * integers of SR belong to groups of 16 elements, group index (first_row+r)*(Kq/16) + k/16.
 * codes: Rq*Kq/2 bytes; scales: linear [Rq, Kq/32].  Kq % 32 == 0. */
uint8_t nvfp4o_e8m0_encode_up(float v);
float nvfp4o_e8m0_decode(uint8_t code);
void nvfp4o_quantize_mx_rows(const float* x, int64_t Rq, int64_t Kq, float g, int mode,
                             uint64_t seed, uint64_t offset, int64_t first_row,
                             uint8_t* codes, uint8_t* scales, int nthreads);
void nvfp4o_dequantize_mx(const uint8_t* codes, const uint8_t* scales, float g, int64_t Rq, int64_t Kq, float* out);
void nvfp4o_gemm_mx(const uint8_t* a_codes, const uint8_t* a_sf, float ga,
                    const uint8_t* b_codes, const uint8_t* b_sf, float gb,
                    int64_t M, int64_t N, int64_t K, float* D, float* T, int nthreads);

/* Transposed quantization of x[rows, cols]: by definition nvfp4o_quantize
 * applied to the materialised transpose (Rq = cols, Kq = rows). */
void nvfp4o_quantize_transposed(const float* x, int64_t rows, int64_t cols, float g, int mode,
                                uint64_t seed, uint64_t offset,
                                uint8_t* codes, uint8_t* scales, int nthreads);

/* out[r, k] = decode(code) * decode(scale) * g  (exact in fp32 when g is a
 * power of two; otherwise one rounding per factor as written). */
void nvfp4o_dequantize(const uint8_t* codes, const uint8_t* scales, float g,
                       int64_t Rq, int64_t Kq, float* out);

/* Section 4 (gradient-to-noise ratio): out[0] = sum over the tensor of (Q(x) - x)^2, out[1] = sum
 * of x^2, in double; x in the quantized orientation [Rq, Kq], linear scales.  The paper's ratio
 * ||x|| / (sigma_q sqrt(d)) is sqrt(out[1]/out[0]); it switches precision when that falls below sqrt(3). */
void nvfp4o_noise_sums(const float* x, const uint8_t* codes, const uint8_t* scales, float g,
                       int64_t Rq, int64_t Kq, double out[2]);

/* QAF phase (Section 5: forward FP4, backward and update BF16): D = A[M,K] . B[N,K]^T on plain
 * (unquantized) operands, double accumulation, rounded to fp32; T = sum |a_k b_k|. */
void nvfp4o_matmul_nt(const float* A, const float* B, int64_t M, int64_t N, int64_t K, float* D, float* T, int nthreads);

/* g = amax / (6*448) in one fp32 division, 1.0f when amax == 0.  Non-finite inputs propagate:
 * NaN if any element is NaN, else +Inf if any element is infinite. */
float nvfp4o_tensor_amax_scale(const float* x, int64_t n);

/* D[i,j] = (gA*gB) * sum_kb sA[i,kb]*sB[j,kb] * sum_{k in kb} a[i,k]*b[j,k]
 * with A[M,K], B[N,K] both K-major, linear scales; double accumulation, result
 * rounded to fp32.  T[i,j] = the same sum over absolute values (the tolerance
 * base).  D and/or T may be NULL. */
void nvfp4o_gemm(const uint8_t* a_codes, const uint8_t* a_sf, float ga,
                 const uint8_t* b_codes, const uint8_t* b_sf, float gb,
                 int64_t M, int64_t N, int64_t K, float* D, float* T, int nthreads);

/* Same contraction with every partial sum kept in fp32 (shows how far plain
 * fp32 accumulation sits from the double result). */
void nvfp4o_gemm_f32acc(const uint8_t* a_codes, const uint8_t* a_sf, float ga,
                        const uint8_t* b_codes, const uint8_t* b_sf, float gb,
                        int64_t M, int64_t N, int64_t K, float* D, int nthreads);

/* The double-accumulated result at n sampled (i,j) positions only. */
void nvfp4o_gemm_sampled(const uint8_t* a_codes, const uint8_t* a_sf, float ga,
                         const uint8_t* b_codes, const uint8_t* b_sf, float gb,
                         int64_t M, int64_t N, int64_t K,
                         const int64_t* ii, const int64_t* jj, int64_t n,
                         float* D, float* T, int nthreads);

/* Scale-factor storage in 128-row x 4-block tiles of 512 bytes (the layout the
 * Blackwell block-scaled MMA consumes): byte offset of scale (r, kb) for a
 * tensor with n_kb blocks per row, total padded size, and a linear->tiled copy
 * that zero-fills the padding. */
int64_t nvfp4o_sf_swizzled_offset(int64_t r, int64_t kb, int64_t n_kb);
int64_t nvfp4o_sf_swizzled_bytes(int64_t Rq, int64_t n_kb);
void nvfp4o_sf_swizzle(const uint8_t* linear, int64_t Rq, int64_t n_kb, uint8_t* out);

#ifdef __cplusplus
}
#endif
#endif
