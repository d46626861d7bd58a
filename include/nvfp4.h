/*
 * nvfp4.h -- C ABI of the B200 (sm_100a) NVFP4 quantize-then-GEMM library.
 *
 * The library implements the quantized linear layer of "FP4 All the Way: Fully
 * Quantized Training of LLMs": every operand of the three training GEMMs
 * (Eq. 1-3) is cut into blocks of 16 values along the contraction axis, each
 * block gets an E4M3 scale, and values become 4-bit E2M1 codes (Section 3),
 * rounded to nearest in the forward pass and stochastically in the backward and
 * update passes (Eq. 4-6).
 *
 * Conventions for every entry point
 *   - Returns an nvfp4_status (int).  Never throws, never exits the process.
 *   - Pointers are DEVICE pointers unless the comment says "host".  The caller
 *     owns every buffer; the library allocates no device memory (scratch comes
 *     from the caller's workspace).
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) and is asynchronous; there is no internal
 *     synchronisation.  Argument errors are detected on the host before any
 *     launch; launch failures map to NVFP4_ERR_CUDA.
 *   - Tensors are row-major.  M = tokens, K = in-features, N = out-features.
 *   - Packed codes: element 2i sits in bits 0-3 and element 2i+1 in bits 4-7 of
 *     byte i.  A code is sign<<3 | exponent(2)<<1 | mantissa(1).
 *   - "Quantized shape" (Rq, Kq): for transposed == 0 it is (rows, cols); for
 *     transposed == 1 it is (cols, rows).  Blocks always run along Kq, codes are
 *     stored [Rq, Kq/2] and scales [Rq, Kq/16], so Kq is the contiguous
 *     (contraction) axis of the output.  Kq must be a multiple of 16.
 */
#ifndef NVFP4_H
#define NVFP4_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define NVFP4_API __attribute__((visibility("default")))
#else
#define NVFP4_API
#endif

typedef enum {
  NVFP4_OK = 0,
  NVFP4_ERR_NULL = 1,       /* a required pointer is NULL */
  NVFP4_ERR_SHAPE = 2,      /* non-positive size, contraction length not a multiple of 16, ld too small */
  NVFP4_ERR_ALIGN = 3,      /* a base pointer or leading dimension breaks the alignment rule below */
  NVFP4_ERR_ENUM = 4,       /* unknown dtype / rounding mode / layout / flag */
  NVFP4_ERR_WORKSPACE = 5,  /* workspace missing or smaller than nvfp4_linear_workspace_bytes */
  NVFP4_ERR_ARCH = 6,       /* current device is not compute capability 10.x */
  NVFP4_ERR_CUDA = 7        /* a CUDA runtime/driver call or a launch failed */
} nvfp4_status;

typedef enum { NVFP4_BF16 = 0, NVFP4_FP32 = 1 } nvfp4_dtype;
typedef enum { NVFP4_RTN = 0, NVFP4_SR = 1 } nvfp4_round_mode;
typedef enum { NVFP4_SF_LINEAR = 0, NVFP4_SF_SWIZZLED_128x4 = 1 } nvfp4_sf_layout;
typedef enum { NVFP4_G_NONE = 0, NVFP4_G_AMAX = 1, NVFP4_G_GIVEN = 2 } nvfp4_gscale_mode;
typedef enum { NVFP4_LINEAR_FWD = 0, NVFP4_LINEAR_BWD_DX = 1, NVFP4_LINEAR_BWD_DW = 2 } nvfp4_linear_kind;

/* Rounding of one operand, chosen per call (Eq. 4-6 fix the paper's choice per
 * site; any site may be overridden, as the paper's per-site ablation does).
 * For NVFP4_SR (Section 1: round to one of the two neighbouring grid values with
 * probability given by the distance) an element whose scaled magnitude sits at
 * fraction f of its grid step is rounded up iff floor(f * 2^16) + r >= 2^16 for
 * a 16-bit random integer r.  Block B (B = r*(Kq/16) + kb in the quantized
 * shape) draws one Philox4x32-10 output with key = seed and counter =
 * (B lo, B hi, offset lo, offset hi); output word q (bytes b0..b3, b0 lowest)
 * serves elements 4q..4q+3: element 4q gets r = b2:b0 (b2 the high byte),
 * element 4q+1 the same 16 bits in mirrored order, element 4q+2 gets b3:b1 and
 * element 4q+3 those mirrored.  The same (seed, offset) reproduces the same
 * codes; distinct offsets give independent streams. */
typedef struct {
  int32_t mode;      /* nvfp4_round_mode */
  int32_t reserved;  /* must be 0 */
  uint64_t seed;
  uint64_t offset;
} nvfp4_rounding;

/* Text for a status code (host pointer to a static string). */
NVFP4_API const char* nvfp4_status_string(int status);

/* Bytes of a scale buffer for a quantized shape (Rq, Kq): linear = Rq*Kq/16;
 * swizzled = ceil(Rq/128)*ceil(Kq/64)*512.  Returns 0 on bad arguments. */
NVFP4_API size_t nvfp4_sf_bytes(int64_t Rq, int64_t Kq, int sf_layout);

/*
 * Quantizer Q(x) of Section 3 / Eq. 4-6: per block of 16 along Kq,
 *   scale  = E4M3( amax * ((1/6)/g) )   nearest-even, saturating at 448, sign unused
 *   code_j = E2M1( min(|x_j| / (decode(scale)*g), 6) )   RtN (ties to even) or SR,
 * sign kept.  g is *global_scale (NULL => 1.0f), a per-tensor fp32 factor.
 *
 *   x            [rows, cols] of `dtype`, leading dimension ld (elements, >= cols)
 *   transposed   0: blocks along cols.  1: blocks along rows and the output is
 *                stored transposed (quantized shape (cols, rows))
 *   codes        Rq*Kq/2 bytes;  scales  nvfp4_sf_bytes(Rq, Kq, sf_layout) bytes.
 *                In the swizzled layout scale (r, kb) lives at
 *                ((r/128)*ceil(Kq/64) + kb/4)*512 + (r%32)*16 + ((r%128)/32)*4 + kb%4
 *                and padding bytes are written as 0.
 * Alignment: x, codes, scales 16-byte aligned; ld a multiple of 8 elements.
 * Errors: NULL pointers, Kq % 16 != 0, ld < cols, bad enums, misalignment.
 */
NVFP4_API int nvfp4_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                   int transposed, const float* global_scale, const nvfp4_rounding* rounding /* host */,
                   uint8_t* codes, uint8_t* scales, int sf_layout, void* cuda_stream);

/*
 * Both quantizations of one tensor from a single read: Q(x) with blocks along cols (as
 * nvfp4_quantize with transposed == 0, rounding_row) and Q(x^T) with blocks along rows (as
 * transposed == 1, rounding_t).  Eq. 4-6 need every operand in both orientations (Q(dY) in Eq. 5 and
 * Q(dY^T) in Eq. 6, Q(X) in Eq. 4 and Q(X^T) in Eq. 6, Q(W) in Eq. 4 and Q(W^T) in Eq. 5); each
 * output is bit-identical to what the corresponding nvfp4_quantize call writes.
 * rows and cols must both be multiples of 16.  codes_row: rows*cols/2 bytes, scales_row:
 * nvfp4_sf_bytes(rows, cols, sf_layout); codes_t: cols*rows/2 bytes, scales_t:
 * nvfp4_sf_bytes(cols, rows, sf_layout).  bf16 tensors whose rows and cols are multiples of 32 take
 * the fused kernel (one read, 3.125 bytes of traffic per element); others run the two
 * single-output kernels.  Alignment and errors as for nvfp4_quantize.
 */
NVFP4_API int nvfp4_quantize_dual(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                        const float* global_scale,
                        const nvfp4_rounding* rounding_row /* host */, uint8_t* codes_row, uint8_t* scales_row,
                        const nvfp4_rounding* rounding_t /* host */, uint8_t* codes_t, uint8_t* scales_t,
                        int sf_layout, void* cuda_stream);

/*
 * Quantization-noise monitor (Section 4): for a tensor and the quantization nvfp4_quantize (or
 * nvfp4_quantize_dual) made of it with the same `transposed`, `global_scale` and `sf_layout`,
 *   sums[0] = sum (Q(x) - x)^2     sums[1] = sum x^2          (device doubles, overwritten)
 * so that the paper's gradient-to-noise ratio ||x|| / (sigma_q sqrt(d)) = sqrt(sums[1] / sums[0]);
 * the paper leaves FP4 for higher precision once this falls below sqrt(3).  One extra read of x and
 * of the codes; sums is 8-byte aligned; other arguments and errors as for nvfp4_quantize.
 */
NVFP4_API int nvfp4_quantization_noise(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int transposed,
                             const float* global_scale, const uint8_t* codes, const uint8_t* scales,
                             int sf_layout, double* sums, void* cuda_stream);

/* Per-tensor scale g = max|x| / (6*448), or 1.0f for an all-zero tensor, written
 * to *global_scale_out (device).  The paper defines only the block scale; this
 * optional factor keeps small-magnitude gradients inside the E4M3 scale range.
 * Non-finite inputs propagate: a tensor that holds a NaN gets g = NaN, one that
 * holds an infinity (and no NaN) gets g = +Inf, and every element of a product
 * computed with such a scale (nvfp4_gemm, nvfp4_linear_*) is NaN, so a diverged
 * step shows in the results.  (With g supplied by the caller, or none, the codes
 * of a block that holds a non-finite value are unspecified.) */
NVFP4_API int nvfp4_tensor_amax_scale(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                            float* global_scale_out, void* cuda_stream);

/*
 * Block-scaled GEMM (the contraction of Eq. 1-3 on quantized operands):
 *   D[m,n] = (gA*gB) * sum_kb sA[m,kb]*sB[n,kb] * sum_{k in kb} a[m,k]*b[n,k]
 * A is [M,K] and B is [N,K], both K-major packed codes with scales in the
 * swizzled layout; a_g / b_g are device fp32 per-tensor scales (NULL => 1).
 * D is [M,N] row-major, leading dimension ldd (elements), fp32 or bf16;
 * accumulation is fp32.  K % 16 == 0; code rows are K/2 bytes (so K % 32 == 0
 * is required for the 16-byte row pitch of the tiled copies); ldd*sizeof(D)
 * a multiple of 16; all base pointers 16-byte aligned.
 */
NVFP4_API int nvfp4_gemm(const uint8_t* a_codes, const uint8_t* a_sf, const float* a_g,
               const uint8_t* b_codes, const uint8_t* b_sf, const float* b_g,
               int64_t M, int64_t N, int64_t K,
               void* d, int d_dtype, int64_t ldd, void* cuda_stream);

/*
 * The same product with the next quantization fused into the epilogue: instead of D, the call writes
 * Q(D) with blocks of 16 along N (as nvfp4_quantize of the fp32 D with transposed == 0 would: codes
 * [M, N/2], scales for the quantized shape (M, N) in `sf_layout`), so that a consumer which would
 * quantize D along N anyway (the next layer's Q(X) of Eq. 4) never sees a high-precision copy.
 * out_global_scale is the per-tensor scale of the OUTPUT (device, NULL => 1; it has to be known before
 * the product runs: from the previous step, or a bound); rounding (host) as for nvfp4_quantize, the
 * block index for SR being m*(N/16) + n/16.  The result equals nvfp4_quantize applied to the fp32
 * output of nvfp4_gemm bit for bit.  N % 32 == 0, K % 32 == 0; alignment as for nvfp4_gemm.
 */
NVFP4_API int nvfp4_gemm_quantized(const uint8_t* a_codes, const uint8_t* a_sf, const float* a_g,
                         const uint8_t* b_codes, const uint8_t* b_sf, const float* b_g,
                         int64_t M, int64_t N, int64_t K,
                         const float* out_global_scale, const nvfp4_rounding* rounding /* host */,
                         uint8_t* out_codes, uint8_t* out_scales, int sf_layout, void* cuda_stream);

/* TEST HOOK, not part of the supported surface: forces the GEMM kernel variant so
 * that the tests can compare the library's independent kernel implementations
 * with each other.  0 restores the automatic choice; 128 / 256 select the
 * single-CTA kernel with a 128 x {128,256} tile; 2128 / 2192 / 2256 select the
 * CTA-pair kernel with a 256 x {128,192,256} tile.  Process-wide and
 * unsynchronised: do not call it while another thread is inside nvfp4_gemm. */
NVFP4_API int nvfp4_gemm_set_tile_n(int bn);

/* Scratch bytes nvfp4_linear_* needs for a layer of shape (M, N, K);
 * `which` is an nvfp4_linear_kind.  Returns 0 for a layer the calls reject
 * (non-positive size, contraction length not a multiple of 32, or a contiguous
 * axis of an operand or of the output not a multiple of 8). */
NVFP4_API size_t nvfp4_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int which);

/*
 * Forward pass, Eq. 1 / Eq. 4:  Y[M,N] = Q(X)[M,K] . Q(W)[N,K]^T, blocks along K.
 * rx / rw (host) choose the rounding (the paper: RtN for both).
 * gscale_mode: NVFP4_G_NONE  g = 1 for both operands;
 *              NVFP4_G_AMAX  g computed here from each operand's amax (one extra read);
 *              NVFP4_G_GIVEN gx / gw are device pointers supplied by the caller.
 * X, W of `dtype` (dense, ld = K); Y of y_dtype (dense, ld = N).
 * workspace: device scratch of at least nvfp4_linear_workspace_bytes(M,N,K,FWD),
 * 256-byte aligned; its contents are undefined afterwards.
 */
NVFP4_API int nvfp4_linear_fwd(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                     int gscale_mode, const float* gx, const float* gw,
                     const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                     void* Y, int y_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Backward pass, Eq. 2 / Eq. 5:  dX[M,K] = Q(dY)[M,N] . Q(W^T)[K,N]^T, blocks
 * along N: dY is quantized along its rows' contiguous axis, W is quantized
 * transposed.  The paper: SR for dY, RtN for W^T. */
NVFP4_API int nvfp4_linear_bwd_dx(const void* dY, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                        int gscale_mode, const float* gdy, const float* gw,
                        const nvfp4_rounding* rdy, const nvfp4_rounding* rw,
                        void* dX, int dx_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Update pass (weight gradient), Eq. 3 / Eq. 6:  dW[N,K] = Q(dY^T)[N,M] . Q(X^T)[K,M]^T,
 * blocks along the token axis M: both operands are quantized transposed.
 * The paper: SR for both. */
NVFP4_API int nvfp4_linear_bwd_dw(const void* dY, const void* X, int dtype, int64_t M, int64_t N, int64_t K,
                        int gscale_mode, const float* gdy, const float* gx,
                        const nvfp4_rounding* rdy, const nvfp4_rounding* rx,
                        void* dW, int dw_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Producer fusion along a chain of layers (Eq. 1 / Eq. 4 applied twice; in Section 5's model the position of
 * the SwiGLU output feeding the down projection): the quantization Q(.) that the NEXT layer would apply to its
 * input is done in the epilogue of the GEMM that produces it, so the intermediate never exists in bf16 or fp32.
 *
 * nvfp4_linear_fwd_qout: as nvfp4_linear_fwd, but instead of Y it writes Q(Y) with blocks of 16 along N
 *   (y_codes [M, N/2], y_scales for the quantized shape (M, N) in `sf_layout`), using the per-tensor scale *gy
 *   of the OUTPUT (device, NULL => 1; it has to be known before the product runs, e.g. carried over from the
 *   previous step) and rounding ry (host).  Bit for bit what nvfp4_quantize makes of nvfp4_linear_fwd's fp32 Y.
 *   N % 32 == 0.  Workspace as for nvfp4_linear_fwd.
 * nvfp4_linear_fwd_qin: as nvfp4_linear_fwd for an input that is already quantized along K: x_codes [M, K/2],
 *   x_scales in the swizzled layout, per-tensor scale *gx (device, NULL => 1), e.g. the output of
 *   nvfp4_linear_fwd_qout with sf_layout = NVFP4_SF_SWIZZLED_128x4.  gscale_mode / gw / rw apply to W only.
 *   Workspace: nvfp4_linear_workspace_bytes(M, N, K, NVFP4_LINEAR_FWD).
 */
NVFP4_API int nvfp4_linear_fwd_qout(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                          int gscale_mode, const float* gx, const float* gw,
                          const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                          const float* gy, const nvfp4_rounding* ry /* host */,
                          uint8_t* y_codes, uint8_t* y_scales, int sf_layout,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
NVFP4_API int nvfp4_linear_fwd_qin(const uint8_t* x_codes, const uint8_t* x_scales, const float* gx,
                         const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                         int gscale_mode, const float* gw, const nvfp4_rounding* rw,
                         void* Y, int y_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The layer of Eq. 1-6 with every tensor read once per pass (fused producers).
 *
 * Eq. 4-6 use X, W and dY in both orientations.  nvfp4_linear_fwd_save computes Y as
 * nvfp4_linear_fwd does and, from the same reads of X and W, also writes Q(X^T) (rounding rxt; the
 * paper: SR, Eq. 6) and Q(W^T) (rounding rwt; the paper: RtN, Eq. 5) with their per-tensor scales
 * into `saved`.  nvfp4_linear_bwd_saved then needs only dY: it quantizes it both ways from one read
 * (rdy for Q(dY) of Eq. 5, rdyt for Q(dY^T) of Eq. 6) and runs both GEMMs, dX[M,K] and dW[N,K].
 * nvfp4_linear_bwd is the same backward + update pass without saved state (it quantizes W^T and X^T
 * itself).  With equal rounding arguments all results equal those of nvfp4_linear_fwd /
 * nvfp4_linear_bwd_dx / nvfp4_linear_bwd_dw bit for bit.
 *
 * M, N, K must be multiples of 32.  `saved`: nvfp4_linear_saved_bytes(M,N,K) bytes, 256-byte
 * aligned, owned by the caller, written by fwd_save and only read by bwd_saved (which must be given
 * the same gscale_mode).  workspace: nvfp4_linear_fused_workspace_bytes(M,N,K,which) bytes, 256-byte
 * aligned, contents undefined afterwards.  gscale_mode as in nvfp4_linear_fwd.
 */
typedef enum { NVFP4_FUSED_FWD_SAVE = 0, NVFP4_FUSED_BWD_SAVED = 1, NVFP4_FUSED_BWD = 2 } nvfp4_fused_kind;
NVFP4_API size_t nvfp4_linear_saved_bytes(int64_t M, int64_t N, int64_t K);
NVFP4_API size_t nvfp4_linear_fused_workspace_bytes(int64_t M, int64_t N, int64_t K, int which);
NVFP4_API int nvfp4_linear_fwd_save(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                          int gscale_mode, const float* gx, const float* gw,
                          const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                          const nvfp4_rounding* rxt, const nvfp4_rounding* rwt,
                          void* Y, int y_dtype, void* saved, size_t saved_bytes,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
NVFP4_API int nvfp4_linear_bwd_saved(const void* dY, int dtype, int64_t M, int64_t N, int64_t K,
                           int gscale_mode, const float* gdy,
                           const nvfp4_rounding* rdy, const nvfp4_rounding* rdyt,
                           const void* saved, size_t saved_bytes,
                           void* dX, int dx_dtype, void* dW, int dw_dtype,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);
NVFP4_API int nvfp4_linear_bwd(const void* dY, const void* W, const void* X, int dtype, int64_t M, int64_t N, int64_t K,
                     int gscale_mode, const float* gdy, const float* gw, const float* gx,
                     const nvfp4_rounding* rdy, const nvfp4_rounding* rdyt,
                     const nvfp4_rounding* rwt, const nvfp4_rounding* rxt,
                     void* dX, int dx_dtype, void* dW, int dw_dtype,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * MXFP4 (Section 3, Table 1: the format the paper compares NVFP4 with): the same E2M1 elements in
 * blocks of 32 along Kq with an E8M0 (power-of-two) scale, scale = amax * ((1/6)/g) rounded UP to a
 * power of two, so that no element exceeds 6.  Codes as for NVFP4; scales one byte per 32 elements,
 * linear [Rq, Kq/32] or in the same 128-row x 4-block tiles of 512 bytes (a tile then covers 128
 * values); nvfp4_sf_bytes_mx gives the size.  The random integers of SR belong to groups of 16
 * elements exactly as for NVFP4 (group index r*(Kq/16) + k/16).  Kq % 32 == 0.
 * nvfp4_quantize_mx: transposed == 1 (bf16 only) quantizes along the rows straight from the source
 * tile (no transpose pass, `workspace` unused and may be NULL); only a tensor with more than 2^24 rows
 * goes through a transpose into `workspace` (rows*cols*2 bytes, 16-byte aligned) and is rejected with
 * NVFP4_ERR_WORKSPACE without one.
 * nvfp4_gemm_mx: as nvfp4_gemm on MXFP4 operands (tcgen05 kind::mxf4, scale_vec::2X).
 */
NVFP4_API size_t nvfp4_sf_bytes_mx(int64_t Rq, int64_t Kq, int sf_layout);
NVFP4_API int nvfp4_quantize_mx(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int transposed,
                      const float* global_scale, const nvfp4_rounding* rounding /* host */,
                      uint8_t* codes, uint8_t* scales, int sf_layout,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);
NVFP4_API int nvfp4_gemm_mx(const uint8_t* a_codes, const uint8_t* a_sf, const float* a_g,
                  const uint8_t* b_codes, const uint8_t* b_sf, const float* b_g,
                  int64_t M, int64_t N, int64_t K, void* d, int d_dtype, int64_t ldd, void* cuda_stream);

/*
 * Quantization-aware fine-tuning phase (Section 5): the forward pass stays in NVFP4
 * (nvfp4_linear_fwd), the backward and update products run in BF16.
 *
 * nvfp4_gemm_bf16: D[M,N] = A[M,K] . B[N,K]^T for dense bf16 A and B (both contiguous along K),
 * fp32 accumulation, D fp32 or bf16 with leading dimension ldd.  K % 16 == 0, pointers 16-byte
 * aligned, ldd*sizeof(D) a multiple of 16.
 * nvfp4_gemm_bf16_ex: the same product for operands stored the other way round: a_mn_major == 1 means A is
 * given as a dense [K, M] array (its output axis contiguous), b_mn_major == 1 means B is given as [K, N]; the
 * tensor cores read them in place (no transposed copy).  M % 8 == 0 / N % 8 == 0 for such an operand.
 * Combinations: (0,0), (0,1), (1,1) -- the three shapes the products of Eq. 1-3 take.
 * nvfp4_transpose_bf16: out[cols, rows] = x[rows, cols]^T (rows, cols multiples of 8; out dense).
 * nvfp4_linear_bwd_bf16: dX[M,K] = dY . W and dW[N,K] = dY^T . X from bf16 dY[M,N], W[N,K], X[M,K]
 * (all dense), each read as it is stored.  `workspace` is unused (nvfp4_linear_bwd_bf16_workspace_bytes
 * returns 0; NULL is accepted).  M, N, K multiples of 16.
 */
NVFP4_API int nvfp4_gemm_bf16(const void* a, const void* b, int64_t M, int64_t N, int64_t K,
                    void* d, int d_dtype, int64_t ldd, void* cuda_stream);
NVFP4_API int nvfp4_gemm_bf16_ex(const void* a, int a_mn_major, const void* b, int b_mn_major, int64_t M, int64_t N, int64_t K,
                       void* d, int d_dtype, int64_t ldd, void* cuda_stream);
NVFP4_API int nvfp4_transpose_bf16(const void* x, int64_t rows, int64_t cols, int64_t ld, void* out, void* cuda_stream);
NVFP4_API size_t nvfp4_linear_bwd_bf16_workspace_bytes(int64_t M, int64_t N, int64_t K);
NVFP4_API int nvfp4_linear_bwd_bf16(const void* dY, const void* W, const void* X, int64_t M, int64_t N, int64_t K,
                          void* dX, int dx_dtype, void* dW, int dw_dtype,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * nvfp4_linear_fwd without a caller-supplied workspace and without any device-memory
 * allocation (the paper has no counterpart; this is a library convenience).
 *
 * It is meant for callers that cannot obtain scratch memory at the call site: a host
 * program whose framework reserved the whole device for its own memory pool at start-up
 * (so a cudaMalloc would fail, or would have to be carved out of that pool through an API
 * the caller does not control), or a latency-critical section in which the implicit
 * device-wide synchronisation of cudaMalloc/cudaFree is not acceptable.
 *
 * The scratch lives in a fixed array of NVFP4_STATIC_WORKSPACE_BYTES in the library's device
 * image; every GPU on which the library's kernels are loaded holds that much memory until the
 * process exits.  Arguments and results are those of nvfp4_linear_fwd (X, W, Y are still the
 * caller's buffers).  A layer whose nvfp4_linear_workspace_bytes(M, N, K, NVFP4_LINEAR_FWD)
 * exceeds NVFP4_STATIC_WORKSPACE_BYTES is rejected with NVFP4_ERR_WORKSPACE before any launch.
 *
 * The first call on each device looks up the array's device address (once per device, with
 * that device current); make that first call outside any stream capture.  Every call on a
 * device uses the same array and finds the previous call's contents in it; each call rewrites
 * all bytes it later reads, so nothing needs clearing by the caller, but two calls that can
 * overlap on the GPU (different streams, or different host threads) race on it: serialise them.
 * No cudaMalloc, cudaFree or allocating library routine is called.
 */
#define NVFP4_STATIC_WORKSPACE_BYTES (8u << 20)
NVFP4_API int nvfp4_linear_fwd_static(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                      int gscale_mode, const float* gx, const float* gw,
                                      const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                                      void* Y, int y_dtype, void* cuda_stream);

/*
 * Measurement aid (the paper has no counterpart): the issue rate of the tensor-core instruction the
 * GEMM is built on, tcgen05.mma kind::mxf4nvf4 on a CTA pair (256 x instr_n x 64 per instruction; instr_n
 * a multiple of 32 up to 256, the GEMM uses 256), issued
 * back to back on operands resident in shared memory and scales resident in tensor memory, one CTA
 * pair per two multiprocessors, `stages` groups of four instructions each (1 .. 2^20).  No loads and
 * no epilogue: it gives the ceiling the tensor pipe sets at the clock the run holds, the denominator
 * of the GEMM's "fraction of issue peak".  out (device, 8-byte aligned, out_bytes >= 24 per pair)
 * receives per pair {cycles of the leader CTA's clock from first issue to completion, instructions
 * issued, 1 if the bounded wait for completion ran out}; *pairs_out (host) the number of pairs.
 * FLOP per instruction: 2 * 256 * instr_n * 64.
 */
NVFP4_API int nvfp4_microbench_mma_peak(int stages, int instr_n, int64_t* out, size_t out_bytes,
                                        int* pairs_out /* host */, void* cuda_stream);

/* Reads and clears the device-side error word of the current device (host
 * out-pointer; synchronises the device).  Non-zero means a kernel gave up on a
 * bounded wait and its output is invalid; bits 0-7 identify the wait site. */
NVFP4_API int nvfp4_device_error_word(uint32_t* host_out);

#ifdef __cplusplus
}
#endif
#endif
