// The quantized linear layer of Eq. 1-6 with every tensor read once per pass.
//
// Eq. 4-6 use each of X, W and dY in two orientations.  nvfp4_linear_fwd_save quantizes X and W
// both ways while it has them (Q(X), Q(W) feed Eq. 4 at once; Q(X^T), Q(W^T) are kept for the
// backward and update passes); nvfp4_linear_bwd_saved quantizes dY both ways from one read and runs
// the GEMMs of Eq. 5 and Eq. 6.  nvfp4_linear_bwd does the same without saved state (it quantizes
// W^T and X^T itself).  Every operand is bit-identical to what the separate entry points produce
// with the same rounding arguments, so the results are too.
#include "common.cuh"

namespace nvfp4 {
namespace {

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct Operand {            // a quantized operand in a buffer: offsets of its codes and scales
  size_t codes, sf;
};

size_t place(size_t& off, int64_t Rq, int64_t Kq, Operand* op) {
  op->codes = off; off = align256(off + (size_t)(Rq * Kq / 2));
  op->sf = off;    off = align256(off + nvfp4_sf_bytes(Rq, Kq, NVFP4_SF_SWIZZLED_128x4));
  return off;
}

struct SavedLayout { Operand wt, xt; size_t gx, gw, total; };
SavedLayout saved_layout(int64_t M, int64_t N, int64_t K) {
  SavedLayout l; size_t off = 0;
  place(off, K, N, &l.wt);                 // Q(W^T): [K, N]
  place(off, K, M, &l.xt);                 // Q(X^T): [K, M]
  l.gx = off; off = align256(off + sizeof(float));
  l.gw = off; off = align256(off + sizeof(float));
  l.total = off;
  return l;
}

struct FwdLayout { Operand x, w; size_t scratch, total; };
FwdLayout fwd_layout(int64_t M, int64_t N, int64_t K) {
  FwdLayout l; size_t off = 0;
  place(off, M, K, &l.x);
  place(off, N, K, &l.w);
  l.scratch = off; off = align256(off + 64);          // zeroed words of the one-launch amax passes
  l.total = off;
  return l;
}

struct BwdLayout { Operand dy, dyt, wt, xt; size_t gdy, gw, gx, scratch, total; };
BwdLayout bwd_layout(int64_t M, int64_t N, int64_t K, bool with_saved) {
  BwdLayout l; size_t off = 0;
  place(off, M, N, &l.dy);                 // Q(dY): [M, N]
  place(off, N, M, &l.dyt);                // Q(dY^T): [N, M]
  l.wt = l.xt = Operand{0, 0};
  if (!with_saved) { place(off, K, N, &l.wt); place(off, K, M, &l.xt); }
  l.gdy = off; off = align256(off + sizeof(float));
  l.gw = off; off = align256(off + sizeof(float));
  l.gx = off; off = align256(off + sizeof(float));
  l.scratch = off; off = align256(off + 64);
  l.total = off;
  return l;
}

bool shapes_ok(int64_t M, int64_t N, int64_t K) {
  return M > 0 && N > 0 && K > 0 && M % 32 == 0 && N % 32 == 0 && K % 32 == 0;
}
bool enums_ok(int dtype, int out_dtype, int gscale_mode) {
  return (dtype == NVFP4_BF16 || dtype == NVFP4_FP32) && (out_dtype == NVFP4_BF16 || out_dtype == NVFP4_FP32) &&
         (gscale_mode == NVFP4_G_NONE || gscale_mode == NVFP4_G_AMAX || gscale_mode == NVFP4_G_GIVEN);
}
bool buffer_ok(const void* p, size_t have, size_t need) {
  return p && have >= need && (reinterpret_cast<uintptr_t>(p) & 255u) == 0;
}

// Per-tensor scale of one operand according to gscale_mode: NULL, computed into `slot` (one launch, with two
// zeroed scratch words), or given.
int resolve_g(int gscale_mode, const void* x, int dtype, int64_t rows, int64_t cols, const float* given, float* slot,
              unsigned int* scratch, void* stream, const float** out) {
  *out = nullptr;
  if (gscale_mode == NVFP4_G_AMAX) {
    if (int st = tensor_amax_scale_ws(x, dtype, rows, cols, cols, slot, scratch, stream)) return st;
    *out = slot;
  } else if (gscale_mode == NVFP4_G_GIVEN) {
    if (!given) return NVFP4_ERR_NULL;
    *out = given;
  }
  return NVFP4_OK;
}

int zero_scratch(int gscale_mode, void* scratch, void* stream) {
  if (gscale_mode != NVFP4_G_AMAX) return NVFP4_OK;
  return cudaMemsetAsync(scratch, 0, 64, static_cast<cudaStream_t>(stream)) == cudaSuccess ? NVFP4_OK : NVFP4_ERR_CUDA;
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

extern "C" size_t nvfp4_linear_saved_bytes(int64_t M, int64_t N, int64_t K) {
  return shapes_ok(M, N, K) ? saved_layout(M, N, K).total : 0;
}

extern "C" size_t nvfp4_linear_fused_workspace_bytes(int64_t M, int64_t N, int64_t K, int which) {
  if (!shapes_ok(M, N, K)) return 0;
  switch (which) {
    case NVFP4_FUSED_FWD_SAVE: return fwd_layout(M, N, K).total;
    case NVFP4_FUSED_BWD_SAVED: return bwd_layout(M, N, K, true).total;
    case NVFP4_FUSED_BWD: return bwd_layout(M, N, K, false).total;
    default: return 0;
  }
}

extern "C" int nvfp4_linear_fwd_save(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                     int gscale_mode, const float* gx, const float* gw,
                                     const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                                     const nvfp4_rounding* rxt, const nvfp4_rounding* rwt,
                                     void* Y, int y_dtype, void* saved, size_t saved_bytes,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!X || !W || !rx || !rw || !rxt || !rwt || !Y) return NVFP4_ERR_NULL;
  if (!enums_ok(dtype, y_dtype, gscale_mode)) return NVFP4_ERR_ENUM;
  if (!shapes_ok(M, N, K)) return NVFP4_ERR_SHAPE;
  const SavedLayout sl = saved_layout(M, N, K);
  const FwdLayout fl = fwd_layout(M, N, K);
  if (!buffer_ok(saved, saved_bytes, sl.total) || !buffer_ok(workspace, workspace_bytes, fl.total)) return NVFP4_ERR_WORKSPACE;
  uint8_t* sv = static_cast<uint8_t*>(saved);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  float* sgx = reinterpret_cast<float*>(sv + sl.gx);
  float* sgw = reinterpret_cast<float*>(sv + sl.gw);
  const float *g_x, *g_w;
  unsigned int* scratch = reinterpret_cast<unsigned int*>(ws + fl.scratch);
  if (int st = zero_scratch(gscale_mode, scratch, cuda_stream)) return st;
  if (gscale_mode == NVFP4_G_GIVEN) {       // the backward pass reads the scales from `saved`
    if (!gx || !gw) return NVFP4_ERR_NULL;
    if (cudaMemcpyAsync(sgx, gx, sizeof(float), cudaMemcpyDeviceToDevice, s) != cudaSuccess) return NVFP4_ERR_CUDA;
    if (cudaMemcpyAsync(sgw, gw, sizeof(float), cudaMemcpyDeviceToDevice, s) != cudaSuccess) return NVFP4_ERR_CUDA;
  }
  // W first: amax(W) leaves the (smaller) weight tensor in L2 for the quantizer that follows it
  if (int st = resolve_g(gscale_mode, W, dtype, N, K, gw, sgw, scratch, cuda_stream, &g_w)) return st;
  if (int st = nvfp4_quantize_dual(W, dtype, N, K, K, g_w, rw, ws + fl.w.codes, ws + fl.w.sf, rwt, sv + sl.wt.codes,
                                   sv + sl.wt.sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))
    return st;
  if (int st = resolve_g(gscale_mode, X, dtype, M, K, gx, sgx, scratch + 2, cuda_stream, &g_x)) return st;
  if (int st = nvfp4_quantize_dual(X, dtype, M, K, K, g_x, rx, ws + fl.x.codes, ws + fl.x.sf, rxt, sv + sl.xt.codes,
                                   sv + sl.xt.sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))
    return st;
  return nvfp4_gemm(ws + fl.x.codes, ws + fl.x.sf, g_x, ws + fl.w.codes, ws + fl.w.sf, g_w, M, N, K, Y, y_dtype, N,
                    cuda_stream);
}

namespace {
// dY both ways from one read, then dX = Q(dY) . Q(W^T)^T and dW = Q(dY^T) . Q(X^T)^T.
int run_bwd(const void* dY, int dtype, int64_t M, int64_t N, int64_t K, const float* g_dy,
            const nvfp4_rounding* rdy, const nvfp4_rounding* rdyt,
            const uint8_t* wt_codes, const uint8_t* wt_sf, const float* g_w,
            const uint8_t* xt_codes, const uint8_t* xt_sf, const float* g_x,
            void* dX, int dx_dtype, void* dW, int dw_dtype, uint8_t* ws, const BwdLayout& bl, void* stream) {
  if (int st = nvfp4_quantize_dual(dY, dtype, M, N, N, g_dy, rdy, ws + bl.dy.codes, ws + bl.dy.sf, rdyt,
                                   ws + bl.dyt.codes, ws + bl.dyt.sf, NVFP4_SF_SWIZZLED_128x4, stream))
    return st;
  if (int st = nvfp4_gemm(ws + bl.dy.codes, ws + bl.dy.sf, g_dy, wt_codes, wt_sf, g_w, M, K, N, dX, dx_dtype, K, stream))
    return st;
  return nvfp4_gemm(ws + bl.dyt.codes, ws + bl.dyt.sf, g_dy, xt_codes, xt_sf, g_x, N, K, M, dW, dw_dtype, K, stream);
}
}  // namespace

extern "C" int nvfp4_linear_bwd_saved(const void* dY, int dtype, int64_t M, int64_t N, int64_t K,
                                      int gscale_mode, const float* gdy,
                                      const nvfp4_rounding* rdy, const nvfp4_rounding* rdyt,
                                      const void* saved, size_t saved_bytes,
                                      void* dX, int dx_dtype, void* dW, int dw_dtype,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!dY || !rdy || !rdyt || !dX || !dW) return NVFP4_ERR_NULL;
  if (!enums_ok(dtype, dx_dtype, gscale_mode) || (dw_dtype != NVFP4_BF16 && dw_dtype != NVFP4_FP32)) return NVFP4_ERR_ENUM;
  if (!shapes_ok(M, N, K)) return NVFP4_ERR_SHAPE;
  const SavedLayout sl = saved_layout(M, N, K);
  const BwdLayout bl = bwd_layout(M, N, K, true);
  if (!buffer_ok(saved, saved_bytes, sl.total) || !buffer_ok(workspace, workspace_bytes, bl.total)) return NVFP4_ERR_WORKSPACE;
  const uint8_t* sv = static_cast<const uint8_t*>(saved);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float* g_dy;
  unsigned int* scratch = reinterpret_cast<unsigned int*>(ws + bl.scratch);
  if (int st = zero_scratch(gscale_mode, scratch, cuda_stream)) return st;
  if (int st = resolve_g(gscale_mode, dY, dtype, M, N, gdy, reinterpret_cast<float*>(ws + bl.gdy), scratch, cuda_stream, &g_dy)) return st;
  const bool scaled = gscale_mode != NVFP4_G_NONE;     // must match the mode nvfp4_linear_fwd_save ran with
  const float* g_x = scaled ? reinterpret_cast<const float*>(sv + sl.gx) : nullptr;
  const float* g_w = scaled ? reinterpret_cast<const float*>(sv + sl.gw) : nullptr;
  return run_bwd(dY, dtype, M, N, K, g_dy, rdy, rdyt, sv + sl.wt.codes, sv + sl.wt.sf, g_w, sv + sl.xt.codes, sv + sl.xt.sf,
                 g_x, dX, dx_dtype, dW, dw_dtype, ws, bl, cuda_stream);
}

extern "C" int nvfp4_linear_bwd(const void* dY, const void* W, const void* X, int dtype, int64_t M, int64_t N, int64_t K,
                                int gscale_mode, const float* gdy, const float* gw, const float* gx,
                                const nvfp4_rounding* rdy, const nvfp4_rounding* rdyt,
                                const nvfp4_rounding* rwt, const nvfp4_rounding* rxt,
                                void* dX, int dx_dtype, void* dW, int dw_dtype,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!dY || !W || !X || !rdy || !rdyt || !rwt || !rxt || !dX || !dW) return NVFP4_ERR_NULL;
  if (!enums_ok(dtype, dx_dtype, gscale_mode) || (dw_dtype != NVFP4_BF16 && dw_dtype != NVFP4_FP32)) return NVFP4_ERR_ENUM;
  if (!shapes_ok(M, N, K)) return NVFP4_ERR_SHAPE;
  const BwdLayout bl = bwd_layout(M, N, K, false);
  if (!buffer_ok(workspace, workspace_bytes, bl.total)) return NVFP4_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float *g_dy, *g_w, *g_x;
  unsigned int* scratch = reinterpret_cast<unsigned int*>(ws + bl.scratch);
  if (int st = zero_scratch(gscale_mode, scratch, cuda_stream)) return st;
  if (int st = resolve_g(gscale_mode, dY, dtype, M, N, gdy, reinterpret_cast<float*>(ws + bl.gdy), scratch, cuda_stream, &g_dy)) return st;
  if (int st = resolve_g(gscale_mode, W, dtype, N, K, gw, reinterpret_cast<float*>(ws + bl.gw), scratch + 2, cuda_stream, &g_w)) return st;
  if (int st = resolve_g(gscale_mode, X, dtype, M, K, gx, reinterpret_cast<float*>(ws + bl.gx), scratch + 4, cuda_stream, &g_x)) return st;
  if (int st = nvfp4_quantize(W, dtype, N, K, K, 1, g_w, rwt, ws + bl.wt.codes, ws + bl.wt.sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))
    return st;
  if (int st = nvfp4_quantize(X, dtype, M, K, K, 1, g_x, rxt, ws + bl.xt.codes, ws + bl.xt.sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))
    return st;
  return run_bwd(dY, dtype, M, N, K, g_dy, rdy, rdyt, ws + bl.wt.codes, ws + bl.wt.sf, g_w, ws + bl.xt.codes, ws + bl.xt.sf,
                 g_x, dX, dx_dtype, dW, dw_dtype, ws, bl, cuda_stream);
}
