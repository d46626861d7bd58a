// The three quantized linear-layer products of Eq. 1-3 with the operand quantization of
// Eq. 4-6: each call quantizes its two operands along the contraction axis into the caller's
// workspace (row or transposed quantizer) and runs the block-scaled GEMM on them.
#include "common.cuh"

namespace nvfp4 {
namespace {

struct Plan {
  int64_t gemm_m, gemm_n, gemm_k;      // D[gemm_m, gemm_n], contraction gemm_k
  int a_transposed, b_transposed;      // how each operand is quantized
  int64_t a_rows, a_cols, b_rows, b_cols;  // source shapes
};

// which: 0 fwd  (A = X[M,K] row,        B = W[N,K] row,         D = Y[M,N])
//        1 dx   (A = dY[M,N] row,       B = W[N,K] transposed,  D = dX[M,K])
//        2 dw   (A = dY[M,N] transposed, B = X[M,K] transposed, D = dW[N,K])
bool make_plan(int64_t M, int64_t N, int64_t K, int which, Plan* pl) {
  if (M <= 0 || N <= 0 || K <= 0) return false;
  switch (which) {
    case NVFP4_LINEAR_FWD: *pl = {M, N, K, 0, 0, M, K, N, K}; return true;
    case NVFP4_LINEAR_BWD_DX: *pl = {M, K, N, 0, 1, M, N, N, K}; return true;
    case NVFP4_LINEAR_BWD_DW: *pl = {N, K, M, 1, 1, M, N, M, K}; return true;
    default: return false;
  }
}

// The shapes the layer calls take (the same predicate sizes the workspace): code rows of K/2 bytes need a
// 16-byte pitch for the tiled copies, source rows and output rows are moved in 16-byte pieces.
bool plan_ok(const Plan& pl) {
  return pl.gemm_k % 32 == 0 && pl.a_cols % 8 == 0 && pl.b_cols % 8 == 0 && pl.gemm_n % 8 == 0;
}

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct Layout {
  size_t a_codes, a_sf, b_codes, b_sf, a_g, b_g, total;
};

Layout make_layout(const Plan& pl) {
  Layout l;
  size_t off = 0;
  l.a_codes = off; off = align256(off + (size_t)(pl.gemm_m * pl.gemm_k / 2));
  l.a_sf = off;    off = align256(off + nvfp4_sf_bytes(pl.gemm_m, pl.gemm_k, NVFP4_SF_SWIZZLED_128x4));
  l.b_codes = off; off = align256(off + (size_t)(pl.gemm_n * pl.gemm_k / 2));
  l.b_sf = off;    off = align256(off + nvfp4_sf_bytes(pl.gemm_n, pl.gemm_k, NVFP4_SF_SWIZZLED_128x4));
  l.a_g = off;     off = align256(off + sizeof(float));
  l.b_g = off;     off = align256(off + sizeof(float));
  l.total = off;
  return l;
}

int run_linear(int which, const void* a, const void* b, int dtype, int64_t M, int64_t N, int64_t K,
               int gscale_mode, const float* ga, const float* gb, const nvfp4_rounding* ra,
               const nvfp4_rounding* rb, void* out, int out_dtype, void* workspace, size_t workspace_bytes,
               void* stream) {
  if (!a || !b || !ra || !rb || !out) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (out_dtype != NVFP4_BF16 && out_dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (gscale_mode != NVFP4_G_NONE && gscale_mode != NVFP4_G_AMAX && gscale_mode != NVFP4_G_GIVEN) return NVFP4_ERR_ENUM;
  if (gscale_mode == NVFP4_G_GIVEN && (!ga || !gb)) return NVFP4_ERR_NULL;
  for (const nvfp4_rounding* r : {ra, rb})              // rejected here, before the amax launches, not by the quantizer after them
    if ((r->mode != NVFP4_RTN && r->mode != NVFP4_SR) || r->reserved != 0) return NVFP4_ERR_ENUM;
  if (!aligned16(a) || !aligned16(b) || !aligned16(out)) return NVFP4_ERR_ALIGN;
  Plan pl;
  if (!make_plan(M, N, K, which, &pl)) return NVFP4_ERR_SHAPE;
  if (!plan_ok(pl)) return NVFP4_ERR_SHAPE;
  const Layout l = make_layout(pl);
  if (!workspace || workspace_bytes < l.total || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return NVFP4_ERR_WORKSPACE;

  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float* g_a = nullptr;
  const float* g_b = nullptr;
  int st;
  if (gscale_mode == NVFP4_G_AMAX) {
    float* wa = reinterpret_cast<float*>(ws + l.a_g);
    float* wb = reinterpret_cast<float*>(ws + l.b_g);
    if ((st = nvfp4_tensor_amax_scale(a, dtype, pl.a_rows, pl.a_cols, pl.a_cols, wa, stream))) return st;
    if ((st = nvfp4_tensor_amax_scale(b, dtype, pl.b_rows, pl.b_cols, pl.b_cols, wb, stream))) return st;
    g_a = wa; g_b = wb;
  } else if (gscale_mode == NVFP4_G_GIVEN) {
    g_a = ga; g_b = gb;
  }
  if ((st = nvfp4_quantize(a, dtype, pl.a_rows, pl.a_cols, pl.a_cols, pl.a_transposed, g_a, ra, ws + l.a_codes,
                           ws + l.a_sf, NVFP4_SF_SWIZZLED_128x4, stream))) return st;
  if ((st = nvfp4_quantize(b, dtype, pl.b_rows, pl.b_cols, pl.b_cols, pl.b_transposed, g_b, rb, ws + l.b_codes,
                           ws + l.b_sf, NVFP4_SF_SWIZZLED_128x4, stream))) return st;
  return nvfp4_gemm(ws + l.a_codes, ws + l.a_sf, g_a, ws + l.b_codes, ws + l.b_sf, g_b, pl.gemm_m, pl.gemm_n,
                    pl.gemm_k, out, out_dtype, pl.gemm_n, stream);
}

}  // namespace
}  // namespace nvfp4

using namespace nvfp4;

extern "C" size_t nvfp4_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, int which) {
  Plan pl;
  if (!make_plan(M, N, K, which, &pl) || !plan_ok(pl)) return 0;
  return make_layout(pl).total;
}

extern "C" int nvfp4_linear_fwd(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                int gscale_mode, const float* gx, const float* gw,
                                const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                                void* Y, int y_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return run_linear(NVFP4_LINEAR_FWD, X, W, dtype, M, N, K, gscale_mode, gx, gw, rx, rw, Y, y_dtype, workspace,
                    workspace_bytes, cuda_stream);
}

extern "C" int nvfp4_linear_bwd_dx(const void* dY, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                   int gscale_mode, const float* gdy, const float* gw,
                                   const nvfp4_rounding* rdy, const nvfp4_rounding* rw,
                                   void* dX, int dx_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return run_linear(NVFP4_LINEAR_BWD_DX, dY, W, dtype, M, N, K, gscale_mode, gdy, gw, rdy, rw, dX, dx_dtype,
                    workspace, workspace_bytes, cuda_stream);
}

extern "C" int nvfp4_linear_bwd_dw(const void* dY, const void* X, int dtype, int64_t M, int64_t N, int64_t K,
                                   int gscale_mode, const float* gdy, const float* gx,
                                   const nvfp4_rounding* rdy, const nvfp4_rounding* rx,
                                   void* dW, int dw_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return run_linear(NVFP4_LINEAR_BWD_DW, dY, X, dtype, M, N, K, gscale_mode, gdy, gx, rdy, rx, dW, dw_dtype,
                    workspace, workspace_bytes, cuda_stream);
}

// ------------------------------------------------------------------------------------------------
// Producer fusion along a chain of layers (no high-precision round trip between them): the first layer
// writes Q(Y) straight from its GEMM epilogue, the next layer takes that quantized operand as its Q(X).
// ------------------------------------------------------------------------------------------------
extern "C" int nvfp4_linear_fwd_qout(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                     int gscale_mode, const float* gx, const float* gw,
                                     const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                                     const float* gy, const nvfp4_rounding* ry,
                                     uint8_t* y_codes, uint8_t* y_scales, int sf_layout,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!X || !W || !rx || !rw || !ry || !y_codes || !y_scales) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (sf_layout != NVFP4_SF_LINEAR && sf_layout != NVFP4_SF_SWIZZLED_128x4) return NVFP4_ERR_ENUM;
  for (const nvfp4_rounding* r : {rx, rw, ry})          // everything the later calls would reject is rejected before the first launch
    if ((r->mode != NVFP4_RTN && r->mode != NVFP4_SR) || r->reserved != 0) return NVFP4_ERR_ENUM;
  if (!aligned16(X) || !aligned16(W) || !aligned16(y_codes) || !aligned16(y_scales)) return NVFP4_ERR_ALIGN;
  if (gscale_mode != NVFP4_G_NONE && gscale_mode != NVFP4_G_AMAX && gscale_mode != NVFP4_G_GIVEN) return NVFP4_ERR_ENUM;
  if (gscale_mode == NVFP4_G_GIVEN && (!gx || !gw)) return NVFP4_ERR_NULL;
  Plan pl;
  if (!make_plan(M, N, K, NVFP4_LINEAR_FWD, &pl) || !plan_ok(pl) || N % 32 != 0) return NVFP4_ERR_SHAPE;
  const Layout l = make_layout(pl);
  if (!workspace || workspace_bytes < l.total || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return NVFP4_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float* g_x = nullptr;
  const float* g_w = nullptr;
  int st;
  if (gscale_mode == NVFP4_G_AMAX) {
    float* wa = reinterpret_cast<float*>(ws + l.a_g);
    float* wb = reinterpret_cast<float*>(ws + l.b_g);
    if ((st = nvfp4_tensor_amax_scale(X, dtype, M, K, K, wa, cuda_stream))) return st;
    if ((st = nvfp4_tensor_amax_scale(W, dtype, N, K, K, wb, cuda_stream))) return st;
    g_x = wa; g_w = wb;
  } else if (gscale_mode == NVFP4_G_GIVEN) {
    g_x = gx; g_w = gw;
  }
  if ((st = nvfp4_quantize(X, dtype, M, K, K, 0, g_x, rx, ws + l.a_codes, ws + l.a_sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))) return st;
  if ((st = nvfp4_quantize(W, dtype, N, K, K, 0, g_w, rw, ws + l.b_codes, ws + l.b_sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))) return st;
  return nvfp4_gemm_quantized(ws + l.a_codes, ws + l.a_sf, g_x, ws + l.b_codes, ws + l.b_sf, g_w, M, N, K, gy, ry, y_codes,
                              y_scales, sf_layout, cuda_stream);
}

extern "C" int nvfp4_linear_fwd_qin(const uint8_t* x_codes, const uint8_t* x_scales, const float* gx,
                                    const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                    int gscale_mode, const float* gw, const nvfp4_rounding* rw,
                                    void* Y, int y_dtype, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!x_codes || !x_scales || !W || !rw || !Y) return NVFP4_ERR_NULL;
  if (dtype != NVFP4_BF16 && dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if ((rw->mode != NVFP4_RTN && rw->mode != NVFP4_SR) || rw->reserved != 0) return NVFP4_ERR_ENUM;
  if (!aligned16(x_codes) || !aligned16(x_scales) || !aligned16(W) || !aligned16(Y)) return NVFP4_ERR_ALIGN;
  if (y_dtype != NVFP4_BF16 && y_dtype != NVFP4_FP32) return NVFP4_ERR_ENUM;
  if (gscale_mode != NVFP4_G_NONE && gscale_mode != NVFP4_G_AMAX && gscale_mode != NVFP4_G_GIVEN) return NVFP4_ERR_ENUM;
  if (gscale_mode == NVFP4_G_GIVEN && !gw) return NVFP4_ERR_NULL;
  Plan pl;
  if (!make_plan(M, N, K, NVFP4_LINEAR_FWD, &pl) || !plan_ok(pl)) return NVFP4_ERR_SHAPE;
  const Layout l = make_layout(pl);
  if (!workspace || workspace_bytes < l.total || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return NVFP4_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float* g_w = nullptr;
  int st;
  if (gscale_mode == NVFP4_G_AMAX) {
    float* wb = reinterpret_cast<float*>(ws + l.b_g);
    if ((st = nvfp4_tensor_amax_scale(W, dtype, N, K, K, wb, cuda_stream))) return st;
    g_w = wb;
  } else if (gscale_mode == NVFP4_G_GIVEN) {
    g_w = gw;
  }
  if ((st = nvfp4_quantize(W, dtype, N, K, K, 0, g_w, rw, ws + l.b_codes, ws + l.b_sf, NVFP4_SF_SWIZZLED_128x4, cuda_stream))) return st;
  return nvfp4_gemm(x_codes, x_scales, gx, ws + l.b_codes, ws + l.b_sf, g_w, M, N, K, Y, y_dtype, N, cuda_stream);
}

// ------------------------------------------------------------------------------------------------
// Forward product with the scratch in a fixed device array (no allocation anywhere on the path).
// For callers that cannot get scratch memory when they call: the device may already be fully
// reserved by the host framework's own pool, or the section may not tolerate the device-wide
// synchronisation that cudaMalloc / cudaFree imply.
// ------------------------------------------------------------------------------------------------
namespace {

// Lives in the device image of this library: each GPU that loads it holds these bytes until exit.
static __device__ __align__(256) unsigned char g_static_workspace[NVFP4_STATIC_WORKSPACE_BYTES];

// In host code `g_static_workspace` is only a handle for the runtime, not a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, looked up once per device with that
// device current.
int static_workspace_address(void** out) {
  static void* address[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NVFP4_ERR_CUDA;
  if (!address[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return NVFP4_ERR_CUDA;
    address[dev] = p;
  }
  *out = address[dev];
  return NVFP4_OK;
}

}  // namespace

extern "C" int nvfp4_linear_fwd_static(const void* X, const void* W, int dtype, int64_t M, int64_t N, int64_t K,
                                       int gscale_mode, const float* gx, const float* gw,
                                       const nvfp4_rounding* rx, const nvfp4_rounding* rw,
                                       void* Y, int y_dtype, void* cuda_stream) {
  const size_t need = nvfp4_linear_workspace_bytes(M, N, K, NVFP4_LINEAR_FWD);
  if (need == 0) return NVFP4_ERR_SHAPE;
  if (need > (size_t)NVFP4_STATIC_WORKSPACE_BYTES) return NVFP4_ERR_WORKSPACE;  // layer too large for the fixed array
  if (int st = check_arch()) return st;
  void* scratch = nullptr;
  if (int st = static_workspace_address(&scratch)) return st;
  // The quantizers rewrite every code and scale byte (padding included) that the GEMM reads and
  // the amax pass clears its own accumulator, so the previous call's contents need no clearing.
  return run_linear(NVFP4_LINEAR_FWD, X, W, dtype, M, N, K, gscale_mode, gx, gw, rx, rw, Y, y_dtype, scratch,
                    (size_t)NVFP4_STATIC_WORKSPACE_BYTES, cuda_stream);
}
