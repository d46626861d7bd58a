"""GPU-vs-oracle parity of the three quantized linear-layer products (Eq. 1-6)."""
import numpy as np
import pytest
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _host(x):
    return x.float().cpu().numpy()


def _oracle_operand(x, transposed, r, use_g):
    h = _host(x)
    g = ob.tensor_amax_scale(h) if use_g else 1.0
    c, s = ob.quantize(h, g=g, mode=r.mode, seed=r.seed, offset=r.offset, transposed=transposed)
    return c, s, g


def oracle_linear(which, a, b, ra, rb, use_g, sample=None):
    ta, tb = {"fwd": (False, False), "dx": (False, True), "dw": (True, True)}[which]
    ac, asf, ga = _oracle_operand(a, ta, ra, use_g)
    bc, bsf, gb = _oracle_operand(b, tb, rb, use_g)
    if sample is None:
        return ob.gemm(ac, asf, ga, bc, bsf, gb)
    return ob.gemm_sampled(ac, asf, ga, bc, bsf, gb, sample[0], sample[1])


def _assert_close(got, ref, T):
    err = np.abs(got - ref)
    assert np.all(err <= TOL * T), f"max err/T = {np.max(err / np.maximum(T, 1e-30)):.3e}"


@pytest.mark.parametrize("use_g", [True, False])
def test_single_layer_all_three_products(use_g):
    # single small layer: X 256x512 N(0,1), W 512x512 N(0,0.02^2), dY 256x512 N(0,1e-3^2)
    t = synth.TINY_LINEAR
    X, W, dY = synth.linear_inputs(t["tokens"], t["K"], t["N"], seed=1001, grad_std=1e-3)
    X, W, dY = X.cuda(), W.cuda(), dY.cuda()
    mode = nb.G_AMAX if use_g else nb.G_NONE
    rt, sr0, sr1, sr2 = nb.Rounding(nb.RTN), nb.Rounding(nb.SR, 0, 0), nb.Rounding(nb.SR, 0, 1), nb.Rounding(nb.SR, 0, 2)
    Y = nb.nvfp4_linear_fwd(X, W, gscale_mode=mode, rx=rt, rw=rt)
    dX = nb.nvfp4_linear_bwd_dx(dY, W, gscale_mode=mode, rdy=sr0, rw=rt)
    dW = nb.nvfp4_linear_bwd_dw(dY, X, gscale_mode=mode, rdy=sr1, rx=sr2)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    _assert_close(_host(Y), *oracle_linear("fwd", X, W, rt, rt, use_g))
    _assert_close(_host(dX), *oracle_linear("dx", dY, W, sr0, rt, use_g))
    _assert_close(_host(dW), *oracle_linear("dw", dY, X, sr1, sr2, use_g))
    if not use_g:
        # without a per-tensor scale the 1e-3 gradients underflow the E4M3 scale range entirely
        assert float(dX.abs().max()) == 0.0 and float(dW.abs().max()) == 0.0
    else:
        assert float(dX.abs().max()) > 0.0 and float(dW.abs().max()) > 0.0


def test_all_sr_backward_variant():
    # the single-layer config also asks for SR on W in the backward product
    t = synth.TINY_LINEAR
    X, W, dY = synth.linear_inputs(t["tokens"], t["K"], t["N"], seed=1001, grad_std=1e-3)
    W, dY = W.cuda(), dY.cuda()
    sr0, sr3 = nb.Rounding(nb.SR, 0, 0), nb.Rounding(nb.SR, 0, 3)
    dX = nb.nvfp4_linear_bwd_dx(dY, W, rdy=sr0, rw=sr3)
    _assert_close(_host(dX), *oracle_linear("dx", dY, W, sr0, sr3, True))


def test_ragged_layer_and_bf16_output():
    X, W, dY = synth.linear_inputs(160, 288, 200, seed=7, grad_std=1e-3)
    X, W, dY = X.cuda(), W.cuda(), dY.cuda()
    rt, sr = nb.Rounding(nb.RTN), nb.Rounding(nb.SR, 9, 0)
    Y = nb.nvfp4_linear_fwd(X, W, rx=rt, rw=rt)
    _assert_close(_host(Y), *oracle_linear("fwd", X, W, rt, rt, True))
    dW = nb.nvfp4_linear_bwd_dw(dY, X, rdy=sr, rx=sr)
    _assert_close(_host(dW), *oracle_linear("dw", dY, X, sr, sr, True))
    Yb = nb.nvfp4_linear_fwd(X, W, rx=rt, rw=rt, out_dtype=torch.bfloat16)
    ref, T = oracle_linear("fwd", X, W, rt, rt, True)
    assert np.all(np.abs(_host(Yb) - ref) <= TOL * T + np.abs(ref) * 2.0 ** -8)


def test_given_global_scales_and_fp32_inputs():
    X, W, _ = synth.linear_inputs(128, 256, 128, seed=8)
    X, W = X.float().cuda(), W.float().cuda()
    gx, gw = nb.nvfp4_tensor_amax_scale(X), nb.nvfp4_tensor_amax_scale(W)
    rt = nb.Rounding(nb.RTN)
    Y = nb.nvfp4_linear_fwd(X, W, gscale_mode=nb.G_GIVEN, gx=gx, gw=gw, rx=rt, rw=rt)
    _assert_close(_host(Y), *oracle_linear("fwd", X, W, rt, rt, True))


@pytest.mark.parametrize("name,K,N", [(n, k, o) for (n, k, o) in synth.LLAMA_350M["linears"] if n in ("qkv", "down")])
def test_350m_block_linears_sampled(name, K, N):
    M = synth.LLAMA_350M["tokens"]
    X, W, dY = synth.linear_inputs(M, K, N, seed=1003)
    X, W, dY = X.cuda(), W.cuda(), dY.cuda()
    rt, sr0, sr1, sr2 = nb.Rounding(nb.RTN), nb.Rounding(nb.SR, 0, 0), nb.Rounding(nb.SR, 0, 1), nb.Rounding(nb.SR, 0, 2)
    rng = np.random.default_rng(3)
    n = 2048

    def sample(R, C):
        return (np.concatenate([rng.integers(0, R, n), [0, R - 1]]), np.concatenate([rng.integers(0, C, n), [C - 1, 0]]))

    Y = nb.nvfp4_linear_fwd(X, W, rx=rt, rw=rt)
    s = sample(M, N)
    _assert_close(_host(Y)[s[0], s[1]], *oracle_linear("fwd", X, W, rt, rt, True, s))
    dX = nb.nvfp4_linear_bwd_dx(dY, W, rdy=sr0, rw=rt)
    s = sample(M, K)
    _assert_close(_host(dX)[s[0], s[1]], *oracle_linear("dx", dY, W, sr0, rt, True, s))
    dW = nb.nvfp4_linear_bwd_dw(dY, X, rdy=sr1, rx=sr2)
    s = sample(N, K)
    _assert_close(_host(dW)[s[0], s[1]], *oracle_linear("dw", dY, X, sr1, sr2, True, s))
    assert nb.nvfp4_device_error_word() == 0


# ---------------------------------------------------------------- fused layer: every tensor read once per pass
@pytest.mark.parametrize("use_g", [True, False])
@pytest.mark.parametrize("shape", [(256, 512, 512), (160, 288, 224), (512, 64, 96)])
def test_fused_layer_equals_the_separate_products(shape, use_g):
    M, K, N = shape
    X, W, dY = synth.linear_inputs(M, K, N, seed=31, grad_std=1e-3)
    X, W, dY = X.cuda(), W.cuda(), dY.cuda()
    mode = nb.G_AMAX if use_g else nb.G_NONE
    rt, sr0, sr1, sr2 = nb.Rounding(nb.RTN), nb.Rounding(nb.SR, 5, 0), nb.Rounding(nb.SR, 5, 1), nb.Rounding(nb.SR, 5, 2)
    Y = nb.nvfp4_linear_fwd(X, W, gscale_mode=mode, rx=rt, rw=rt)
    dX = nb.nvfp4_linear_bwd_dx(dY, W, gscale_mode=mode, rdy=sr0, rw=rt)
    dW = nb.nvfp4_linear_bwd_dw(dY, X, gscale_mode=mode, rdy=sr1, rx=sr2)
    Yf, saved = nb.nvfp4_linear_fwd_save(X, W, gscale_mode=mode, rx=rt, rw=rt, rxt=sr2, rwt=rt)
    dXf, dWf = nb.nvfp4_linear_bwd_saved(dY, saved, K, gscale_mode=mode, rdy=sr0, rdyt=sr1)
    dXb, dWb = nb.nvfp4_linear_bwd(dY, W, X, gscale_mode=mode, rdy=sr0, rdyt=sr1, rwt=rt, rxt=sr2)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    assert torch.equal(Y, Yf) and torch.equal(dX, dXf) and torch.equal(dW, dWf)
    assert torch.equal(dX, dXb) and torch.equal(dW, dWb)
    _assert_close(_host(Yf), *oracle_linear("fwd", X, W, rt, rt, use_g))
    _assert_close(_host(dXf), *oracle_linear("dx", dY, W, sr0, rt, use_g))
    _assert_close(_host(dWf), *oracle_linear("dw", dY, X, sr1, sr2, use_g))


def test_fused_layer_with_given_scales_and_bf16_outputs():
    M, K, N = 256, 256, 384
    X, W, dY = synth.linear_inputs(M, K, N, seed=32, grad_std=1e-3)
    X, W, dY = X.cuda(), W.cuda(), dY.cuda()
    gx, gw, gdy = (nb.nvfp4_tensor_amax_scale(t) for t in (X, W, dY))
    Y, saved = nb.nvfp4_linear_fwd_save(X, W, gscale_mode=nb.G_GIVEN, gx=gx, gw=gw, out_dtype=torch.bfloat16)
    dX, dW = nb.nvfp4_linear_bwd_saved(dY, saved, K, gscale_mode=nb.G_GIVEN, gdy=gdy, dx_dtype=torch.bfloat16)
    rt = nb.Rounding(nb.RTN)
    ref, T = oracle_linear("fwd", X, W, rt, rt, True)
    assert np.all(np.abs(_host(Y) - ref) <= TOL * T + np.abs(ref) * 2.0 ** -8)
    ref, T = oracle_linear("dx", dY, W, nb.Rounding(nb.SR, 0, 0), rt, True)
    assert np.all(np.abs(_host(dX) - ref) <= TOL * T + np.abs(ref) * 2.0 ** -8)
    _assert_close(_host(dW), *oracle_linear("dw", dY, X, nb.Rounding(nb.SR, 0, 1), nb.Rounding(nb.SR, 0, 2), True))


# ---------------------------------------------------------------- non-finite inputs stay visible
@pytest.mark.parametrize("bad", [float("nan"), float("inf"), float("-inf")])
def test_non_finite_input_propagates_through_the_per_tensor_scale(bad):
    # A NaN (or an infinity) anywhere in an operand makes its amax scale NaN (+Inf), as the oracle's does, and
    # every element of a product computed with that scale NaN; products of the other operands stay finite.
    M, K, N = 256, 512, 384
    X, W, dY = synth.linear_inputs(M, K, N, seed=77, grad_std=1e-3)
    X[131, 257] = bad
    Xd, Wd, dYd = X.cuda(), W.cuda(), dY.cuda()
    g = nb.nvfp4_tensor_amax_scale(Xd)
    want = ob.tensor_amax_scale(_host(Xd))
    got = float(g.item())
    assert (np.isnan(want) and np.isnan(got)) or (np.isinf(want) and got == want)
    for Xin in (Xd, Xd.float()):                        # bf16 and fp32 sources take different amax paths
        g32 = float(nb.nvfp4_tensor_amax_scale(Xin).item())
        assert (np.isnan(want) and np.isnan(g32)) or g32 == want
    Y = nb.nvfp4_linear_fwd(Xd, Wd)
    dW = nb.nvfp4_linear_bwd_dw(dYd, Xd)
    dX = nb.nvfp4_linear_bwd_dx(dYd, Wd)
    Yf, saved = nb.nvfp4_linear_fwd_save(Xd, Wd)
    dXf, dWf = nb.nvfp4_linear_bwd_saved(dYd, saved, K)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    for t in (Y, dW, Yf, dWf):
        assert bool(torch.isnan(t).all())
    for t in (dX, dXf):                                 # dX = Q(dY) Q(W^T)^T does not involve X
        assert bool(torch.isfinite(t).all())
    # the oracle's dequantize-then-matmul says the same
    ref, _ = oracle_linear("fwd", Xd, Wd, nb.Rounding(nb.RTN), nb.Rounding(nb.RTN), True)
    assert np.all(np.isnan(ref))


# ---------------------------------------------------------------- a chain of layers without a high-precision intermediate
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", [(256, 512, 768, 256), (300, 288, 544, 200)])
def test_chained_layers_quantize_in_the_producer(shape, mode):
    # layer 1 writes Q(H) from its GEMM epilogue (nvfp4_linear_fwd_qout), layer 2 consumes it (nvfp4_linear_fwd_qin).
    # H itself (layer 1 through nvfp4_linear_fwd) is checked against the oracle's product; the quantized H must then
    # be the ORACLE's quantization of that H byte for byte, and the second product the oracle's product of those codes.
    M, K1, N1, N2 = shape
    X, W1, _ = synth.linear_inputs(M, K1, N1, seed=41)
    _, W2, _ = synth.linear_inputs(M, N1, N2, seed=42)
    X, W1, W2 = X.cuda(), W1.cuda(), W2.cuda()
    rt, ry = nb.Rounding(nb.RTN), nb.Rounding(mode, 77, 4)
    H = nb.nvfp4_linear_fwd(X, W1, rx=rt, rw=rt)
    ref, T = oracle_linear("fwd", X, W1, rt, rt, True)
    Hh = _host(H)
    _assert_close(Hh, ref, T)
    gh_t = nb.nvfp4_tensor_amax_scale(H)                  # the consumer's scale has to be known beforehand
    gh = ob.tensor_amax_scale(Hh)
    assert np.float32(gh) == np.float32(gh_t.item())
    hc, hs = nb.nvfp4_linear_fwd_qout(X, W1, gy=gh_t, ry=ry, rx=rt, rw=rt, sf_layout=nb.SF_SWIZZLED)
    Y = nb.nvfp4_linear_fwd_qin(hc, hs, gh_t, W2, rw=rt)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    oc, osf = ob.quantize(Hh, g=gh, mode=ry.mode, seed=ry.seed, offset=ry.offset)
    assert np.array_equal(hc.cpu().numpy(), oc)
    assert np.array_equal(hs.cpu().numpy().reshape(-1), ob.sf_swizzle(osf).reshape(-1))
    w2h = _host(W2)
    g2 = ob.tensor_amax_scale(w2h)
    wc, wsf = ob.quantize(w2h, g=g2)
    ref2, T2 = ob.gemm(oc, osf, gh, wc, wsf, g2)
    _assert_close(_host(Y), ref2, T2)
    # and the unfused pair (fp32 H, quantized by the next layer's own quantizer) gives the same bits when the
    # roundings agree (the next layer would use RtN on its input, Eq. 4)
    if mode == nb.RTN:
        Y_unfused = nb.nvfp4_linear_fwd(H, W2.float(), gscale_mode=nb.G_AMAX, rx=rt, rw=rt)   # bf16 -> fp32 is exact
        assert torch.equal(Y, Y_unfused)
