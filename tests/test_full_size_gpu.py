"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot multiply whole 7B-size tensors in seconds, but it can QUANTIZE them whole (a few
hundred million elements per second on the host cores).  So at full size:

  * every quantized operand is compared with the oracle byte for byte, codes and swizzled scales,
    over the whole tensor (through nvfp4_quantize_dual / nvfp4_quantize, the kernels the layer calls
    launch);
  * every product of the fused layer calls is compared with the oracle's dequantize-then-matmul at
    4096 random (i, j), two full rows, two full columns, and nine 32 x 32 blocks at the first, a
    middle (not tile-aligned) and the last rows of each operand.

Inputs are the seeded synthetic tensors of the benchmark (drawn on the device, copied to the host, so
that both sides see the same bytes).
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5
B = 32   # rows per checked block


def _host(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()


def _t(h: np.ndarray) -> np.ndarray:
    """Materialised transpose: the transposed quantization is by definition the row quantization of it."""
    return np.ascontiguousarray(h.T)


def _oq(h, g, r):
    return ob.quantize(h, g=g, mode=r.mode, seed=r.seed, offset=r.offset)


def _assert_operand_bytes(got_codes, got_scales, oc, osf, what):
    """Whole-tensor byte comparison: packed codes and scales in the 128 x 4 tile layout."""
    gc = got_codes.cpu().numpy()
    assert gc.shape == oc.shape, what
    bad = np.flatnonzero(gc.reshape(-1) != oc.reshape(-1))
    assert bad.size == 0, f"{what}: {bad.size} code bytes differ, first at {bad[:4]}"
    gs = got_scales.cpu().numpy().reshape(-1)
    want = ob.sf_swizzle(osf).reshape(-1)
    assert gs.shape == want.shape, what
    bad = np.flatnonzero(gs != want)
    assert bad.size == 0, f"{what}: {bad.size} scale bytes differ, first at {bad[:4]}"


def _samples(R, C, rng, n=4096):
    """n random (i, j), two full rows (first, a random one) and two full columns (last, a random one)."""
    rows = [0, int(rng.integers(1, R))]
    cols = [C - 1, int(rng.integers(0, C - 1))]
    ii = [rng.integers(0, R, n)] + [np.full(C, r) for r in rows] + [np.arange(R) for _ in cols]
    jj = [rng.integers(0, C, n)] + [np.arange(C) for _ in rows] + [np.full(R, c) for c in cols]
    return np.concatenate(ii), np.concatenate(jj)


def _assert_product(D, a, b, ga, gb, rng, what, mids):
    """D[R, C] (device) against the oracle product of whole quantized operands a = (codes, scales), b."""
    R, C = D.shape
    ii, jj = _samples(R, C, rng)
    ref, T = ob.gemm_sampled(a[0], a[1], ga, b[0], b[1], gb, ii, jj)
    got = D[torch.from_numpy(ii).cuda(), torch.from_numpy(jj).cuda()].float().cpu().numpy()
    err = np.abs(got - ref)
    bad = np.flatnonzero(err > TOL * T)
    assert bad.size == 0, f"{what}: {bad.size} of {err.size} samples beyond tolerance, max err/T {np.max(err / np.maximum(T, 1e-30)):.3e}"
    assert np.count_nonzero(ref) > ref.size // 2
    # blocks at the first, a middle and the last rows of each operand
    for r0, c0 in itertools.product((0, mids[0], R - B), (0, mids[1], C - B)):
        bref, bT = ob.gemm(a[0][r0:r0 + B], a[1][r0:r0 + B], ga, b[0][c0:c0 + B], b[1][c0:c0 + B], gb)
        bgot = D[r0:r0 + B, c0:c0 + B].float().cpu().numpy()
        assert np.all(np.abs(bgot - bref) <= TOL * bT), f"{what}[{r0}:, {c0}:]"


def _scale(t_dev, h):
    """Per-tensor scale: the GPU's value must be the oracle's, bit for bit."""
    g_t = nb.nvfp4_tensor_amax_scale(t_dev)
    g = ob.tensor_amax_scale(h)
    assert np.float32(g_t.item()) == np.float32(g)
    return g_t, g


def _layer_parity(M, K, N, seed, mids):
    """One linear layer at full size: operands byte for byte, the three products sampled."""
    X, W, dY = synth.linear_inputs(M, K, N, seed=seed, device="cuda")
    rt, sr = nb.Rounding(nb.RTN), [nb.Rounding(nb.SR, 0, o) for o in range(3)]
    Y, saved = nb.nvfp4_linear_fwd_save(X, W, nb.G_AMAX, rx=rt, rw=rt, rxt=sr[2], rwt=rt)
    dX, dW = nb.nvfp4_linear_bwd_saved(dY, saved, K, nb.G_AMAX, rdy=sr[0], rdyt=sr[1])
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    del saved
    rng = np.random.default_rng(seed)

    hX, hW, hdY = _host(X), _host(W), _host(dY)
    (gx_t, gx), (gw_t, gw), (gdy_t, gdy) = _scale(X, hX), _scale(W, hW), _scale(dY, hdY)

    # ---- the six quantization sites of Eq. 4-6, whole tensors, byte for byte ----
    qX, qW = _oq(hX, gx, rt), _oq(hW, gw, rt)                       # Eq. 4
    qdY, qWt = _oq(hdY, gdy, sr[0]), _oq(_t(hW), gw, rt)            # Eq. 5
    qdYt, qXt = _oq(_t(hdY), gdy, sr[1]), _oq(_t(hX), gx, sr[2])    # Eq. 6
    del hX, hW, hdY
    for t, g_t, r_row, r_t, o_row, o_t, name in ((X, gx_t, rt, sr[2], qX, qXt, "X"), (W, gw_t, rt, rt, qW, qWt, "W"),
                                                  (dY, gdy_t, sr[0], sr[1], qdY, qdYt, "dY")):
        cr, s_r, ct, s_t = nb.nvfp4_quantize_dual(t, g_t, r_row, r_t, nb.SF_SWIZZLED)
        torch.cuda.synchronize()
        _assert_operand_bytes(cr, s_r, *o_row, f"Q({name})")
        _assert_operand_bytes(ct, s_t, *o_t, f"Q({name}^T)")
        del cr, s_r, ct, s_t
    assert nb.nvfp4_device_error_word() == 0

    # ---- the three products of Eq. 1-3 from the fused layer calls ----
    _assert_product(Y, qX, qW, gx, gw, rng, "Y", (mids[0], mids[2]))
    _assert_product(dX, qdY, qWt, gdy, gw, rng, "dX", (mids[0], mids[1]))
    _assert_product(dW, qdYt, qXt, gdy, gx, rng, "dW", (mids[2], mids[1]))


# middle starts of the 32-row blocks (tokens, K, N): not aligned to 128 or 256
_MIDS = {4096: 2072, 11008: 5528, 12288: 6168, 1024: 520, 2816: 1416, 3072: 1544, 16384: 8200}


@pytest.mark.parametrize("name,K,N", synth.LLAMA_7B["linears"])
def test_llama7b_block_linear(name, K, N):
    M = synth.LLAMA_7B["tokens"]
    seed = 1004 + [n for n, _, _ in synth.LLAMA_7B["linears"]].index(name)
    _layer_parity(M, K, N, seed, (_MIDS[M], _MIDS[K], _MIDS[N]))


@pytest.mark.parametrize("name,K,N", synth.LLAMA_350M["linears"])
def test_llama350m_block_linear(name, K, N):
    M = synth.LLAMA_350M["tokens"]
    seed = 1003 + 10 * [n for n, _, _ in synth.LLAMA_350M["linears"]].index(name)
    _layer_parity(M, K, N, seed, (_MIDS[M], _MIDS[K], _MIDS[N]))


def test_ffn_weight_gradient_with_long_token_axis():
    # dW = dY^T X with dY 65536 x 11008 and X 65536 x 4096, both SR (seed 2) in blocks along the tokens
    M, N, K = 65536, 11008, 4096
    dY = synth.normal((M, N), 1e-4, 2005, device="cuda")
    X = synth.normal((M, K), 1.0, 2006, device="cuda")
    r_dy, r_x = nb.Rounding(nb.SR, 2, 1), nb.Rounding(nb.SR, 2, 2)
    dW = nb.nvfp4_linear_bwd_dw(dY, X, nb.G_AMAX, rdy=r_dy, rx=r_x)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    rng = np.random.default_rng(2005)
    hdY, hX = _host(dY), _host(X)
    (gdy_t, gdy), (gx_t, gx) = _scale(dY, hdY), _scale(X, hX)
    qdYt = _oq(_t(hdY), gdy, r_dy)
    del hdY
    qXt = _oq(_t(hX), gx, r_x)
    del hX
    for t, g_t, r, o, name in ((dY, gdy_t, r_dy, qdYt, "dY"), (X, gx_t, r_x, qXt, "X")):
        c, s = nb.nvfp4_quantize(t, True, g_t, r, nb.SF_SWIZZLED)
        torch.cuda.synchronize()
        _assert_operand_bytes(c, s, *o, f"Q({name}^T)")
        del c, s
    _assert_product(dW, qdYt, qXt, gdy, gx, rng, "dW", (5528, 2072))


def test_quantizer_sweep_at_2p28_elements():
    # the size every quantizer bandwidth figure is quoted on: 0.05 * Student-t(3) with 0.1 % outliers x 100,
    # row and transposed, RtN and SR (seed 1), and both orientations from one read; whole tensor, every byte
    x = synth.heavy_tailed(synth.square_shape(2 ** 28), seed=1002, device="cuda")
    h = _host(x)
    g_t, g = _scale(x, h)
    rt, sr0, sr1 = nb.Rounding(nb.RTN), nb.Rounding(nb.SR, 1, 0), nb.Rounding(nb.SR, 1, 1)
    want = {("row", "rtn"): _oq(h, g, rt), ("row", "sr0"): _oq(h, g, sr0)}
    h = _t(h)
    want.update({("t", "rtn"): _oq(h, g, rt), ("t", "sr0"): _oq(h, g, sr0), ("t", "sr1"): _oq(h, g, sr1)})
    del h
    for (orient, rname), r in ((("row", "rtn"), rt), (("row", "sr0"), sr0), (("t", "rtn"), rt), (("t", "sr0"), sr0)):
        c, s = nb.nvfp4_quantize(x, orient == "t", g_t, r, nb.SF_SWIZZLED)
        torch.cuda.synchronize()
        _assert_operand_bytes(c, s, *want[(orient, rname)], f"{orient} {rname}")
        del c, s
    for r_row, r_t, k_row, k_t in ((rt, rt, "rtn", "rtn"), (sr0, sr1, "sr0", "sr1")):
        cr, s_r, ct, s_t = nb.nvfp4_quantize_dual(x, g_t, r_row, r_t, nb.SF_SWIZZLED)
        torch.cuda.synchronize()
        _assert_operand_bytes(cr, s_r, *want[("row", k_row)], f"dual row {k_row}")
        _assert_operand_bytes(ct, s_t, *want[("t", k_t)], f"dual transposed {k_t}")
        del cr, s_r, ct, s_t
    assert nb.nvfp4_device_error_word() == 0


def test_chained_up_and_down_projection_at_llama7b_size():
    # the chain bench.py times: the up projection's product leaves its GEMM quantized (nvfp4_linear_fwd_qout) and feeds
    # the down projection (nvfp4_linear_fwd_qin).  The fp32 product of the same layer is sampled against the oracle; the
    # quantized product must then be the oracle's quantization of that fp32 product over the whole tensor, byte for
    # byte, and the second product the oracle's product of those codes at the sampled positions.
    M, K1, N1, N2 = synth.LLAMA_7B["tokens"], 4096, 11008, 4096
    X, W1, _ = synth.linear_inputs(M, K1, N1, seed=1021, device="cuda")
    _, W2, _ = synth.linear_inputs(M, N1, N2, seed=1022, device="cuda")
    rt = nb.Rounding(nb.RTN)
    rng = np.random.default_rng(1021)
    H = nb.nvfp4_linear_fwd(X, W1, rx=rt, rw=rt)
    hX, hW1 = _host(X), _host(W1)
    (gx_t, gx), (g1_t, g1) = _scale(X, hX), _scale(W1, hW1)
    _assert_product(H, _oq(hX, gx, rt), _oq(hW1, g1, rt), gx, g1, rng, "H", (_MIDS[M], _MIDS[N1]))
    del hX, hW1
    hH = H.cpu().numpy()
    gh_t, gh = _scale(H, hH)
    hc, hs = nb.nvfp4_linear_fwd_qout(X, W1, gy=gh_t, ry=rt, rx=rt, rw=rt, sf_layout=nb.SF_SWIZZLED)
    Y = nb.nvfp4_linear_fwd_qin(hc, hs, gh_t, W2, rw=rt)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    qH = _oq(hH, gh, rt)
    del hH
    _assert_operand_bytes(hc, hs, *qH, "Q(H) from the GEMM epilogue")
    hW2 = _host(W2)
    g2_t, g2 = _scale(W2, hW2)
    _assert_product(Y, qH, _oq(hW2, g2, rt), gh, g2, rng, "Y", (_MIDS[M], _MIDS[N2]))
