"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot quantize and multiply whole 7B-size tensors in seconds, so these tests check
blocks of outputs whose operand slices it can compute one by one: an output block D[r0:r0+32,
c0:c0+32] of a GEMM depends only on 32 quantized rows of each operand, and a quantized row depends
only on one row (or, for the transposed quantizations, one column) of the source tensor, the
per-tensor scale, and its own row index (which keys the random integers).  Blocks are taken at the
first, a middle (not tile-aligned) and the last rows of every operand.
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
B = 32   # rows per checked slice


def _g(t: torch.Tensor) -> float:
    """Oracle per-tensor scale of a full host tensor: its largest magnitude (library max) fed to the oracle's rule."""
    amax = float(t.abs().max().float())
    return ob.tensor_amax_scale(np.array([amax], dtype=np.float32))


def _rows(t: torch.Tensor, r0: int) -> np.ndarray:
    return t[r0:r0 + B].float().numpy()


def _cols_as_rows(t: torch.Tensor, c0: int) -> np.ndarray:
    return np.ascontiguousarray(t[:, c0:c0 + B].float().numpy().T)


def _starts(n: int, mid: int):
    return [0, mid, n - B]


def _check_blocks(D: torch.Tensor, a_slices, b_slices, ga, gb, what):
    """a_slices / b_slices: {start: (codes, scales)} of 32 quantized rows each."""
    for (r0, (ac, asf)), (c0, (bc, bsf)) in itertools.product(a_slices.items(), b_slices.items()):
        ref, T = ob.gemm(ac, asf, ga, bc, bsf, gb)
        got = D[r0:r0 + B, c0:c0 + B].float().cpu().numpy()
        err = np.abs(got - ref)
        assert np.all(err <= TOL * T), f"{what}[{r0}:, {c0}:] max err/T {np.max(err / np.maximum(T, 1e-30)):.3e}"
        assert np.any(ref != 0)


def test_llama7b_down_projection_fused_layer():
    # tokens 16384, down projection 11008 -> 4096: the layer with the longest forward contraction
    M, K, N = synth.LLAMA_7B["tokens"], 11008, 4096
    X, W, dY = synth.linear_inputs(M, K, N, seed=1004)
    rt, sr = nb.Rounding(nb.RTN), [nb.Rounding(nb.SR, 0, o) for o in range(3)]
    Xd, Wd, dYd = X.cuda(), W.cuda(), dY.cuda()
    Y, saved = nb.nvfp4_linear_fwd_save(Xd, Wd, nb.G_AMAX, rx=rt, rw=rt, rxt=sr[2], rwt=rt)
    dX, dW = nb.nvfp4_linear_bwd_saved(dYd, saved, K, nb.G_AMAX, rdy=sr[0], rdyt=sr[1])
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    gx, gw, gdy = _g(X), _g(W), _g(dY)
    ms, ns, ks = _starts(M, 8200), _starts(N, 2072), _starts(K, 5528)

    # Eq. 1/4: Y = Q(X) Q(W)^T, blocks along K
    xa = {m: ob.quantize_rows(_rows(X, m), m, g=gx) for m in ms}
    wb = {n: ob.quantize_rows(_rows(W, n), n, g=gw) for n in ns}
    _check_blocks(Y, xa, wb, gx, gw, "Y")
    # two full rows of Y against the whole of Q(W)
    wc, wsf = ob.quantize(W.float().numpy(), g=gw)
    for m in (0, M - 1):
        ac, asf = ob.quantize_rows(X[m:m + 1].float().numpy(), m, g=gx)
        ref, T = ob.gemm(ac, asf, gx, wc, wsf, gw)
        assert np.all(np.abs(Y[m:m + 1].cpu().numpy() - ref) <= TOL * T)

    # Eq. 2/5: dX = Q_SR(dY) Q_RtN(W^T)^T, blocks along N
    dya = {m: ob.quantize_rows(_rows(dY, m), m, g=gdy, mode=ob.SR, seed=0, offset=0) for m in ms}
    wtb = {k: ob.quantize_rows(_cols_as_rows(W, k), k, g=gw) for k in ks}
    _check_blocks(dX, dya, wtb, gdy, gw, "dX")

    # Eq. 3/6: dW = Q_SR(dY^T) Q_SR(X^T)^T, blocks along the token axis
    dyta = {n: ob.quantize_rows(_cols_as_rows(dY, n), n, g=gdy, mode=ob.SR, seed=0, offset=1) for n in ns}
    xtb = {k: ob.quantize_rows(_cols_as_rows(X, k), k, g=gx, mode=ob.SR, seed=0, offset=2) for k in ks}
    _check_blocks(dW, dyta, xtb, gdy, gx, "dW")


def test_ffn_weight_gradient_with_long_token_axis():
    # dW = dY^T X with dY 65536 x 11008 and X 65536 x 4096, both SR (seed 2) in blocks along the tokens
    M, N, K = 65536, 11008, 4096
    dY = synth.normal((M, N), 1e-4, 2005, device="cpu")
    X = synth.normal((M, K), 1.0, 2006, device="cpu")
    r_dy, r_x = nb.Rounding(nb.SR, 2, 1), nb.Rounding(nb.SR, 2, 2)
    dW = nb.nvfp4_linear_bwd_dw(dY.cuda(), X.cuda(), nb.G_AMAX, rdy=r_dy, rx=r_x)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    gdy, gx = _g(dY), _g(X)
    dyta = {n: ob.quantize_rows(_cols_as_rows(dY, n), n, g=gdy, mode=ob.SR, seed=2, offset=1) for n in _starts(N, 5528)}
    xtb = {k: ob.quantize_rows(_cols_as_rows(X, k), k, g=gx, mode=ob.SR, seed=2, offset=2) for k in _starts(K, 2072)}
    _check_blocks(dW, dyta, xtb, gdy, gx, "dW")
