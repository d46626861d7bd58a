"""MXFP4 variant (Section 3, Table 1: blocks of 32, E8M0 scales) through the same kernels: quantizer
bit-exact against the oracle, GEMM within 1e-5 * sum|a_i b_i|, the three products of a layer."""
import numpy as np
import pytest
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _h(t):
    return t.float().cpu().numpy()


def _swz(sf_lin):
    return ob.sf_swizzle(sf_lin)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", [(1, 32), (130, 96), (128, 512), (257, 1056), (129, 4128)])
def test_row_quantizer_matches_the_oracle(shape, mode, sf_layout, dtype):
    x = synth.normal(shape, 1.0, 3, device="cpu", dtype=dtype).cuda()
    r = nb.Rounding(mode, 12, 7)
    for use_g in (False, True):
        g_t = nb.nvfp4_tensor_amax_scale(x) if use_g else None
        g = float(g_t.item()) if use_g else 1.0
        codes, scales = nb.nvfp4_quantize_mx(x, False, g_t, r, sf_layout)
        oc, osf = ob.quantize_mx(_h(x), g=g, mode=mode, seed=12, offset=7)
        assert np.array_equal(codes.cpu().numpy(), oc)
        want = _swz(osf) if sf_layout == nb.SF_SWIZZLED else osf
        assert np.array_equal(scales.cpu().numpy().reshape(-1), want.reshape(-1))


@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", [(32, 8), (64, 72), (512, 200), (1056, 264), (288, 136), (2048, 1024)])
def test_transposed_quantizer_matches_the_oracle(shape, mode, sf_layout):
    # blocks of 32 along the rows, straight from the source tile (no transpose pass): ragged tiles in both directions
    x = synth.normal(shape, 1e-3, 4, device="cpu").cuda()
    g_t = nb.nvfp4_tensor_amax_scale(x)
    r = nb.Rounding(mode, 2, 1)
    codes, scales = nb.nvfp4_quantize_mx(x, True, g_t, r, sf_layout)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    oc, osf = ob.quantize_mx(_h(x), g=float(g_t.item()), mode=mode, seed=2, offset=1, transposed=True)
    assert np.array_equal(codes.cpu().numpy(), oc)
    want = _swz(osf) if sf_layout == nb.SF_SWIZZLED else osf
    assert np.array_equal(scales.cpu().numpy().reshape(-1), want.reshape(-1))


def test_transposed_special_blocks_and_no_global_scale():
    x = torch.zeros((64, 16), dtype=torch.float32)
    x[:8, 0] = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0])   # amax 6 -> scale 1, the tie points
    x[32:40, 1] = -x[:8, 0]
    x[5, 2] = -0.0
    x[0, 3] = 3.0                                                            # amax/6 = 0.5 exactly: a power of two
    x[0, 4] = 3.0001
    x[:32, 5] = 1e-30
    x[40, 6] = 1e30
    xs = x.to(torch.bfloat16).cuda()
    for mode in (nb.RTN, nb.SR):
        codes, scales = nb.nvfp4_quantize_mx(xs, True, None, nb.Rounding(mode, 3, 3), nb.SF_LINEAR)
        oc, osf = ob.quantize_mx(_h(xs), mode=mode, seed=3, offset=3, transposed=True)
        assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(scales.cpu().numpy(), osf)


def test_special_blocks():
    x = torch.zeros((8, 64), dtype=torch.float32)
    x[0, :8] = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0])   # amax 6 -> scale 1, the tie points
    x[1, 32:40] = -x[0, :8]
    x[2, 5] = -0.0
    x[3, 0] = 3.0                                                            # amax/6 = 0.5 exactly: a power of two
    x[4, 0] = 3.0001
    x[5, :32] = 1e-30
    x[6, 0] = 1e30
    for dt in (torch.bfloat16, torch.float32):
        xs = x.to(dt).cuda()
        for mode in (nb.RTN, nb.SR):
            codes, scales = nb.nvfp4_quantize_mx(xs, False, None, nb.Rounding(mode, 3, 3), nb.SF_LINEAR)
            oc, osf = ob.quantize_mx(_h(xs), mode=mode, seed=3, offset=3)
            assert np.array_equal(codes.cpu().numpy(), oc) and np.array_equal(scales.cpu().numpy(), osf)


def _pair(M, N, K, seed):
    A = synth.normal((M, K), 1.0, seed, device="cpu").cuda()
    B = synth.normal((N, K), 0.02, seed + 1, device="cpu").cuda()
    ga, gb = nb.nvfp4_tensor_amax_scale(A), nb.nvfp4_tensor_amax_scale(B)
    ac, asf = nb.nvfp4_quantize_mx(A, False, ga, None, nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize_mx(B, False, gb, None, nb.SF_SWIZZLED)
    oa = ob.quantize_mx(_h(A), g=float(ga.item()))
    obq = ob.quantize_mx(_h(B), g=float(gb.item()))
    return (ac, asf, ga, bc, bsf, gb), (oa[0], oa[1], float(ga.item()), obq[0], obq[1], float(gb.item()))


def test_gemm_one_hot_rows_read_back_the_dequantized_operand():
    # a row of A with a single 6.0 (scale 1) selects one column of dequantized B: any mistake in the
    # scale-tile layout or in which half of a scale column an instruction uses shows up exactly
    M, N, K = 256, 384, 512
    A = torch.zeros((M, K), dtype=torch.float32)
    for m in range(M):
        A[m, (m * 37) % K] = 6.0
    B = synth.normal((N, K), 1.0, 5, device="cpu").float()
    ac, asf = nb.nvfp4_quantize_mx(A.cuda(), False, None, None, nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize_mx(B.cuda(), False, None, None, nb.SF_SWIZZLED)
    D = nb.nvfp4_gemm_mx(ac, asf, None, bc, bsf, None).cpu().numpy()
    assert nb.nvfp4_device_error_word() == 0
    deqB = ob.dequantize_mx(*ob.quantize_mx(B.numpy()))
    want = np.stack([6.0 * deqB[:, (m * 37) % K] for m in range(M)])
    assert np.array_equal(D, want)


@pytest.mark.parametrize("shape", [(256, 256, 256), (130, 136, 320), (257, 392, 1056), (1, 8, 32), (384, 520, 2080), (128, 128, 16384)])
def test_gemm_within_tolerance(shape):
    M, N, K = shape
    gpu_ops, ora_ops = _pair(M, N, K, 10 + M)
    D = nb.nvfp4_gemm_mx(*gpu_ops)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    ref, T = ob.gemm_mx(*ora_ops)
    err = np.abs(_h(D) - ref)
    assert np.all(err <= TOL * T), f"max err/T {np.max(err / np.maximum(T, 1e-30)):.3e}"
    Db = nb.nvfp4_gemm_mx(*gpu_ops, out_dtype=torch.bfloat16)
    assert np.all(np.abs(_h(Db) - ref) <= TOL * T + np.abs(ref) * 2.0 ** -8)


def test_three_products_of_a_layer_in_mxfp4():
    # Eq. 1-6 with the MXFP4 format: the single-layer shapes
    t = synth.TINY_LINEAR
    M, K, N = t["tokens"], t["K"], t["N"]
    X, W, dY = synth.linear_inputs(M, K, N, seed=1001, grad_std=1e-3)
    Xd, Wd, dYd = X.cuda(), W.cuda(), dY.cuda()
    g = {k: nb.nvfp4_tensor_amax_scale(v) for k, v in (("x", Xd), ("w", Wd), ("dy", dYd))}
    gf = {k: float(v.item()) for k, v in g.items()}
    rt, sr = nb.Rounding(nb.RTN), [nb.Rounding(nb.SR, 0, o) for o in range(3)]

    def q(t_, tr, gk, r):
        return nb.nvfp4_quantize_mx(t_, tr, g[gk], r, nb.SF_SWIZZLED)

    def oq(t_, tr, gk, r):
        return ob.quantize_mx(_h(t_), g=gf[gk], mode=r.mode, seed=r.seed, offset=r.offset, transposed=tr)

    for name, (a, ta, ga, ra), (b, tb, gb, rb) in (
            ("Y", (Xd, False, "x", rt), (Wd, False, "w", rt)),
            ("dX", (dYd, False, "dy", sr[0]), (Wd, True, "w", rt)),
            ("dW", (dYd, True, "dy", sr[1]), (Xd, True, "x", sr[2]))):
        ac, asf = q(a, ta, ga, ra)
        bc, bsf = q(b, tb, gb, rb)
        D = nb.nvfp4_gemm_mx(ac, asf, g[ga], bc, bsf, g[gb])
        oa, ob_ = oq(a, ta, ga, ra), oq(b, tb, gb, rb)
        assert np.array_equal(ac.cpu().numpy(), oa[0]) and np.array_equal(bc.cpu().numpy(), ob_[0]), name
        ref, T = ob.gemm_mx(oa[0], oa[1], gf[ga], ob_[0], ob_[1], gf[gb])
        assert np.all(np.abs(_h(D) - ref) <= TOL * T), name
        assert float(D.abs().max()) > 0.0
