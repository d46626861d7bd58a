"""QAF phase (Section 5): backward and update products in BF16 on the CTA-pair tensor-core kernel."""
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


@pytest.mark.parametrize("shape", [(256, 256, 64), (256, 256, 512), (300, 520, 336), (1000, 1304, 1040), (16, 8, 16), (128, 128, 65536)])
def test_gemm_bf16_within_tolerance(shape):
    M, N, K = shape
    A = synth.normal((M, K), 1.0, 5, device="cpu").cuda()
    B = synth.normal((N, K), 0.02, 6, device="cpu").cuda()
    D = nb.nvfp4_gemm_bf16(A, B)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    ref, T = ob.matmul_nt(_h(A), _h(B))
    err = np.abs(_h(D) - ref)
    assert np.all(err <= TOL * T), f"max err/T {np.max(err / np.maximum(T, 1e-30)):.3e}"
    Db = nb.nvfp4_gemm_bf16(A, B, out_dtype=torch.bfloat16)
    assert np.all(np.abs(_h(Db) - ref) <= TOL * T + np.abs(ref) * 2.0 ** -8)


def test_gemm_bf16_exact_on_small_integers():
    rng = np.random.default_rng(1)
    A = torch.from_numpy(rng.integers(-4, 5, (256, 128)).astype(np.float32)).to(torch.bfloat16).cuda()
    B = torch.from_numpy(rng.integers(-4, 5, (384, 128)).astype(np.float32)).to(torch.bfloat16).cuda()
    D = nb.nvfp4_gemm_bf16(A, B)
    assert np.array_equal(_h(D), _h(A).astype(np.float64) @ _h(B).astype(np.float64).T)


@pytest.mark.parametrize("shape", [(64, 64), (200, 72), (8, 8), (1000, 520)])
def test_transpose_bf16_is_exact(shape):
    x = synth.normal(shape, 1.0, 9, device="cpu").cuda()
    assert torch.equal(nb.nvfp4_transpose_bf16(x), x.t().contiguous())
    wide = synth.normal((shape[0], shape[1] + 16), 1.0, 10, device="cpu").cuda()
    assert torch.equal(nb.nvfp4_transpose_bf16(wide[:, 8:8 + shape[1]]), wide[:, 8:8 + shape[1]].t().contiguous())


@pytest.mark.parametrize("shape", [(256, 512, 512), (160, 288, 208)])
def test_backward_and_update_in_bf16(shape):
    M, K, N = shape
    X, W, dY = synth.linear_inputs(M, K, N, seed=41, grad_std=1e-3)
    Xd, Wd, dYd = X.cuda(), W.cuda(), dY.cuda()
    dX, dW = nb.nvfp4_linear_bwd_bf16(dYd, Wd, Xd)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    ref, T = ob.matmul_nt(_h(dY), np.ascontiguousarray(_h(W).T))           # dX = dY . W
    assert np.all(np.abs(_h(dX) - ref) <= TOL * T)
    ref, T = ob.matmul_nt(np.ascontiguousarray(_h(dY).T), np.ascontiguousarray(_h(X).T))   # dW = dY^T . X
    assert np.all(np.abs(_h(dW) - ref) <= TOL * T)


# ---------------------------------------------------------------- operands read as they are stored (no transposed copies)
@pytest.mark.parametrize("majors", [(0, 1), (1, 1)])
@pytest.mark.parametrize("shape", [(256, 256, 64), (256, 512, 512), (304, 520, 336), (1000, 1304, 1040), (16, 8, 16), (128, 128, 16384)])
def test_gemm_bf16_mn_major_operands(shape, majors):
    # an MN-major operand is the [K, M] (or [K, N]) array: the product must equal the one on its transpose
    M, N, K = shape
    a_mn, b_mn = majors
    A = synth.normal((M, K), 1.0, 15, device="cpu")
    B = synth.normal((N, K), 0.02, 16, device="cpu")
    Ad = (A.t().contiguous() if a_mn else A).cuda()
    Bd = (B.t().contiguous() if b_mn else B).cuda()
    D = nb.nvfp4_gemm_bf16_ex(Ad, a_mn, Bd, b_mn)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    ref, T = ob.matmul_nt(_h(A), _h(B))
    err = np.abs(_h(D) - ref)
    assert np.all(err <= TOL * T), f"max err/T {np.max(err / np.maximum(T, 1e-30)):.3e}"
    # the same instruction order as the K-major kernel: identical bits
    assert torch.equal(D, nb.nvfp4_gemm_bf16(A.cuda(), B.cuda()))


def test_gemm_bf16_mn_major_exact_and_one_hot():
    rng = np.random.default_rng(2)
    A = torch.from_numpy(rng.integers(-4, 5, (256, 192)).astype(np.float32)).to(torch.bfloat16)
    B = torch.from_numpy(rng.integers(-4, 5, (384, 192)).astype(np.float32)).to(torch.bfloat16)
    want = _h(A).astype(np.float64) @ _h(B).astype(np.float64).T
    for a_mn, b_mn in ((0, 1), (1, 1)):
        Ad = (A.t().contiguous() if a_mn else A).cuda()
        D = nb.nvfp4_gemm_bf16_ex(Ad, a_mn, B.t().contiguous().cuda(), b_mn)
        assert np.array_equal(_h(D), want)
    # one-hot rows of A pick single columns of B^T: any error in the MN-major box layout or descriptor strides shows exactly
    M, N, K = 256, 320, 256
    A1 = torch.zeros((M, K), dtype=torch.bfloat16)
    for m in range(M):
        A1[m, (m * 37) % K] = 1.0
    B1 = synth.normal((N, K), 1.0, 21, device="cpu")
    D = nb.nvfp4_gemm_bf16_ex(A1.t().contiguous().cuda(), 1, B1.t().contiguous().cuda(), 1)
    want = np.stack([_h(B1)[:, (m * 37) % K] for m in range(M)])
    assert np.array_equal(_h(D), want)


def test_backward_and_update_in_bf16_at_layer_size():
    # Llama-7B O projection: dX and dW sampled against the oracle
    M, K, N = 16384, 4096, 4096
    X, W, dY = synth.linear_inputs(M, K, N, seed=43, device="cuda", grad_std=1e-3)
    dX, dW = nb.nvfp4_linear_bwd_bf16(dY, W, X)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    rng = np.random.default_rng(3)
    hX, hW, hdY = _h(X), _h(W), _h(dY)
    ii, jj = rng.integers(0, M, 512), rng.integers(0, K, 512)
    ref = np.einsum("sn,ns->s", hdY[ii].astype(np.float64), hW[:, jj].astype(np.float64))
    T = np.einsum("sn,ns->s", np.abs(hdY[ii]).astype(np.float64), np.abs(hW[:, jj]).astype(np.float64))
    assert np.all(np.abs(_h(dX)[ii, jj] - ref) <= TOL * T + 1e-30)
    ii, jj = rng.integers(0, N, 256), rng.integers(0, K, 256)
    ref = np.einsum("ms,ms->s", hdY[:, ii].astype(np.float64), hX[:, jj].astype(np.float64))
    T = np.einsum("ms,ms->s", np.abs(hdY[:, ii]).astype(np.float64), np.abs(hX[:, jj]).astype(np.float64))
    assert np.all(np.abs(_h(dW)[ii, jj] - ref) <= TOL * T + 1e-30)
