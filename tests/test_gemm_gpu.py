"""GPU-vs-oracle parity of the block-scaled GEMM: |gpu - oracle| <= 1e-5 * sum|a_i b_i| elementwise,
exact equality where every partial sum is exactly representable."""
import numpy as np
import pytest
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _quantized_pair(M, N, K, seed, a_std=1.0, b_std=0.02, use_g=True, sr=False):
    A = synth.normal((M, K), a_std, seed, device="cpu").cuda()
    B = synth.normal((N, K), b_std, seed + 1, device="cpu").cuda()
    ga = nb.nvfp4_tensor_amax_scale(A) if use_g else None
    gb = nb.nvfp4_tensor_amax_scale(B) if use_g else None
    r = nb.Rounding(nb.SR, 3, 1) if sr else nb.Rounding()
    ac, asf = nb.nvfp4_quantize(A, global_scale=ga, rounding=r, sf_layout=nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize(B, global_scale=gb, rounding=r, sf_layout=nb.SF_SWIZZLED)
    # the oracle consumes linear scales produced by the oracle's own quantizer (bit-identical
    # to the GPU's, which the quantizer parity tests establish)
    gaf = float(ga.item()) if use_g else 1.0
    gbf = float(gb.item()) if use_g else 1.0
    oac, oasf = ob.quantize(A.float().cpu().numpy(), g=gaf, mode=r.mode, seed=r.seed, offset=r.offset)
    obc, obsf = ob.quantize(B.float().cpu().numpy(), g=gbf, mode=r.mode, seed=r.seed, offset=r.offset)
    assert np.array_equal(oac, ac.cpu().numpy()) and np.array_equal(obc, bc.cpu().numpy())
    return (ac, asf, ga, bc, bsf, gb), (oac, oasf, gaf, obc, obsf, gbf)


def _check(gpu_ops, ora_ops, out_dtype=torch.float32):
    D = nb.nvfp4_gemm(*gpu_ops, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    ref, T = ob.gemm(*ora_ops)
    got = D.float().cpu().numpy()
    if out_dtype == torch.bfloat16:
        assert np.all(np.abs(got - ref) <= TOL * T + np.abs(ref) * 2.0 ** -8)
    else:
        err = np.abs(got - ref)
        bad = np.argwhere(err > TOL * T)
        assert bad.size == 0, f"{bad.shape[0]} of {err.size} outputs beyond tolerance, first {bad[:3]}, " \
                              f"max ratio {np.max(err / np.maximum(T, 1e-30)):.3e}"
    return got, ref


@pytest.fixture(params=[128, 256, 2128, 2192, 2256])
def tile_n(request):
    nb.nvfp4_gemm_set_tile_n(request.param)
    yield request.param
    nb.nvfp4_gemm_set_tile_n(0)


def test_one_hot_rows_read_back_dequantized_operand(tile_n):
    # A row with a single 6.0 (scale 1, code 7) selects one column of dequantized B: any error in
    # the scale-tile layout, the operand descriptors or the nibble order shows up exactly.
    M, N, K = 256, 384, 512
    A = torch.zeros((M, K), dtype=torch.float32)
    for m in range(M):
        A[m, (m * 37) % K] = 6.0
    B = synth.normal((N, K), 1.0, 5, device="cpu").float()
    ac, asf = nb.nvfp4_quantize(A.cuda(), sf_layout=nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize(B.cuda(), sf_layout=nb.SF_SWIZZLED)
    D = nb.nvfp4_gemm(ac, asf, None, bc, bsf, None).cpu().numpy()
    assert nb.nvfp4_device_error_word() == 0
    obc, obsf = ob.quantize(B.numpy())
    deqB = ob.dequantize(obc, obsf)
    want = np.stack([6.0 * deqB[:, (m * 37) % K] for m in range(M)])
    assert np.array_equal(D, want)


def test_exact_when_all_partial_sums_are_representable(tile_n):
    rng = np.random.default_rng(0)
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.5, -1, -1.5, -2, -3, -4, -6], dtype=np.float32)
    M, N, K = 128, 256, 256
    A = rng.choice(grid, size=(M, K)).astype(np.float32)
    B = rng.choice(grid, size=(N, K)).astype(np.float32)
    A[:, ::16] = 6.0
    B[:, ::16] = -6.0                                  # every block has amax 6 -> scale exactly 1
    ac, asf = nb.nvfp4_quantize(torch.from_numpy(A).cuda(), sf_layout=nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize(torch.from_numpy(B).cuda(), sf_layout=nb.SF_SWIZZLED)
    D = nb.nvfp4_gemm(ac, asf, None, bc, bsf, None).cpu().numpy()
    assert np.array_equal(D, (A.astype(np.float64) @ B.astype(np.float64).T).astype(np.float32))


@pytest.mark.parametrize("shape", [(128, 128, 256), (256, 256, 512), (130, 136, 320), (257, 392, 1056),
                                   (1, 8, 32), (64, 200, 96), (384, 520, 2080)])
def test_random_operands_within_tolerance(shape, tile_n):
    M, N, K = shape
    gpu_ops, ora_ops = _quantized_pair(M, N, K, seed=10 + M)
    _check(gpu_ops, ora_ops)


def test_stochastically_rounded_operands_and_no_global_scale(tile_n):
    gpu_ops, ora_ops = _quantized_pair(256, 256, 512, seed=40, b_std=1.0, use_g=False, sr=True)
    _check(gpu_ops, ora_ops)


def test_bf16_output(tile_n):
    gpu_ops, ora_ops = _quantized_pair(256, 256, 512, seed=50)
    _check(gpu_ops, ora_ops, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("K", [64, 256, 1024, 4096, 16384, 65536])
def test_error_stays_under_tolerance_as_K_grows(K):
    # detects reduced-precision accumulation in the tensor core: the oracle accumulates in double
    gpu_ops, ora_ops = _quantized_pair(128, 128, K, seed=60, b_std=1.0)
    got, ref = _check(gpu_ops, ora_ops)


def test_many_tiles_persistent_schedule():
    # more tiles than SMs, ragged edges in both directions
    gpu_ops, ora_ops = _quantized_pair(2000, 2600, 512, seed=70)
    D = nb.nvfp4_gemm(*gpu_ops)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    rng = np.random.default_rng(1)
    ii = np.concatenate([rng.integers(0, 2000, 4096), np.full(2600, 1999), np.arange(2000)])
    jj = np.concatenate([rng.integers(0, 2600, 4096), np.arange(2600), np.full(2000, 2599)])
    ref, T = ob.gemm_sampled(*ora_ops, ii, jj)
    got = D.cpu().numpy()[ii, jj]
    assert np.all(np.abs(got - ref) <= TOL * T)


# ---------------------------------------------------------------- quantization fused into the epilogue
@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", [(256, 256, 256), (300, 544, 512), (1000, 1312, 1056), (64, 32, 64)])
def test_quantized_epilogue_equals_quantizing_the_fp32_product(shape, mode, sf_layout):
    M, N, K = shape
    gpu_ops, ora_ops = _quantized_pair(M, N, K, seed=90 + M)
    D = nb.nvfp4_gemm(*gpu_ops)
    g_out = nb.nvfp4_tensor_amax_scale(D)
    r = nb.Rounding(mode, 17, 3)
    want_c, want_s = nb.nvfp4_quantize(D, False, g_out, r, sf_layout)
    got_c, got_s = nb.nvfp4_gemm_quantized(*gpu_ops, out_global_scale=g_out, rounding=r, sf_layout=sf_layout)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    assert torch.equal(got_c, want_c)
    assert torch.equal(got_s.reshape(-1), want_s.reshape(-1))
    # oracle-anchored: the oracle's quantization of the host copy of D (itself within tolerance of the oracle's
    # product, checked below), with the oracle's per-tensor scale, byte for byte
    Dh = D.cpu().numpy()
    g = ob.tensor_amax_scale(Dh)
    assert np.float32(g) == np.float32(g_out.item())
    oc, osf = ob.quantize(Dh, g=g, mode=r.mode, seed=r.seed, offset=r.offset)
    assert np.array_equal(got_c.cpu().numpy(), oc)
    want_sf = osf if sf_layout == nb.SF_LINEAR else ob.sf_swizzle(osf)
    assert np.array_equal(got_s.cpu().numpy().reshape(-1), want_sf.reshape(-1))
    ref, T = ob.gemm(*ora_ops)
    assert np.all(np.abs(Dh - ref) <= TOL * T)
    if sf_layout == nb.SF_LINEAR:
        # against the oracle's product: every dequantized output within one grid step (two under SR) of it
        ref, T = ob.gemm(*ora_ops)
        g = float(g_out.item())
        deq = ob.dequantize(got_c.cpu().numpy(), got_s.cpu().numpy(), g)
        step = np.repeat(np.array([ob.e4m3_decode(int(b)) for b in got_s.cpu().numpy().reshape(-1)],
                                  dtype=np.float64).reshape(M, N // 16), 16, axis=1) * g * 2.0
        slack = (1.0 if mode == nb.RTN else 2.0) * step + TOL * T      # also covers the clip of a block's maximum at 6
        assert np.all(np.abs(deq - ref) <= slack)


# ---------------------------------------------------------------- the two kernel designs against each other
@pytest.mark.parametrize("shape", [(4096, 4096, 4096), (2048, 5120, 11008), (5000, 3000, 2080)])
def test_pair_and_single_cta_kernels_agree_on_large_shapes(shape):
    # Both kernels add the 64-value products of a row in the same order, so their fp32 results are the
    # same numbers; a scale tile or a stage consumed one step early or late by either of them would show.
    M, N, K = shape
    A = synth.normal((M, K), 1.0, 7, device="cuda")
    B = synth.normal((N, K), 0.02, 8, device="cuda")
    ga, gb = nb.nvfp4_tensor_amax_scale(A), nb.nvfp4_tensor_amax_scale(B)
    ac, asf = nb.nvfp4_quantize(A, global_scale=ga, sf_layout=nb.SF_SWIZZLED)
    bc, bsf = nb.nvfp4_quantize(B, global_scale=gb, sf_layout=nb.SF_SWIZZLED)
    outs = {}
    try:
        for tile in (256, 2256, 2192):
            nb.nvfp4_gemm_set_tile_n(tile)
            # back-to-back launches: the result may not depend on timing (the pair kernel's roles hand stages
            # and scale buffers to each other through barriers polled with relaxed loads)
            for rep in range(24 if tile == 2256 else 3):
                D = nb.nvfp4_gemm(ac, asf, ga, bc, bsf, gb)
                if tile in outs:
                    assert torch.equal(outs[tile], D)
                else:
                    outs[tile] = D
    finally:
        nb.nvfp4_gemm_set_tile_n(0)
    assert nb.nvfp4_device_error_word() == 0
    assert torch.equal(outs[256], outs[2256]) and torch.equal(outs[256], outs[2192])
    # and a sample of the outputs against the oracle
    rng = np.random.default_rng(5)
    ii, jj = rng.integers(0, M, 512), rng.integers(0, N, 512)
    oa = ob.quantize(A.float().cpu().numpy(), g=float(ga.item()))
    obq = ob.quantize(B.float().cpu().numpy(), g=float(gb.item()))
    ref, T = ob.gemm_sampled(oa[0], oa[1], float(ga.item()), obq[0], obq[1], float(gb.item()), ii, jj)
    assert np.all(np.abs(outs[2256].cpu().numpy()[ii, jj] - ref) <= TOL * T)
