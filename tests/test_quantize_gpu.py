"""GPU-vs-oracle parity of the quantizer kernels, bit-exact on codes and scales."""
import numpy as np
import pytest
import torch

from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth
from tests.util import assert_quantize_parity

pytestmark = pytest.mark.gpu

ROW_SHAPES = [(1, 16), (3, 48), (130, 80), (128, 512), (257, 1040), (256, 512), (129, 4112)]
# rows % 32 == 0 takes the tiled-copy kernel (ragged tiles in both directions), the others the fallback kernel
T_SHAPES = [(16, 8), (48, 24), (272, 72), (512, 200), (256, 64), (1040, 264), (4112, 136), (288, 72), (32, 8), (1056, 328)]


def _x(shape, seed, dtype=torch.bfloat16, std=1.0):
    return synth.normal(shape, std, seed, device="cpu", dtype=dtype).cuda()


@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", ROW_SHAPES)
def test_row_bf16(shape, mode, sf_layout):
    assert_quantize_parity(_x(shape, 1), False, False, nb.Rounding(mode, 1234, 5), sf_layout)


@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", T_SHAPES)
def test_transposed_bf16(shape, mode, sf_layout):
    assert_quantize_parity(_x(shape, 2), True, False, nb.Rounding(mode, 99, 1), sf_layout)


@pytest.mark.parametrize("transposed", [False, True])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
def test_fp32_input(mode, transposed):
    shape = (272, 136) if transposed else (131, 272)
    x = _x(shape, 3, dtype=torch.float32)
    assert_quantize_parity(x, transposed, False, nb.Rounding(mode, 7, 0), nb.SF_SWIZZLED)
    assert_quantize_parity(x, transposed, True, nb.Rounding(mode, 7, 0), nb.SF_LINEAR)


@pytest.mark.parametrize("transposed", [False, True])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("std", [1e-4, 1e-3, 0.02, 50.0])
def test_global_scale_from_amax(std, mode, transposed):
    x = _x((256, 512), 4, std=std)
    assert_quantize_parity(x, transposed, True, nb.Rounding(mode, 0, 2), nb.SF_SWIZZLED)


def test_gradient_scale_underflow_without_global_scale():
    # N(0, 1e-4^2) with g = 1: every block scale underflows to 0 and only sign bits survive
    x = _x((128, 256), 5, std=1e-4)
    assert_quantize_parity(x, False, False, nb.Rounding(nb.RTN), nb.SF_LINEAR)
    codes, scales = nb.nvfp4_quantize(x)
    assert int(scales.max()) == 0 and int((codes & 0x77).max()) == 0


def test_special_values():
    x = torch.zeros((16, 64), dtype=torch.float32)
    x[0, :8] = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0])       # tie points, scale 1
    x[1, :8] = -x[0, :8]
    x[2, 3] = -0.0
    x[3, 0] = 6.0 * 448.0 * 4                                                    # saturating scale
    x[3, 1:16] = 3000.0
    x[4, :16] = torch.linspace(-6, 6, 16)
    x[5, 16:32] = 1e-30
    x[6, 0] = 2.0 ** -9 * 6
    x[6, 1] = 2.0 ** -10 * 6
    x[7, 0] = 448.0 * 6
    x[7, 1] = 447.0
    for dt in (torch.bfloat16, torch.float32):
        xs = x.to(dt).cuda()
        for mode in (nb.RTN, nb.SR):
            assert_quantize_parity(xs, False, False, nb.Rounding(mode, 3, 3), nb.SF_LINEAR)
            assert_quantize_parity(xs, True, False, nb.Rounding(mode, 3, 3), nb.SF_LINEAR)


def test_sr_reproducible_and_offset_sensitive():
    x = _x((256, 512), 6)
    a, _ = nb.nvfp4_quantize(x, rounding=nb.Rounding(nb.SR, 1, 0))
    b, _ = nb.nvfp4_quantize(x, rounding=nb.Rounding(nb.SR, 1, 0))
    c, _ = nb.nvfp4_quantize(x, rounding=nb.Rounding(nb.SR, 1, 1))
    assert torch.equal(a, b) and not torch.equal(a, c)


def test_strided_input():
    base = _x((64, 1024), 7)
    view = base[:, 256:768]
    assert_quantize_parity(view, False, False, nb.Rounding(nb.SR, 5, 5), nb.SF_SWIZZLED)
    assert_quantize_parity(view, True, False, nb.Rounding(nb.SR, 5, 5), nb.SF_SWIZZLED)


@pytest.mark.parametrize("n_elem", [2 ** 20, 2 ** 24])
@pytest.mark.parametrize("transposed", [False, True])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
def test_heavy_tailed_sweep(n_elem, transposed, mode):
    x = synth.heavy_tailed(synth.square_shape(n_elem), seed=1001, device="cpu").cuda()
    assert_quantize_parity(x, transposed, True, nb.Rounding(mode, 1, 0), nb.SF_SWIZZLED)


# ---------------------------------------------------------------- both orientations from one read
DUAL_SHAPES = [(256, 64), (512, 192), (288, 96), (32, 32), (1056, 352), (48, 80), (272, 48)]   # the last two: fallback path


@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("modes", [(nb.RTN, nb.SR), (nb.SR, nb.SR), (nb.RTN, nb.RTN), (nb.SR, nb.RTN)])
@pytest.mark.parametrize("shape", DUAL_SHAPES)
def test_dual_matches_the_oracle_in_both_orientations(shape, modes, sf_layout):
    from oracle import binding as ob
    from tests.util import oracle_quantize
    x = _x(shape, 11)
    g_t = nb.nvfp4_tensor_amax_scale(x)
    g = float(g_t.item())
    rr, rt = nb.Rounding(modes[0], 21, 4), nb.Rounding(modes[1], 21, 5)
    cr, sr, ct, st = nb.nvfp4_quantize_dual(x, g_t, rr, rt, sf_layout)
    torch.cuda.synchronize()
    assert nb.nvfp4_device_error_word() == 0
    for got_c, got_s, transposed, r in ((cr, sr, False, rr), (ct, st, True, rt)):
        oc, osf = oracle_quantize(x, transposed, g, r)
        if sf_layout == nb.SF_SWIZZLED:
            osf = ob.sf_swizzle(osf)
        assert np.array_equal(got_c.cpu().numpy(), oc)
        assert np.array_equal(got_s.cpu().numpy().reshape(-1), osf.reshape(-1))


def test_dual_heavy_tailed_2p24():
    from oracle import binding as ob
    from tests.util import oracle_quantize
    x = synth.heavy_tailed(synth.square_shape(2 ** 24), seed=1001, device="cpu").cuda()
    g_t = nb.nvfp4_tensor_amax_scale(x)
    rr, rt = nb.Rounding(nb.SR, 1, 0), nb.Rounding(nb.SR, 1, 1)
    cr, sr, ct, st = nb.nvfp4_quantize_dual(x, g_t, rr, rt, nb.SF_SWIZZLED)
    for got_c, got_s, transposed, r in ((cr, sr, False, rr), (ct, st, True, rt)):
        oc, osf = oracle_quantize(x, transposed, float(g_t.item()), r)
        assert np.array_equal(got_c.cpu().numpy(), oc)
        assert np.array_equal(got_s.cpu().numpy().reshape(-1), ob.sf_swizzle(osf).reshape(-1))
