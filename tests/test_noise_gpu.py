"""GPU-vs-oracle parity of the quantization-noise monitor (Section 4): sum (Q(x)-x)^2 and sum x^2."""
import numpy as np
import pytest
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth

pytestmark = pytest.mark.gpu

RTOL = 1e-5   # fp32 products and short fp32 partial sums, double accumulation across threads


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("sf_layout", [nb.SF_LINEAR, nb.SF_SWIZZLED])
@pytest.mark.parametrize("transposed", [False, True])
@pytest.mark.parametrize("mode", [nb.RTN, nb.SR])
@pytest.mark.parametrize("shape", [(256, 512), (272, 144), (32, 64)])
def test_noise_sums_match_the_oracle(shape, mode, transposed, sf_layout, dtype):
    x = synth.normal(shape, 1e-3, 77, device="cpu", dtype=dtype).cuda()
    g_t = nb.nvfp4_tensor_amax_scale(x)
    r = nb.Rounding(mode, 6, 2)
    codes, scales = nb.nvfp4_quantize(x, transposed, g_t, r, sf_layout)
    sums = nb.nvfp4_quantization_noise(x, codes, scales, transposed, g_t, sf_layout).cpu().numpy()
    h = x.float().cpu().numpy()
    g = ob.tensor_amax_scale(h)
    oc, osf = ob.quantize(h, g=g, mode=mode, seed=6, offset=2, transposed=transposed)
    e2, x2 = ob.noise_sums(np.ascontiguousarray(h.T) if transposed else h, oc, osf, g)
    assert abs(sums[0] - e2) <= RTOL * e2 and abs(sums[1] - x2) <= RTOL * x2
    assert e2 > 0 and x2 / e2 > 3.0          # a healthy tensor sits well above the paper's sqrt(3) threshold


def test_noise_ratio_of_the_two_roundings_on_gradient_like_data():
    # SR's mean squared error is about twice RtN's on the same tensor (spacing^2/6 against spacing^2/12)
    x = synth.normal((2048, 2048), 1e-4, 78, device="cuda")
    g_t = nb.nvfp4_tensor_amax_scale(x)
    out = {}
    for mode in (nb.RTN, nb.SR):
        codes, scales = nb.nvfp4_quantize(x, False, g_t, nb.Rounding(mode, 1, 0), nb.SF_SWIZZLED)
        out[mode] = nb.nvfp4_quantization_noise(x, codes, scales, False, g_t, nb.SF_SWIZZLED).cpu().numpy()
    assert out[nb.RTN][1] == out[nb.SR][1]
    ratio = out[nb.SR][0] / out[nb.RTN][0]
    assert 1.7 < ratio < 2.3
