"""nvfp4_linear_fwd_static: the forward product for callers that cannot allocate or hand over
scratch memory (the device may be fully reserved by the host framework's pool, or the section may
not tolerate cudaMalloc's device-wide synchronisation).  Its scratch is a fixed array inside the
library that every call on a device shares, so the test makes two calls in a row, with different
shapes, and checks each against nvfp4_linear_fwd, whose scratch the caller supplies."""
import numpy as np
import pytest
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb
from paper_2505_19115_b200 import synth

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _tolerance_base(X, W):
    hx, hw = X.float().cpu().numpy(), W.float().cpu().numpy()
    gx, gw = ob.tensor_amax_scale(hx), ob.tensor_amax_scale(hw)
    xc, xs = ob.quantize(hx, g=gx)
    wc, ws = ob.quantize(hw, g=gw)
    return ob.gemm(xc, xs, gx, wc, ws, gw)


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    rt = nb.Rounding(nb.RTN)
    # the second layer is smaller and ragged: it finds the first call's bytes in the shared array
    for (M, K, N), seed in (((256, 512, 512), 11), ((160, 288, 200), 12)):
        X, W, _ = synth.linear_inputs(M, K, N, seed=seed)
        X, W = X.cuda(), W.cuda()
        assert nb.nvfp4_linear_workspace_bytes(M, N, K, nb.LINEAR_FWD) <= nb.STATIC_WORKSPACE_BYTES
        got = nb.nvfp4_linear_fwd_static(X, W, rx=rt, rw=rt)
        want = nb.nvfp4_linear_fwd(X, W, rx=rt, rw=rt)
        torch.cuda.synchronize()
        assert nb.nvfp4_device_error_word() == 0
        ref, T = _tolerance_base(X, W)
        g, w = got.cpu().numpy(), want.cpu().numpy()
        assert np.all(np.abs(g - w) <= TOL * T)
        assert np.all(np.abs(g - ref) <= TOL * T)


def test_layer_beyond_the_fixed_array_is_rejected():
    M, K, N = 16384, 4096, 4096
    assert nb.nvfp4_linear_workspace_bytes(M, N, K, nb.LINEAR_FWD) > nb.STATIC_WORKSPACE_BYTES
    X = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(nb.NvFp4Error) as e:
        nb.nvfp4_linear_fwd_static(X, W)
    assert e.value.status == 5


def test_the_call_leaves_the_free_device_memory_unchanged():
    # The property in the entry point's name: with the output preallocated, a call takes no device memory
    # (cudaMemGetInfo's free bytes are the same before and after).  The first call on a device loads the
    # kernels and looks up the array's address, so it is made before the measurement.
    rt = nb.Rounding(nb.RTN)
    X, W, _ = synth.linear_inputs(256, 512, 512, seed=13)
    X, W = X.cuda(), W.cuda()
    out = torch.empty((256, 512), dtype=torch.float32, device="cuda")
    nb.nvfp4_linear_fwd_static(X, W, rx=rt, rw=rt, out=out)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        nb.nvfp4_linear_fwd_static(X, W, rx=rt, rw=rt, out=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    want = nb.nvfp4_linear_fwd(X, W, rx=rt, rw=rt)
    assert torch.equal(out, want)
