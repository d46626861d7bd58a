"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import binding as ob
from paper_2505_19115_b200 import binding as nb


def to_host_f32(x: torch.Tensor) -> np.ndarray:
    return x.detach().float().cpu().numpy()


def oracle_quantize(x: torch.Tensor, transposed=False, g=1.0, rounding=None):
    r = rounding or nb.Rounding()
    return ob.quantize(to_host_f32(x), g=g, mode=r.mode, seed=r.seed, offset=r.offset, transposed=transposed)


CANARY = 0xA5


def guarded_u8(nbytes: int, device="cuda"):
    """A uint8 buffer with 64 canary bytes on each side; returns (whole, view)."""
    whole = torch.full((nbytes + 128,), CANARY, dtype=torch.uint8, device=device)
    return whole, whole[64:64 + nbytes]


def canaries_intact(whole: torch.Tensor) -> bool:
    h = whole.cpu().numpy()
    return bool(np.all(h[:64] == CANARY) and np.all(h[-64:] == CANARY))


def gpu_quantize_checked(x, transposed, g_tensor, rounding, sf_layout):
    rows, cols = x.shape
    Rq, Kq = (cols, rows) if transposed else (rows, cols)
    cw, cv = guarded_u8(Rq * Kq // 2)
    sw, sv = guarded_u8(nb.nvfp4_sf_bytes(Rq, Kq, sf_layout))
    nb.nvfp4_quantize(x, transposed=transposed, global_scale=g_tensor, rounding=rounding, sf_layout=sf_layout,
                      codes=cv, scales=sv)
    torch.cuda.synchronize()
    assert canaries_intact(cw) and canaries_intact(sw)
    return cv.cpu().numpy().reshape(Rq, Kq // 2), sv.cpu().numpy()


def assert_quantize_parity(x, transposed=False, use_g=False, rounding=None, sf_layout=nb.SF_LINEAR):
    rows, cols = x.shape
    Rq, Kq = (cols, rows) if transposed else (rows, cols)
    g_tensor, g = None, 1.0
    if use_g:
        g_tensor = nb.nvfp4_tensor_amax_scale(x)
        g = float(g_tensor.cpu().item())
        assert np.float32(g) == np.float32(ob.tensor_amax_scale(to_host_f32(x)))
    codes, scales = gpu_quantize_checked(x, transposed, g_tensor, rounding, sf_layout)
    oc, osf = oracle_quantize(x, transposed, g, rounding)
    if sf_layout == nb.SF_SWIZZLED:
        osf = ob.sf_swizzle(osf)
    else:
        scales = scales.reshape(Rq, Kq // 16)
    bad_s = np.flatnonzero(scales.reshape(-1) != osf.reshape(-1))
    assert bad_s.size == 0, f"{bad_s.size} scale bytes differ, first at {bad_s[:5]}"
    bad_c = np.flatnonzero(codes.reshape(-1) != oc.reshape(-1))
    assert bad_c.size == 0, f"{bad_c.size} code bytes differ, first at {bad_c[:5]}"
