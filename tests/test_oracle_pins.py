"""Pins for the CPU oracle: each test fixes oracle behaviour with something other
than the oracle itself -- the format definitions, exhaustive search in exact
rational arithmetic, closed forms, published known-answer vectors, a library cast."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import binding as ob

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


GRID = [float(v) for _, v in _rows("e2m1_grid.txt")]
GRID_F = [Fraction(v) for v in GRID]
# every E4M3 bit pattern decoded by the library cast (independent of the oracle)
E4M3_LIB = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()


# ---------------------------------------------------------------- formats
def test_e2m1_decode_matches_grid():
    for code in range(16):
        mag = GRID[code & 7]
        assert ob.e2m1_decode(code) == (-mag if code & 8 else mag)
    # sign of zero is kept as a code but decodes to (-)0
    assert np.signbit(np.float32(ob.e2m1_decode(8)))


def test_e4m3_decode_matches_library_cast():
    for code in range(127):
        assert ob.e4m3_decode(code) == float(E4M3_LIB[code])
    assert ob.e4m3_decode(0x7E) == 448.0
    assert ob.e4m3_decode(1) == 2.0 ** -9
    assert ob.e4m3_decode(8) == 2.0 ** -6


def test_e4m3_roundtrip_all_finite_codes():
    for code in range(127):
        assert ob.e4m3_encode(ob.e4m3_decode(code)) == code


def test_e4m3_encode_matches_library_cast_in_range():
    rng = np.random.default_rng(0)
    v = np.concatenate([
        np.exp(rng.uniform(np.log(2.0 ** -12), np.log(448.0), 20000)),
        rng.uniform(0, 2.0 ** -5, 2000), rng.uniform(400, 448, 500)]).astype(np.float32)
    lib = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    ours = np.array([ob.e4m3_encode(x) for x in v], dtype=np.uint8)
    assert np.array_equal(lib, ours)


def test_e4m3_encode_is_nearest_with_even_ties():
    vals = [Fraction(float(E4M3_LIB[c])) for c in range(127)]
    # exact midpoints between neighbours go to the even code
    for c in range(126):
        mid = (vals[c] + vals[c + 1]) / 2
        got = ob.e4m3_encode(float(mid))
        assert got == (c if c % 2 == 0 else c + 1), (c, float(mid), got)
        # just off the midpoint goes to the nearer side
        for eps, want in ((-1, c), (1, c + 1)):
            x = np.nextafter(np.float32(float(mid)), np.float32(np.inf if eps > 0 else 0))
            assert ob.e4m3_encode(float(x)) == want
    # brute force: nearest in exact arithmetic
    rng = np.random.default_rng(1)
    for x in np.exp(rng.uniform(np.log(1e-4), np.log(447.0), 3000)).astype(np.float32):
        fx = Fraction(float(x))
        dist = [abs(fx - v) for v in vals]
        best = min(dist)
        got = ob.e4m3_encode(float(x))
        assert dist[got] == best


def test_e4m3_encode_saturates_and_handles_zero():
    assert ob.e4m3_encode(0.0) == 0
    assert ob.e4m3_encode(448.0) == 0x7E
    assert ob.e4m3_encode(449.0) == 0x7E
    assert ob.e4m3_encode(463.9) == 0x7E
    assert ob.e4m3_encode(1e9) == 0x7E
    assert ob.e4m3_encode(float("inf")) == 0x7E
    assert ob.e4m3_encode(2.0 ** -10) == 0            # tie between 0 and the least subnormal
    assert ob.e4m3_encode(float(np.nextafter(np.float32(2.0 ** -10), np.float32(1)))) == 1


# ---------------------------------------------------------------- Philox
def test_philox_known_answers():
    for row in _rows("philox4x32_10_kat.txt"):
        v = [int(t, 16) for t in row]
        out = ob.philox4x32_10(v[4:6], v[0:4])
        assert [int(o) for o in out] == v[6:10]


def _rev16(v):
    return int(f"{v:016b}"[::-1], 2)


def test_word_random_integers_use_every_bit_twice_and_pairs_mirror_each_other():
    # one-hot words: bit b of bytes 0/2 reaches elements 0 and 1 only, of bytes 1/3 elements 2 and 3
    # only; the even element takes the byte pair as (low, high), the odd one the same 16 bits mirrored
    for bit in range(32):
        byte, k = divmod(bit, 8)
        r = [int(v) for v in ob.word_random_u16(1 << bit)]
        pos = k + (8 if byte >= 2 else 0)
        if byte in (0, 2):
            assert r == [1 << pos, 1 << (15 - pos), 0, 0]
        else:
            assert r == [0, 0, 1 << pos, 1 << (15 - pos)]
    rng = np.random.default_rng(5)
    for w in rng.integers(0, 2 ** 32, 200):
        r = [int(v) for v in ob.word_random_u16(int(w))]
        assert r[1] == _rev16(r[0]) and r[3] == _rev16(r[2])
        assert r[0] | (r[2] << 16) == (w & 0xFF) | ((w >> 16 & 0xFF) << 8) | ((w >> 8 & 0xFF) << 16) | ((w >> 24) << 24)


def test_block_random_integers_come_from_the_words_of_the_counter():
    seed, offset, block = 0x0123456789ABCDEF, 0x1122334455667788, 0xA1B2C3D4E5F60718
    words = ob.philox4x32_10([seed & 0xFFFFFFFF, seed >> 32],
                             [block & 0xFFFFFFFF, block >> 32, offset & 0xFFFFFFFF, offset >> 32])
    want = np.concatenate([ob.word_random_u16(int(w)) for w in words])
    assert np.array_equal(ob.block_random_u16(seed, offset, block), want)
    # different block / offset / seed -> different integers
    assert not np.array_equal(ob.block_random_u16(seed, offset, block + 1), want)
    assert not np.array_equal(ob.block_random_u16(seed, offset + 1, block), want)
    assert not np.array_equal(ob.block_random_u16(seed + 1, offset, block), want)


# ---------------------------------------------------------------- rounding
def test_rtn_golden_ties():
    for y, code, val in _rows("rtn_ties.txt"):
        assert ob.round_rtn(float(y)) == int(code)
        assert GRID[int(code)] == float(val)


def test_rtn_is_argmin_for_every_bf16_value_in_range():
    # all non-negative bf16 bit patterns up to 6.0
    bits = np.arange(0, 0x40C1, dtype=np.uint32)           # 0x40C0 = 6.0 in bf16
    ys = (bits << 16).view(np.float32)
    for y in ys:
        fy = Fraction(float(y))
        dist = [abs(fy - g) for g in GRID_F]
        best = min(dist)
        got = ob.round_rtn(float(y))
        assert dist[got] == best
        ties = [c for c in range(8) if dist[c] == best]
        if len(ties) == 2:
            assert got % 2 == 0


def _sr_neighbours(y):
    lo = max(g for g in GRID if g <= y)
    hi = min(g for g in GRID if g >= y)
    return lo, hi


def test_sr_exact_distribution_over_all_random_integers():
    # all 2^16 random integers for a few values: support, exact count of round-ups, monotonicity
    for y in np.array([0.3, 1.26, 2.9, 4.000001, 5.999, 0.0001], dtype=np.float32):
        lo, hi = _sr_neighbours(float(y))
        delta = hi - lo
        f = (Fraction(float(y)) - Fraction(lo)) / Fraction(delta)
        ups = int(f * 65536)                                  # floor
        vals = np.array([GRID[ob.round_sr(float(y), r)] for r in range(65536)])
        assert set(vals.tolist()) <= {lo, hi}
        assert int(np.sum(vals == hi)) == ups
        assert np.all(np.diff((vals == hi).astype(int)) >= 0)  # the largest integers round up
        assert 0 <= float(y) - vals.mean() <= delta / 65536 + 1e-12


def test_sr_threshold_for_many_values():
    rng = np.random.default_rng(2)
    ys = np.concatenate([rng.uniform(0, 6, 2000), np.array(GRID), [0.001, 5.999, 1.999, 2.001, 3.999, 4.001, 1e-6]])
    for y in ys.astype(np.float32):
        lo, hi = _sr_neighbours(float(y))
        if lo == hi:                                          # representable values never move
            assert all(GRID[ob.round_sr(float(y), r)] == lo for r in (0, 1, 32768, 65535))
            continue
        f = (Fraction(float(y)) - Fraction(lo)) / Fraction(hi - lo)
        F = int(f * 65536)
        assert GRID[ob.round_sr(float(y), 0)] == lo
        assert GRID[ob.round_sr(float(y), 65535 - F)] == lo
        if F > 0:
            assert GRID[ob.round_sr(float(y), 65536 - F)] == hi
            assert GRID[ob.round_sr(float(y), 65535)] == hi


def test_sr_unbiased_over_seeded_draws():
    # 10^4 Philox-seeded draws of the same block: mean within 3 sigma (+ the 16-bit truncation bound)
    x = np.array([[0.3, -0.7, 1.1, 1.6, 2.2, -2.9, 3.3, 4.7, 5.5, 0.05, 6.0, -0.26, 0.9, 1.9, 3.9, -5.9]],
                 dtype=np.float32)
    n = 10000
    acc = np.zeros(16)
    acc2 = np.zeros(16)
    for s in range(n):
        codes, scales = ob.quantize(x, mode=ob.SR, seed=s, offset=7, nthreads=1)
        assert scales[0, 0] == ob.e4m3_encode(1.0)           # amax 6 -> scale 1
        deq = ob.dequantize(codes, scales)[0].astype(np.float64)
        acc += deq
        acc2 += deq * deq
    mean = acc / n
    var = np.maximum(acc2 / n - mean ** 2, 0)
    for j in range(16):
        lo, hi = _sr_neighbours(abs(float(x[0, j])))
        bound = 3 * np.sqrt(var[j] / n) + (hi - lo) / 65536 + 1e-9
        assert abs(mean[j] - float(x[0, j])) <= bound, (j, mean[j], x[0, j], bound)


def test_sr_neighbouring_elements_round_independently_enough():
    # elements 0/1 (and 2/3) of a word share their 16 random bits in mirrored order: the joint
    # frequency of "both round up" must still be the product of the two probabilities
    y = np.float32(1.25)                                      # f = 1/2 for both
    rng = np.random.default_rng(9)
    both = n = 0
    for w in rng.integers(0, 2 ** 32, 20000):
        r = ob.word_random_u16(int(w))
        a, b = ob.round_sr(float(y), int(r[0])) == 3, ob.round_sr(float(y), int(r[1])) == 3
        both += a and b
        n += 1
    assert abs(both / n - 0.25) < 0.015


def test_sr_pair_joint_probability_over_all_random_integers():
    # The two elements of a pair read the same 16 random bits, one in mirrored order.  For the noise model of
    # Section 4 / App. B.1 (independent zero-mean errors) their round-up decisions must be close to independent
    # at every (f0, f1), not only at f = 1/2.  Element 0 rounds up iff r >= 2^16 - F0, which the top byte H of
    # r decides unless H equals the threshold's top byte (probability 2^-8); element 1 rounds up iff
    # mirror(r) >= 2^16 - F1, which the mirrored low byte L decides unless it ties (2^-8).  H and L are
    # independent, and a tie's decision depends on the other byte only through an indicator whose covariance
    # with the other decision is at most 1/4, so |P(both up) - P0 P1| <= 2 * 2^-8 / 4 + 2^-16.
    bound = 2.0 ** -9 + 2.0 ** -16
    rng = np.random.default_rng(11)
    base = int(rng.integers(0, 2 ** 32))
    worst = 0.0
    for pair, (lo_shift, hi_shift) in enumerate(((0, 16), (8, 24))):        # bytes (0, 2) serve elements 0/1, bytes (1, 3) elements 2/3
        keep = base & ~((0xFF << lo_shift) | (0xFF << hi_shift)) & 0xFFFFFFFF
        ints = np.array([ob.word_random_u16(keep | ((v & 0xFF) << lo_shift) | ((v >> 8) << hi_shift)) for v in range(65536)],
                        dtype=np.uint16)
        r_even, r_odd = ints[:, 2 * pair], ints[:, 2 * pair + 1]
        assert np.array_equal(np.sort(r_even), np.arange(65536)) and np.array_equal(np.sort(r_odd), np.arange(65536))
        for _ in range(110):
            y0, y1 = (np.float32(v) for v in rng.uniform(0.0, 6.0, 2))
            (lo0, hi0), (lo1, hi1) = _sr_neighbours(float(y0)), _sr_neighbours(float(y1))
            if lo0 == hi0 or lo1 == hi1:
                continue
            up0 = np.array(GRID)[ob.round_sr_many(float(y0), r_even)] == hi0
            up1 = np.array(GRID)[ob.round_sr_many(float(y1), r_odd)] == hi1
            d = abs(float(np.mean(up0 & up1)) - float(np.mean(up0)) * float(np.mean(up1)))
            worst = max(worst, d)
            assert d <= bound, (pair, float(y0), float(y1), d)
    assert worst > 0.0                                                       # the pairs are dependent, only weakly


def test_sr_errors_of_a_block_behave_like_independent_noise():
    # 2 * 10^4 seeded draws of one block: the rounding errors of paired elements (0/1, 2/3, ...) are uncorrelated
    # within 3 sigma, and the variance of the block's summed error equals the sum of the per-element
    # variances, as independent zero-mean noise would give (App. B.1 assumes E[eps eps^T] = sigma^2 I).
    x1 = np.array([0.3, -0.7, 1.1, 1.6, 2.2, -2.9, 3.3, 4.7, 5.5, 0.05, 6.0, -0.26, 0.9, 1.9, 3.9, -5.9], dtype=np.float32)
    n = 20000
    x = np.tile(x1, (n, 1))                                                  # row r draws block index r
    codes, scales = ob.quantize(x, mode=ob.SR, seed=123, offset=5)
    err = ob.dequantize(codes, scales).astype(np.float64) - x.astype(np.float64)
    sd = err.std(axis=0)
    assert abs(err.mean(axis=0)).max() <= 3 * sd.max() / np.sqrt(n) + 2.0 / 65536
    moving = [j for j in range(16) if sd[j] > 0]
    assert len(moving) >= 14
    for a in range(0, 16, 2):
        if sd[a] > 0 and sd[a + 1] > 0:
            corr = np.mean((err[:, a] - err[:, a].mean()) * (err[:, a + 1] - err[:, a + 1].mean())) / (sd[a] * sd[a + 1])
            assert abs(corr) <= 3 / np.sqrt(n) + 2.0 ** -7, (a, corr)
    total = err.sum(axis=1)
    want = float(np.sum(sd ** 2))
    # the sample variance of n draws of a sum of bounded terms: relative standard error about sqrt(2/n)
    assert abs(total.var() - want) <= 4 * np.sqrt(2.0 / n) * want + 0.01 * want


def test_tensor_scale_propagates_non_finite_values():
    # A diverged step must stay visible: NaN anywhere -> NaN, otherwise an infinity -> +Inf.
    assert np.isnan(ob.tensor_amax_scale(np.array([1.0, np.nan, 3.0], dtype=np.float32)))
    assert np.isnan(ob.tensor_amax_scale(np.array([np.inf, np.nan], dtype=np.float32)))
    assert ob.tensor_amax_scale(np.array([1.0, -np.inf], dtype=np.float32)) == np.inf
    assert ob.tensor_amax_scale(np.array([0.0, 2688.0], dtype=np.float32)) == 1.0
    # ... and every output of a product computed with such a scale is NaN
    rng = np.random.default_rng(4)
    X = rng.standard_normal((8, 64)).astype(np.float32)
    W = rng.standard_normal((16, 64)).astype(np.float32)
    for bad in (np.nan, np.inf, -np.inf):
        Xb = X.copy()
        Xb[3, 17] = bad
        gx, gw = ob.tensor_amax_scale(Xb), ob.tensor_amax_scale(W)
        xc, xs = ob.quantize(Xb, g=gx)
        wc, ws = ob.quantize(W, g=gw)
        D, _ = ob.gemm(xc, xs, gx, wc, ws, gw)
        assert np.all(np.isnan(D)), bad


def test_sr_variance_closed_form():
    # y uniform within one grid step: E[err^2] = delta^2/6 under SR, delta^2/12 under RtN
    rng = np.random.default_rng(3)
    ys = rng.uniform(2.0, 3.0, 40000).astype(np.float32)
    us = rng.integers(0, 65536, ys.size)
    sr = np.array([GRID[ob.round_sr(float(y), int(u))] for y, u in zip(ys, us)])
    rt = np.array([GRID[ob.round_rtn(float(y))] for y in ys])
    assert abs(np.mean((sr - ys) ** 2) - 1 / 6) < 0.01
    assert abs(np.mean((rt - ys) ** 2) - 1 / 12) < 0.005
    assert abs(np.mean(sr - ys)) < 0.01


# ---------------------------------------------------------------- block quantizer
def _exact_block_check(x, codes, scales):
    """Exhaustive-search definition in rational arithmetic: the scale is a nearest
    E4M3 value to amax/6 and every code a nearest grid value to |x|/scale (up to
    the fp32 roundings the oracle is allowed: a relative slack of 2^-20)."""
    e4 = [Fraction(float(E4M3_LIB[c])) for c in range(127)]
    R, K = x.shape
    for r in range(R):
        for kb in range(K // 16):
            blk = x[r, kb * 16:(kb + 1) * 16]
            amax = Fraction(float(np.max(np.abs(blk))))
            target = amax / 6
            dist = [abs(target - v) for v in e4]
            sq = int(scales[r, kb])
            assert dist[sq] <= min(dist) + target * Fraction(1, 2 ** 20)
            s = e4[sq]
            for j in range(16):
                byte = codes[r, (kb * 16 + j) // 2]
                nib = (byte >> 4) if j & 1 else (byte & 15)
                assert (nib >> 3) == int(np.signbit(blk[j]))
                if s == 0:
                    assert nib & 7 == 0
                    continue
                y = min(abs(Fraction(float(blk[j]))) / s, Fraction(6))
                d = [abs(y - g) for g in GRID_F]
                assert d[nib & 7] <= min(d) + y * Fraction(1, 2 ** 20)


def test_quantize_rtn_brute_force_tiny():
    rng = np.random.default_rng(4)
    for scale in (1.0, 0.02, 37.0):
        x = (rng.standard_normal((3, 48)) * scale).astype(np.float32)
        x = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
        codes, scales = ob.quantize(x, nthreads=1)
        _exact_block_check(x, codes, scales)


def test_quantize_layout_nibbles_and_scale_index():
    # one non-zero element at a time: its nibble position and block scale index are fixed
    for (r, k) in [(0, 0), (0, 1), (1, 17), (2, 46), (1, 31)]:
        x = np.zeros((3, 48), dtype=np.float32)
        x[r, k] = -3.0                                      # amax 3 -> scale 0.5, value 6 -> code 7, sign 1
        codes, scales = ob.quantize(x, nthreads=1)
        want_codes = np.zeros_like(codes)
        want_codes[r, k // 2] = 0xF << (4 * (k & 1))
        want_scales = np.zeros_like(scales)
        want_scales[r, k // 16] = ob.e4m3_encode(0.5)
        assert np.array_equal(codes, want_codes)
        assert np.array_equal(scales, want_scales)
        assert ob.e4m3_decode(int(scales[r, k // 16])) == 0.5


def test_quantize_scale_invariants():
    rng = np.random.default_rng(5)
    x = torch.from_numpy(rng.standard_normal((8, 256)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    codes, scales = ob.quantize(x, nthreads=1)
    # amax maps near 6: the largest magnitude code of every normal-scale block is 7
    mags = np.maximum(codes & 7, (codes >> 4) & 7).reshape(8, 16, 8).max(axis=2)
    assert np.all(mags[scales >= 8] == 7)
    # power-of-two equivariance: same codes, scale exponent shifted
    for k in (-3, 2):
        c2, s2 = ob.quantize(x * np.float32(2.0 ** k), nthreads=1)
        assert np.array_equal(c2, codes)
        assert np.array_equal(s2.astype(int), scales.astype(int) + 8 * k)
    # idempotence under RtN
    deq = ob.dequantize(codes, scales)
    c3, s3 = ob.quantize(deq, nthreads=1)
    assert np.array_equal(c3, codes) and np.array_equal(s3, scales)
    # sign symmetry
    c4, s4 = ob.quantize(-x, nthreads=1)
    assert np.array_equal(c4, codes ^ 0x88) and np.array_equal(s4, scales)


def test_quantize_zero_block_and_underflow():
    x = np.zeros((1, 32), dtype=np.float32)
    x[0, 3] = -0.0
    x[0, 16:] = 1e-4                                         # amax/6 far below the smallest E4M3 step
    codes, scales = ob.quantize(x, nthreads=1)
    assert np.all(scales == 0)
    want = np.zeros((1, 16), dtype=np.uint8)
    want[0, 1] = 0x80                                        # only the sign bit of -0.0 survives
    assert np.array_equal(codes, want)
    assert np.all(np.isfinite(ob.dequantize(codes, scales)))


def test_quantize_saturating_scale_clamps_values():
    x = np.full((1, 16), 10.0, dtype=np.float32)
    x[0, 0] = 6.0 * 448.0 * 4                                # scale saturates at 448, value/scale = 24 -> clamp 6
    codes, scales = ob.quantize(x, nthreads=1)
    assert scales[0, 0] == 0x7E
    assert codes[0, 0] & 7 == 7


def test_quantize_global_scale():
    rng = np.random.default_rng(6)
    x = torch.from_numpy((rng.standard_normal((4, 64)) * 1e-4).astype(np.float32)).to(torch.bfloat16).float().numpy()
    g = ob.tensor_amax_scale(x)
    assert g == float(np.float32(np.max(np.abs(x))) / np.float32(2688.0))
    codes, scales = ob.quantize(x, g=g, nthreads=1)
    assert scales.max() == 0x7E or scales.max() == 0x7D      # the largest block lands at (or next to) 448
    # with a power-of-two g the result equals quantizing x/g without g
    g2 = 2.0 ** -20
    c1, s1 = ob.quantize(x, g=g2, nthreads=1)
    c2, s2 = ob.quantize(x / np.float32(g2), nthreads=1)
    assert np.array_equal(c1, c2) and np.array_equal(s1, s2)
    deq = ob.dequantize(c1, s1, g=g2)
    assert np.max(np.abs(deq - x)) <= np.max(np.abs(x)) * 0.26
    assert ob.tensor_amax_scale(np.zeros(5, dtype=np.float32)) == 1.0


def test_quantize_sr_uses_block_indexed_integers_and_is_reproducible():
    rng = np.random.default_rng(7)
    x = torch.from_numpy(rng.standard_normal((5, 64)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    c1, s1 = ob.quantize(x, mode=ob.SR, seed=11, offset=3, nthreads=1)
    c2, s2 = ob.quantize(x, mode=ob.SR, seed=11, offset=3, nthreads=4)
    assert np.array_equal(c1, c2) and np.array_equal(s1, s2)
    c3, _ = ob.quantize(x, mode=ob.SR, seed=11, offset=4, nthreads=1)
    assert not np.array_equal(c1, c3)
    crt, srt = ob.quantize(x, nthreads=1)
    assert np.array_equal(srt, s1)                           # scales do not depend on the rounding mode
    # rebuild every code from the per-element rule and the bytes of block r*(K/16)+kb
    for r in range(5):
        for kb in range(4):
            rnd = ob.block_random_u16(11, 3, r * 4 + kb)
            d = np.float32(ob.e4m3_decode(int(s1[r, kb])))
            inv = np.float32(1.0) / d
            for j in range(16):
                v = x[r, kb * 16 + j]
                y = min(np.float32(abs(v)) * inv, np.float32(6.0))
                m = ob.round_sr(float(y), int(rnd[j]))
                byte = c1[r, (kb * 16 + j) // 2]
                nib = (byte >> 4) if j & 1 else (byte & 15)
                assert nib == (m | (8 if np.signbit(v) else 0))


def test_quantize_rows_of_a_slice_equals_the_slice_of_the_whole():
    rng = np.random.default_rng(12)
    x = torch.from_numpy(rng.standard_normal((40, 64)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    for mode in (ob.RTN, ob.SR):
        c, s_ = ob.quantize(x, g=0.5, mode=mode, seed=3, offset=9, nthreads=1)
        c2, s2 = ob.quantize_rows(x[17:29], 17, g=0.5, mode=mode, seed=3, offset=9, nthreads=2)
        assert np.array_equal(c[17:29], c2) and np.array_equal(s_[17:29], s2)


def test_noise_sums_against_numpy_and_the_uniform_noise_closed_form():
    rng = np.random.default_rng(21)
    x = rng.uniform(-6, 6, (64, 256)).astype(np.float32)
    x[:, ::16] = 6.0                                          # every block: amax 6, scale exactly 1
    for mode in (ob.RTN, ob.SR):
        c, s_ = ob.quantize(x, mode=mode, seed=4, offset=0)
        e2, x2 = ob.noise_sums(x, c, s_)
        deq = ob.dequantize(c, s_).astype(np.float64)
        assert abs(e2 - np.sum((deq - x) ** 2)) <= 1e-9 * e2 and abs(x2 - np.sum(x.astype(np.float64) ** 2)) <= 1e-9 * x2
    # values uniform in [2, 3) (spacing 1): mean squared error 1/12 under RtN and 1/6 under SR (Section 4's
    # variance of the two roundings); blocks padded with one 6.0 so that the scale is 1
    y = rng.uniform(2, 3, (256, 256)).astype(np.float32)
    y[:, ::16] = 6.0
    n = y.size - y.size // 16
    for mode, want in ((ob.RTN, 1 / 12), (ob.SR, 1 / 6)):
        c, s_ = ob.quantize(y, mode=mode, seed=8, offset=1)
        e2, _ = ob.noise_sums(y, c, s_)
        assert abs(e2 / n - want) < 0.01 * want * 3


def test_matmul_nt_against_float64_library_matmul():
    rng = np.random.default_rng(31)
    A = rng.standard_normal((37, 96)).astype(np.float32)
    B = rng.standard_normal((21, 96)).astype(np.float32)
    D, T = ob.matmul_nt(A, B, nthreads=3)
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    assert np.array_equal(D, ref.astype(np.float32)) or np.max(np.abs(D - ref)) <= 1e-6 * np.max(np.abs(ref))
    assert np.allclose(T, np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64).T, rtol=1e-6)
    e = np.zeros((4, 16), dtype=np.float32); e[2, 5] = 1.0              # one-hot row picks a column of B
    D, _ = ob.matmul_nt(e, B[:, :16].copy())
    assert np.array_equal(D[2], B[:, 5]) and not D[[0, 1, 3]].any()


def test_quantize_transposed_is_row_quantize_of_the_transpose():
    rng = np.random.default_rng(8)
    x = torch.from_numpy(rng.standard_normal((32, 24)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    for mode in (ob.RTN, ob.SR):
        ct, st = ob.quantize(x, mode=mode, seed=5, offset=1, transposed=True, nthreads=1)
        cr, sr_ = ob.quantize(np.ascontiguousarray(x.T), mode=mode, seed=5, offset=1, nthreads=1)
        assert ct.shape == (24, 16) and st.shape == (24, 2)
        assert np.array_equal(ct, cr) and np.array_equal(st, sr_)


# ---------------------------------------------------------------- scale layout
def test_swizzled_scale_layout_structure():
    for Rq, nkb in [(128, 4), (256, 8), (130, 5), (1, 1), (384, 12)]:
        total = ob.sf_swizzled_bytes(Rq, nkb)
        assert total == -(-Rq // 128) * -(-nkb // 4) * 512
        offs = np.array([[ob.sf_swizzled_offset(r, kb, nkb) for kb in range(nkb)] for r in range(Rq)])
        assert len(np.unique(offs)) == Rq * nkb and offs.min() >= 0 and offs.max() < total
        if Rq % 128 == 0 and nkb % 4 == 0:
            assert sorted(offs.reshape(-1).tolist()) == list(range(total))   # a permutation
        lin = np.arange(Rq * nkb, dtype=np.uint32).astype(np.uint8).reshape(Rq, nkb)
        sw = ob.sf_swizzle(lin)
        assert np.array_equal(sw[offs.reshape(-1)], lin.reshape(-1))
        mask = np.ones(total, bool)
        mask[offs.reshape(-1)] = False
        assert np.all(sw[mask] == 0)
    o = lambda r, kb: ob.sf_swizzled_offset(r, kb, 8)
    # one 128x4 tile is 512 contiguous bytes; 4 blocks of a row are adjacent; rows r, r+32,
    # r+64, r+96 share a 16-byte group; consecutive rows are 16 bytes apart
    assert o(0, 0) == 0 and o(0, 3) == 3 and o(0, 4) == 512 and o(128, 0) == 1024
    assert o(1, 0) == 16 and o(31, 0) == 31 * 16
    assert o(32, 0) == 4 and o(64, 0) == 8 and o(96, 0) == 12 and o(127, 3) == 511


# ---------------------------------------------------------------- GEMM
def _rand_quantized(rng, R, K, std=1.0):
    x = torch.from_numpy((rng.standard_normal((R, K)) * std).astype(np.float32)).to(torch.bfloat16).float().numpy()
    return ob.quantize(x, nthreads=1)


def test_gemm_matches_library_matmul_in_float64():
    rng = np.random.default_rng(9)
    ac, asf = _rand_quantized(rng, 7, 96)
    bc, bsf = _rand_quantized(rng, 5, 96, std=0.02)
    ga, gb = 0.5, 2.0 ** -3
    D, T = ob.gemm(ac, asf, ga, bc, bsf, gb)
    A = torch.from_numpy(ob.dequantize(ac, asf)).double() * ga
    B = torch.from_numpy(ob.dequantize(bc, bsf)).double() * gb
    ref = (A @ B.T).numpy()
    refT = (A.abs() @ B.abs().T).numpy()
    assert np.allclose(D, ref, rtol=1e-6, atol=0)
    assert np.allclose(T, refT, rtol=1e-6, atol=0)
    Ds, Ts = ob.gemm_sampled(ac, asf, ga, bc, bsf, gb, [0, 6, 3], [4, 0, 2])
    assert np.array_equal(Ds, D[[0, 6, 3], [4, 0, 2]]) and np.array_equal(Ts, T[[0, 6, 3], [4, 0, 2]])
    D32 = ob.gemm_f32acc(ac, asf, ga, bc, bsf, gb)
    assert np.all(np.abs(D32 - D) <= 1e-6 * T)


def test_gemm_exact_small_integers_and_one_hot():
    # power-of-two scales, small K: every partial sum is exact -> equality with integer arithmetic
    rng = np.random.default_rng(10)
    grid = np.array(GRID + [-g for g in GRID], dtype=np.float32)
    A = rng.choice(grid, size=(6, 32))
    A[:, 0] = 6.0
    A[:, 16] = -6.0                                          # amax 6 per block -> scale exactly 1
    B = rng.choice(grid, size=(4, 32))
    B[:, 1] = 6.0
    B[:, 17] = 6.0
    ac, asf = ob.quantize(A.astype(np.float32), nthreads=1)
    bc, bsf = ob.quantize(B.astype(np.float32), nthreads=1)
    assert np.all(asf == ob.e4m3_encode(1.0)) and np.all(bsf == ob.e4m3_encode(1.0))
    D, T = ob.gemm(ac, asf, 1.0, bc, bsf, 1.0)
    assert np.array_equal(D, (A.astype(np.float64) @ B.astype(np.float64).T).astype(np.float32))
    # a one-hot row of A reads back a column of dequantized B
    E = np.zeros((32, 32), dtype=np.float32)
    E[np.arange(32), np.arange(32)] = 6.0
    ec, esf = ob.quantize(E, nthreads=1)
    D2 = ob.gemm(ec, esf, 1.0, bc, bsf, 1.0, want_T=False)
    assert np.array_equal(D2, 6.0 * ob.dequantize(bc, bsf).T)


def test_gemm_transposed_operand_detected():
    # a swapped-operand or transposed-output mistake changes the shape-asymmetric result
    rng = np.random.default_rng(11)
    ac, asf = _rand_quantized(rng, 3, 32)
    bc, bsf = _rand_quantized(rng, 5, 32)
    D = ob.gemm(ac, asf, 1.0, bc, bsf, 1.0, want_T=False)
    A, B = ob.dequantize(ac, asf).astype(np.float64), ob.dequantize(bc, bsf).astype(np.float64)
    assert D.shape == (3, 5)
    assert np.allclose(D, A @ B.T, rtol=1e-6)


# ---------------------------------------------------------------- MXFP4 (blocks of 32, E8M0 scales)
def test_e8m0_is_the_power_of_two_ladder_and_encode_rounds_up():
    import math
    for code in range(0, 255):
        assert ob.e8m0_decode(code) == math.ldexp(1.0, code - 127)
        assert ob.e8m0_encode_up(ob.e8m0_decode(code)) == code               # powers of two map to themselves
    rng = np.random.default_rng(41)
    for v in np.concatenate([rng.uniform(1e-30, 1e30, 300), 2.0 ** rng.uniform(-120, 120, 300)]).astype(np.float32):
        c = ob.e8m0_encode_up(float(v))
        assert Fraction(ob.e8m0_decode(c)) >= Fraction(float(v))             # never below the value ...
        assert c == 0 or Fraction(ob.e8m0_decode(c - 1)) < Fraction(float(v))   # ... and the smallest such power
    assert ob.e8m0_encode_up(0.0) == 0 and ob.e8m0_encode_up(float(np.float32(3e38))) == 254


def test_mx_block_quantizer_by_exhaustive_definition():
    rng = np.random.default_rng(42)
    x = torch.from_numpy((rng.standard_normal((6, 96)) * rng.choice([1e-3, 1.0, 40.0], (6, 1))).astype(np.float32)) \
        .to(torch.bfloat16).float().numpy()
    codes, scales = ob.quantize_mx(x, nthreads=1)
    assert codes.shape == (6, 48) and scales.shape == (6, 3)
    for r in range(6):
        for kb in range(3):
            blk = x[r, kb * 32:(kb + 1) * 32]
            amax = Fraction(float(np.max(np.abs(blk))))
            d = Fraction(ob.e8m0_decode(int(scales[r, kb])))
            assert d * 6 >= amax * Fraction(1 - 2 ** -20) and d * 3 < amax * Fraction(1 + 2 ** -20)   # amax/d in (3, 6]
            for j in range(32):
                byte = codes[r, (kb * 32 + j) // 2]
                nib = (byte >> 4) if j & 1 else (byte & 15)
                y = Fraction(float(abs(blk[j]))) / d
                dist = [abs(y - g) for g in GRID_F]
                assert dist[nib & 7] == min(dist) and (nib >> 3) == int(np.signbit(blk[j]))
    # nothing clips: the largest element of every block lands on code 5, 6 or 7 (3 < y <= 6)
    assert np.all(np.maximum((codes & 7), (codes >> 4) & 7).reshape(6, 3, 16).max(axis=2) >= 5)
    deq = ob.dequantize_mx(codes, scales)
    d_all = np.array([[ob.e8m0_decode(int(b)) for b in row] for row in scales]).repeat(32, axis=1)
    assert np.all(np.abs(deq - x) <= d_all)                  # half of the widest grid step (2) times the scale


def test_mx_sr_draws_per_group_of_16_like_nvfp4_and_slices_compose():
    rng = np.random.default_rng(43)
    x = torch.from_numpy(rng.standard_normal((9, 64)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    c, s_ = ob.quantize_mx(x, mode=ob.SR, seed=5, offset=2, nthreads=1)
    for r in range(9):
        for k16 in range(4):
            rnd = ob.block_random_u16(5, 2, r * 4 + k16)
            inv = np.float32(1.0) / np.float32(ob.e8m0_decode(int(s_[r, k16 // 2])))
            for j in range(16):
                v = x[r, k16 * 16 + j]
                y = min(np.float32(abs(v)) * inv, np.float32(6.0))
                byte = c[r, (k16 * 16 + j) // 2]
                nib = (byte >> 4) if j & 1 else (byte & 15)
                assert nib == (ob.round_sr(float(y), int(rnd[j])) | (8 if np.signbit(v) else 0))
    c2, s2 = ob.quantize_mx(x[3:7], mode=ob.SR, seed=5, offset=2, first_row=3, nthreads=2)
    assert np.array_equal(c[3:7], c2) and np.array_equal(s_[3:7], s2)
    # transposed = row quantization of the materialised transpose
    y = np.ascontiguousarray(x[:, :32])                                              # [9, 32] -> transpose has Kq = 9: pad rows
    y = np.concatenate([y, np.zeros((23, 32), dtype=np.float32)])                    # [32, 32]
    ct, st = ob.quantize_mx(y, mode=ob.SR, seed=5, offset=2, transposed=True)
    cr, sr_ = ob.quantize_mx(np.ascontiguousarray(y.T), mode=ob.SR, seed=5, offset=2)
    assert np.array_equal(ct, cr) and np.array_equal(st, sr_)


def test_mx_gemm_against_float64_matmul_of_dequantized_operands():
    rng = np.random.default_rng(44)
    A = rng.standard_normal((20, 128)).astype(np.float32)
    B = (rng.standard_normal((12, 128)) * 0.03).astype(np.float32)
    ac, asf = ob.quantize_mx(A, g=0.5)
    bc, bsf = ob.quantize_mx(B, g=0.25)
    D, T = ob.gemm_mx(ac, asf, 0.5, bc, bsf, 0.25, nthreads=2)
    da = ob.dequantize_mx(ac, asf, 0.5).astype(np.float64)
    db = ob.dequantize_mx(bc, bsf, 0.25).astype(np.float64)
    assert np.allclose(D, da @ db.T, rtol=1e-6, atol=1e-9)
    assert np.allclose(T, np.abs(da) @ np.abs(db).T, rtol=1e-6)
