"""Pins of the oracle's power-of-two block scales (one exponent byte per block of 32 elements, the
shared-scale layout of microscaling formats that Sec. 3.1 cites among the group-wise schemes).

The scale is the smallest power of two s with s * rho >= max|x| (like s = max|x| / rho of Sec. 3.1 it
prevents overflow).  Pinned here against exact rational arithmetic, a library decode of the exponent byte,
the power-of-two invariance that only such scales have, and the block layout."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import FP8_E4M3, FP8_E5M2, INT4, PER_BLOCK, RTN, SCALE_E8M0, SR

RHO = {FP8_E4M3: 448, FP8_E5M2: 57344, INT4: 7}


def _cfg(fmt, rnd=RTN, block=32):
    return oracle.Config(format=fmt, granularity=PER_BLOCK, block=block, scale_dtype=SCALE_E8M0, rounding=rnd)


def _exponent_by_search(amax: float, rho: int) -> int:
    """Smallest e in -127..127 with 2^e * rho >= amax, by exact rational comparison of every candidate."""
    a = Fraction(amax)
    for e in range(-127, 128):
        if Fraction(2) ** e * rho >= a:
            return e
    return 127


@pytest.mark.parametrize("fmt", [FP8_E4M3, FP8_E5M2, INT4])
def test_exponent_byte_is_the_smallest_power_of_two_that_avoids_overflow(fmt):
    rng = np.random.default_rng(3)
    rho = RHO[fmt]
    vals = list(np.exp2(rng.uniform(-125, 110, 300)).astype(np.float32))
    for k in (-100, -20, -1, 0, 1, 9, 60):          # exactly rho * 2^k and its two binary32 neighbours
        c = np.float32(rho * 2.0 ** k)
        vals += [c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(0))]
    vals += [np.float32(1.0), np.float32(2.0 ** -140), np.float32(3e38)]
    x = np.zeros((len(vals), 32), dtype=np.float32)
    x[np.arange(len(vals)), rng.integers(0, 32, len(vals))] = np.array(vals) * rng.choice([-1.0, 1.0], len(vals))
    _, s = oracle.quantize(_cfg(fmt), x)
    assert s.dtype == np.uint8 and s.shape == (len(vals),)
    want = np.array([_exponent_by_search(float(v), rho) + 127 for v in vals])
    assert (s == want).all()
    assert s.max() < 255


def test_exponent_byte_decodes_like_the_library_type_and_zero_block_is_one():
    x = np.zeros((3, 64), dtype=np.float32)
    x[0, :32] = 448.0 * 2.0 ** -30
    x[1, 40] = -448.0 * 2.0 ** 20
    x[2, 5] = 1.0
    w, s = oracle.quantize(_cfg(FP8_E4M3), x)
    lib = torch.from_numpy(s.copy()).view(torch.float8_e8m0fnu).to(torch.float32).numpy()
    assert list(lib) == [2.0 ** -30, 1.0, 1.0, 2.0 ** 20, 2.0 ** -8, 1.0]     # all-zero blocks: s = 1
    back = oracle.dequantize(_cfg(FP8_E4M3), w, s, 3, 64)
    assert (back == x).all()                                                   # these values are on the grid


@pytest.mark.parametrize("fmt,rnd", [(FP8_E4M3, SR), (FP8_E5M2, RTN), (INT4, SR)])
def test_scaling_by_a_power_of_two_moves_only_the_exponent_byte(fmt, rnd):
    """With s a power of two, x / s is exact, so q(2^k x) has the codes of q(x) and exponent bytes k higher;
    no other scale choice has this property, and it ties make_scale, the grid factor and the rounding together."""
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((5, 200)) * 0.02).astype(np.float32)
    w0, s0 = oracle.quantize(_cfg(fmt, rnd), x, seed=9, step=4, tensor_id=2)
    for k in (-13, 7):
        w1, s1 = oracle.quantize(_cfg(fmt, rnd), x * np.float32(2.0 ** k), seed=9, step=4, tensor_id=2)
        assert (w1 == w0).all() and (s1.astype(int) == s0.astype(int) + k).all()
    # and the reconstruction error of round-to-nearest is at most half a grid step of the block
    if rnd == RTN:
        back = oracle.dequantize(_cfg(fmt, rnd), w0, s0, 5, 200)
        step = np.repeat(np.exp2(s0.astype(float) - 127).reshape(5, 7), 32, axis=1)[:, :200] * RHO[fmt] / 4
        assert (np.abs(back - x) <= step / 2).all()      # mantissa of 2 bits: gap <= rho * s / 4 at the top binade


def test_block_layout_ragged_columns_and_locality():
    """Blocks are 32 consecutive elements of one row, a row's last block may be short, and a scale depends on
    its own block only."""
    rng = np.random.default_rng(6)
    rows, cols = 4, 75                                 # 3 blocks per row: 32, 32, 11
    cfg = _cfg(FP8_E4M3)
    assert cfg.n_scales(rows, cols) == 12
    x = (rng.standard_normal((rows, cols)) * 0.1).astype(np.float32)
    w0, s0 = oracle.quantize(cfg, x)
    for (r, c) in [(0, 0), (1, 31), (2, 32), (3, 74), (1, 64)]:
        y = x.copy()
        y[r, c] = 1000.0
        w1, s1 = oracle.quantize(cfg, y)
        changed = np.flatnonzero(s1 != s0)
        assert list(changed) == [r * 3 + c // 32]
        same = np.ones((rows, cols), dtype=bool)
        same[r, (c // 32) * 32:(c // 32) * 32 + 32] = False
        assert (w1.reshape(rows, cols)[same] == w0.reshape(rows, cols)[same]).all()
    # equal to quantizing every block on its own as a one-row tensor
    for r in range(rows):
        for j in range(3):
            blk = x[r:r + 1, j * 32:min(cols, j * 32 + 32)]
            wb, sb = oracle.quantize(cfg, blk)
            assert sb[0] == s0[r * 3 + j] and (wb == w0.reshape(rows, cols)[r, j * 32:j * 32 + blk.shape[1]]).all()
