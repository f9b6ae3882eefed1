"""Pins of the oracle's number formats and rounding rules (Sec. 3.1, "Quantization":
grid, rho, round-to-nearest, stochastic rounding) against closed forms, brute
force over every code, and a library cast."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import FP8_E4M3, INT4, RTN, SR


def _e4m3_closed_form(code: int) -> float:
    s, E, M = code >> 7, (code >> 3) & 15, code & 7
    if E == 15 and M == 7:
        return math.nan
    mag = M * 2.0 ** -9 if E == 0 else 2.0 ** (E - 7) * (1 + M / 8)
    return -mag if s else mag


def test_e4m3_decode_all_codes_closed_form_and_library():
    lib_vals = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    for c in range(256):
        v = oracle.code_value(FP8_E4M3, c)
        ref = _e4m3_closed_form(c)
        if math.isnan(ref):
            assert math.isnan(v) and math.isnan(lib_vals[c])
        else:
            assert v == ref == lib_vals[c], c
    assert oracle.code_value(FP8_E4M3, 0x7E) == 448.0        # rho: largest finite magnitude
    assert oracle.code_value(FP8_E4M3, 0x01) == 2.0 ** -9    # smallest subnormal
    assert oracle.code_value(FP8_E4M3, 0x08) == 2.0 ** -6    # smallest normal


def test_int4_decode_all_codes():
    for c in range(16):
        assert oracle.code_value(INT4, c) == (c - 16 if c >= 8 else c)


def test_e4m3_monotone_and_round_trip():
    mags = [oracle.code_value(FP8_E4M3, c) for c in range(0x7F)]
    assert all(b > a for a, b in zip(mags, mags[1:]))
    for dtype in (np.float32, np.float64):
        y = np.array(mags + [-m for m in mags], dtype=dtype)
        codes = oracle.round_to_codes(FP8_E4M3, RTN, y)
        assert list(codes[:0x7F]) == list(range(0x7F))
        assert list(codes[0x7F:]) == [0x80 | c for c in range(0x7F)]
        # on-grid values never move under stochastic rounding either, whatever the word
        for r in (0, 0xFFFFFFFF, 0x80000000):
            assert (oracle.round_to_codes(FP8_E4M3, SR, y, np.full(y.size, r, np.uint32)) == codes).all()


def test_e4m3_midpoints_go_to_even_code_and_neighbours_to_nearest():
    for c in range(0x7E):
        lo, hi = oracle.code_value(FP8_E4M3, c), oracle.code_value(FP8_E4M3, c + 1)
        mid = (lo + hi) / 2          # exact in binary32: one more mantissa bit
        even = c if c % 2 == 0 else c + 1
        for dtype in (np.float32, np.float64):
            y = np.array([mid, np.nextafter(dtype(mid), dtype(0)), np.nextafter(dtype(mid), dtype(1e9)),
                          -mid], dtype=dtype)
            got = oracle.round_to_codes(FP8_E4M3, RTN, y)
            assert list(got) == [even, c, c + 1, 0x80 | even], (c, list(got))


def test_saturation_and_never_nan_or_minus_eight():
    y = np.array([448.0, 449.0, 464.0, 1e9, np.inf, np.nan, -449.0, -np.inf, -1e30], dtype=np.float32)
    for mode in (RTN, SR):
        codes = oracle.round_to_codes(FP8_E4M3, mode, y, np.full(y.size, 1, np.uint32))
        assert all((c & 0x7F) == 0x7E for c in codes)
        assert list(codes[6:] >> 7) == [1, 1, 1]
    # a NaN takes +rho whatever its sign bit (processors differ in the sign of the NaN an operation returns)
    nans = np.array([0x7FC00000, 0xFFC00000, 0x7F800001, 0xFFFFFFFF], np.uint32).view(np.float32)
    for mode in (RTN, SR):
        assert list(oracle.round_to_codes(FP8_E4M3, mode, nans, np.zeros(4, np.uint32))) == [0x7E] * 4
        assert list(oracle.round_to_codes(INT4, mode, nans, np.zeros(4, np.uint32))) == [7] * 4
    y4 = np.array([7.0, 7.4, 7.5, 8.0, 100.0, np.inf, -7.5, -100.0], dtype=np.float32)
    for mode in (RTN, SR):
        codes = oracle.round_to_codes(INT4, mode, y4, np.zeros(y4.size, np.uint32))
        assert list(codes) == [7, 7, 7, 7, 7, 7, 9, 9]       # 9 = -7 in a two's-complement nibble
    rng = np.random.default_rng(0)
    y = (rng.standard_normal(200000) * 300).astype(np.float32)
    r = rng.integers(0, 2 ** 32, y.size, dtype=np.uint32)
    c8 = oracle.round_to_codes(FP8_E4M3, SR, y, r)
    assert ((c8 & 0x7F) != 0x7F).all()
    c4 = oracle.round_to_codes(INT4, SR, (y / 40).astype(np.float32), r)
    assert (c4 != 8).all()


def test_e4m3_rtn_matches_library_cast():
    rng = np.random.default_rng(1)
    parts = [rng.uniform(-448, 448, 200000), rng.standard_normal(200000) * 0.01,
             rng.standard_normal(200000) * 2.0 ** -8, rng.standard_normal(100000) * 30]
    y = np.clip(np.concatenate(parts), -448, 448).astype(np.float32)
    lib_codes = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = oracle.round_to_codes(FP8_E4M3, RTN, y)
    assert (got == lib_codes).all()


def test_int4_rtn_matches_rint():
    rng = np.random.default_rng(2)
    y = np.concatenate([rng.uniform(-7, 7, 100000), np.arange(-7, 7.5, 0.5)]).astype(np.float32)
    got = oracle.round_to_codes(INT4, RTN, y).astype(np.int64)
    vals = np.where(got >= 8, got - 16, got)
    assert (vals == np.rint(y).astype(np.int64)).all()    # np.rint: ties to even


@pytest.mark.parametrize("fmt,lo,gap", [
    (FP8_E4M3, 1.0, 0.125), (FP8_E4M3, 320.0, 32.0), (FP8_E4M3, 3 * 2.0 ** -9, 2.0 ** -9),
    (FP8_E4M3, 2.0 ** -6, 2.0 ** -9), (INT4, 3.0, 1.0), (INT4, 0.0, 1.0)])
def test_sr_probability_by_enumeration(fmt, lo, gap):
    """P(up) = ceil(frac * 2^24) / 2^24, counted over every 24-bit threshold."""
    u = np.arange(2 ** 24, dtype=np.uint32)
    r = (u << 8) | 0x5A                       # the low 8 bits of the word are ignored
    code_lo = int(oracle.round_to_codes(fmt, RTN, np.array([lo], np.float32))[0])
    for frac in (0.0, 2.0 ** -24, 3 * 2.0 ** -24, 0.25, 1 / 3, 0.5, 1 - 2.0 ** -20):
        y = np.float32(lo + frac * gap)
        true_frac = (float(y) - lo) / gap     # after the cast to binary32
        codes = oracle.round_to_codes(fmt, SR, np.full(u.size, y, np.float32), r)
        ups = int((codes == code_lo + 1).sum())
        assert ups + int((codes == code_lo).sum()) == u.size   # only the two neighbours
        assert ups == math.ceil(true_frac * 2 ** 24), (frac, ups)


@pytest.mark.parametrize("fmt,scale", [(FP8_E4M3, 300.0), (FP8_E4M3, 1.0), (FP8_E4M3, 2.0 ** -7), (INT4, 6.9)])
def test_sr_unbiased_monte_carlo(fmt, scale):
    """Mean of the rounded value equals the value (Sec. 3.1: SR is an unbiased estimator)."""
    rng = np.random.default_rng(3)
    vals = np.array([oracle.code_value(fmt, c) for c in range(256 if fmt == FP8_E4M3 else 16)])
    y = (rng.uniform(-1, 1, 64) * scale).astype(np.float32)
    n = 200000
    for yi in y:
        r = rng.integers(0, 2 ** 32, n, dtype=np.uint32)
        codes = oracle.round_to_codes(fmt, SR, np.full(n, yi, np.float32), r)
        q = vals[codes]
        distinct = np.unique(q)
        assert distinct.size <= 2
        if distinct.size == 2:
            gap = distinct[1] - distinct[0]
            assert distinct[0] < yi < distinct[1]
            sigma = gap / 2 / math.sqrt(n)
            assert abs(q.mean() - float(yi)) < 5 * sigma
        else:
            assert distinct[0] == float(yi)


def test_bf16_rounding_matches_library():
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-30, 30, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38]]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().astype(np.uint16)
    got = np.array([oracle.f32_to_bf16(v) for v in x], dtype=np.uint16)
    assert (got == ref).all()


# --------------------------------------------------------------------------- FP8-E5M2 (a further format on the same skeleton)
def _e5m2_closed_form(code: int) -> float:
    s, E, M = code >> 7, (code >> 2) & 31, code & 3
    if E == 31:
        mag = math.inf if M == 0 else math.nan
    else:
        mag = M * 2.0 ** -16 if E == 0 else 2.0 ** (E - 15) * (1 + M / 4)
    return -mag if s else mag


def test_e5m2_decode_all_codes_closed_form_and_library():
    from oracle import FP8_E5M2
    lib_vals = torch.arange(256, dtype=torch.uint8).view(torch.float8_e5m2).to(torch.float64).numpy()
    for c in range(256):
        v, ref = oracle.code_value(FP8_E5M2, c), _e5m2_closed_form(c)
        if math.isnan(ref):
            assert math.isnan(v) and math.isnan(lib_vals[c])
        else:
            assert v == ref == lib_vals[c], c
    assert oracle.code_value(FP8_E5M2, 0x7B) == 57344.0       # rho: largest finite magnitude
    assert oracle.code_value(FP8_E5M2, 0x01) == 2.0 ** -16    # smallest subnormal
    assert oracle.code_value(FP8_E5M2, 0x04) == 2.0 ** -14    # smallest normal


def test_e5m2_round_trip_midpoints_saturation_and_library_cast():
    from oracle import FP8_E5M2
    mags = [oracle.code_value(FP8_E5M2, c) for c in range(0x7C)]          # finite magnitudes
    assert all(b > a for a, b in zip(mags, mags[1:]))
    for dtype in (np.float32, np.float64):
        y = np.array(mags + [-m for m in mags], dtype=dtype)
        codes = oracle.round_to_codes(FP8_E5M2, RTN, y)
        assert list(codes[:0x7C]) == list(range(0x7C)) and list(codes[0x7C:]) == [0x80 | c for c in range(0x7C)]
        for r in (0, 0xFFFFFFFF):
            assert (oracle.round_to_codes(FP8_E5M2, SR, y, np.full(y.size, r, np.uint32)) == codes).all()
    for c in range(0x7B):                                                    # midpoints go to the even code
        mid = (mags[c] + mags[c + 1]) / 2
        even = c if c % 2 == 0 else c + 1
        got = oracle.round_to_codes(FP8_E5M2, RTN, np.array([mid, np.nextafter(np.float32(mid), np.float32(0)),
                                                             np.nextafter(np.float32(mid), np.float32(1e9))], np.float32))
        assert list(got) == [even, c, c + 1], c
    big = np.array([57344.0, 60000.0, 1e9, np.inf, -1e9, np.nan], np.float32)   # saturate, never inf / NaN codes
    assert list(oracle.round_to_codes(FP8_E5M2, RTN, big)) == [0x7B, 0x7B, 0x7B, 0x7B, 0xFB, 0x7B]
    rng = np.random.default_rng(5)
    y = np.concatenate([rng.standard_normal(20000) * s for s in (1e-6, 1e-3, 1.0, 1e3)]).astype(np.float32)
    y = y[np.abs(y) < 57344]
    lib = torch.from_numpy(y).to(torch.float8_e5m2).view(torch.uint8).numpy()
    assert (oracle.round_to_codes(FP8_E5M2, RTN, y) == lib).all()


def test_e5m2_sr_probability_by_enumeration():
    from oracle import FP8_E5M2
    lo, gap = 1.25, 0.25                                     # between codes 1.25 and 1.5 (binade [1, 2), spacing 1/4)
    for frac in (0.0, 2.0 ** -21, 0.3, 0.5, 1 - 2.0 ** -21):
        y = np.float32(lo + frac * gap)
        f = (float(y) - lo) / gap
        words = (np.arange(0, 1 << 24, 4099, dtype=np.uint64) << 8).astype(np.uint32)
        codes = oracle.round_to_codes(FP8_E5M2, SR, np.full(words.size, y, np.float32), words)
        up = codes != oracle.round_to_codes(FP8_E5M2, RTN, np.array([lo], np.float32))[0]
        expect = (words >> 8).astype(np.float64) < f * 2 ** 24
        assert (up == expect).all()
