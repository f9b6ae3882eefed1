"""Pins of the SCALE the oracle's quantizer computes, against the definition of Sec. 3.1:

    s = max|x| / rho,      x^ = s * round(x / s) = (max|x| / rho) * round(rho x / max|x|)

with rho the largest magnitude of the format.  Consequences that hold for that scale and for no other:
the largest element of every scale block lands exactly on the last grid point (+-rho), the stored scale
times rho gives the block's maximum back, and so does dequantizing that element.  The block extents, the
code layout and rho are written out here independently of the oracle (numpy slicing, closed-form code
values), so a wrong constant, a wrong extent or a swapped operand in the oracle's make_scale fails.
"""
import numpy as np
import pytest

import oracle
from oracle import (ADAM, FP8_E4M3, FP8_E5M2, GRAD_NATIVE, INT4, PER_BLOCK, PER_ROW, PER_TENSOR, RTN, SCALE_BF16,
                    SCALE_NATIVE, SGDM, SR)

# format -> (rho, magnitude code of rho): E4M3 S.1111.110 = 448, E5M2 S.11110.11 = 57344, INT4 7
RHO = {FP8_E4M3: (448.0, 0x7E), FP8_E5M2: (57344.0, 0x7B), INT4: (7.0, 7)}


def blocks_of(gran, block, rows, cols):
    """(row-major begin, length) of every scale block, from the granularity's plain meaning."""
    if gran == PER_TENSOR:
        return [(0, rows * cols)]
    if gran == PER_ROW:
        return [(r * cols, cols) for r in range(rows)]
    return [(r * cols + c0, min(block, cols - c0)) for r in range(rows) for c0 in range(0, cols, block)]


def code_of(fmt, w, i):
    """(magnitude code, negative?) of element i."""
    if fmt == INT4:
        nib = (int(w[i >> 1]) >> (4 * (i & 1))) & 0xF          # even element in the low nibble
        v = nib - 16 if nib >= 8 else nib
        return abs(v), v < 0
    return int(w[i]) & 0x7F, bool(int(w[i]) & 0x80)


def scale_values(s):
    return (s.astype(np.uint32) << 16).view(np.float32) if s.dtype == np.uint16 else s


def check_blocks(fmt, gran, block, sdt, x, w, s):
    """x: what was quantized (float32 [rows, cols]); w, s: the oracle's codes and scales."""
    rho, rho_code = RHO[fmt]
    rows, cols = x.shape
    flat = x.ravel().astype(np.float64)
    sv = scale_values(s).astype(np.float64)
    deq = oracle.dequantize(oracle.Config(format=fmt, granularity=gran, block=block, scale_dtype=sdt), w, s, rows, cols,
                            np.float32).ravel().astype(np.float64)
    # one unit in the last place of the stored scale's type, relative
    ulp = 2.0 ** -7 if sdt == SCALE_BF16 else 2.0 ** -23
    ext = blocks_of(gran, block, rows, cols)
    assert len(ext) == s.size
    seen_nonzero = 0
    for k, (b, n) in enumerate(ext):
        seg = flat[b: b + n]
        amax = np.abs(seg).max()
        if amax == 0.0:
            assert sv[k] == 1.0                                              # all-zero block: s = 1, codes 0
            assert all(code_of(fmt, w, b + j)[0] == 0 for j in range(n))
            continue
        seen_nonzero += 1
        j = int(np.abs(seg).argmax())
        mag, neg = code_of(fmt, w, b + j)
        assert mag == rho_code, f"block {k}: the largest element has code {mag:#x}, not rho's {rho_code:#x}"
        assert neg == (seg[j] < 0)
        assert abs(sv[k] * rho - amax) <= ulp * amax, f"block {k}: s*rho = {sv[k] * rho!r}, max|x| = {amax!r}"
        assert abs(abs(deq[b + j]) - amax) <= ulp * amax                   # x^ of the largest element is max|x|
        assert (np.abs(deq[b: b + n]) <= sv[k] * rho * (1 + 2.0 ** -23)).all()  # nothing overflows the grid (binary32 product)
    assert seen_nonzero >= 1


CASES = [(fmt, gran, block, sdt)
         for fmt in (FP8_E4M3, FP8_E5M2, INT4)
         for gran, block in ((PER_TENSOR, 128), (PER_ROW, 128), (PER_BLOCK, 128), (PER_BLOCK, 32))
         for sdt in (SCALE_NATIVE, SCALE_BF16)]


def pin_quantize(fmt, gran, block, sdt, seed=31):
    rng = np.random.default_rng(seed)
    rows, cols = 5, 334                                  # 334 = 2*128 + 78 = 10*32 + 14: ragged last blocks
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    x[1, :128] = 0.0                                      # an all-zero 1x128 (and four 1x32) block
    x[3, 300] = -0.5                                      # a negative maximum inside a ragged last block
    cfg = oracle.Config(format=fmt, granularity=gran, block=block, scale_dtype=sdt, rounding=RTN)
    w, s = oracle.quantize(cfg, x)
    check_blocks(fmt, gran, block, sdt, x, w, s)


def pin_step(fmt, gran, block, sdt, opt, seed=32):
    """The same through one training step: the scale written by ECO_QUANTIZE is max|theta~| / rho of the
    tentative weights theta~ (Algorithm 1, line 2, with q of Sec. 3.1)."""
    rng = np.random.default_rng(seed)
    rows, cols = 4, 334
    n = rows * cols
    cfg = oracle.Config(format=fmt, granularity=gran, block=block, scale_dtype=sdt, optimizer=opt, rounding=RTN,
                        grad_dtype=GRAD_NATIVE)
    w, s = oracle.quantize(cfg, (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32))
    m = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    v = rng.uniform(1e-7, 1e-5, n).astype(np.float32) if opt == ADAM else None
    g = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    tht = np.zeros(n, np.float32)
    oracle.step(cfg, lr=1e-2, beta1=0.9, beta2=0.95, eps=1e-8, step=3, seed=5, w=w, scale=s, grad=g, m=m, v=v,
                rows=rows, cols=cols, dbg_theta_tilde=tht)
    check_blocks(fmt, gran, block, sdt, tht.reshape(rows, cols), w, s)


@pytest.mark.parametrize("fmt,gran,block,sdt", CASES)
def test_largest_element_of_every_block_lands_on_rho_and_scale_times_rho_is_the_maximum(fmt, gran, block, sdt):
    pin_quantize(fmt, gran, block, sdt)


@pytest.mark.parametrize("opt", [SGDM, ADAM])
@pytest.mark.parametrize("fmt,gran,block,sdt", CASES[::3])
def test_scale_after_a_step_is_the_maximum_of_the_tentative_weights_over_rho(fmt, gran, block, sdt, opt):
    pin_step(fmt, gran, block, sdt, opt)


def test_worked_example_by_hand():
    """A block small enough to do on paper.  INT4, rho = 7: x = (0.7, -0.35, 0.16, 0) has max 0.7, s = 0.1,
    x / s = (7, -3.5, 1.6, 0) -> (7, -4, 2, 0) (the tie -3.5 goes to the even -4).  E4M3, rho = 448:
    x = (448, 100, -13, 0.5) has s = 1 and codes 0x7E, 0x6C (100 is the midpoint of the
    neighbours 96 and 104; the tie goes to the even code, 96), 0xD5 (-13), 0x30 (0.5)."""
    cfg = oracle.Config(format=INT4, granularity=PER_TENSOR, rounding=RTN)
    w, s = oracle.quantize(cfg, np.array([[0.7, -0.35, 0.16, 0.0]], np.float64))
    assert abs(s[0] - 0.1) < 1e-15
    assert [code_of(INT4, w, i) for i in range(4)] == [(7, False), (4, True), (2, False), (0, False)]
    cfg = oracle.Config(format=FP8_E4M3, granularity=PER_TENSOR, rounding=RTN)
    w, s = oracle.quantize(cfg, np.array([[448.0, 100.0, -13.0, 0.5]], np.float64))
    assert s[0] == 1.0
    assert list(w) == [0x7E, 0x6C, 0xD5, 0x30]


@pytest.mark.parametrize("gran,block", [(PER_BLOCK, 128), (PER_ROW, 128), (PER_BLOCK, 32)])
@pytest.mark.parametrize("fmt", [FP8_E4M3, INT4])
def test_a_slice_of_rows_with_its_position_rounds_like_the_whole_tensor(fmt, gran, block):
    """Stochastic rounding draws one word per POSITION in the whole tensor (row-major index, words grouped by four):
    quantizing or stepping rows r0..r1 alone, told where they sit, gives the bits those rows get inside the whole
    tensor.  Scales per row or per block do not see the cut."""
    rng = np.random.default_rng(33)
    rows, cols, r0, r1 = 9, 200, 3, 7
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    cfg = oracle.Config(format=fmt, granularity=gran, block=block, rounding=SR, optimizer=SGDM)
    bpe = 2 if fmt == INT4 else 1                            # elements per code byte
    spr = 1 if gran == PER_ROW else -(-cols // block)        # scales per row
    w, s = oracle.quantize(cfg, x, seed=9, step=4, tensor_id=6)
    ws, ss = oracle.quantize(cfg, x[r0:r1], seed=9, step=4, tensor_id=6, index_base=r0 * cols)
    assert (ws == w[r0 * cols // bpe: r1 * cols // bpe]).all() and (ss == s[r0 * spr: r1 * spr]).all()
    w0, _ = oracle.quantize(cfg, x[r0:r1], seed=9, step=4, tensor_id=6)          # without its position: other words
    assert (w0 != ws).any()
    # and through a step
    from paper_2601_22101_b200.workloads import f32_to_bf16_bits
    g = f32_to_bf16_bits((rng.standard_normal(rows * cols) * 1e-3).astype(np.float32))
    m = (rng.standard_normal(rows * cols) * 1e-4).astype(np.float32)
    sl = slice(r0 * cols, r1 * cols)
    ms, gs = m[sl].copy(), g[sl].copy()
    oracle.step(cfg, lr=1e-2, beta1=0.9, step=2, seed=11, w=w, scale=s, grad=g, m=m, rows=rows, cols=cols, tensor_id=6)
    oracle.step(cfg, lr=1e-2, beta1=0.9, step=2, seed=11, w=ws, scale=ss, grad=gs, m=ms, rows=r1 - r0, cols=cols,
                tensor_id=6, index_base=r0 * cols)
    assert (ws == w[r0 * cols // bpe: r1 * cols // bpe]).all() and (ss == s[r0 * spr: r1 * spr]).all()
    assert (ms.view(np.int32) == m[sl].view(np.int32)).all()


def test_position_enters_the_counter_as_a_64_bit_sum():
    """Word of local element i at position base + i, for bases around 2^32 (the counter is (base + i) div 4)."""
    seed, step, tid = 77, 5, 3
    for base in (0, 4, 2 ** 32 - 8, 2 ** 32, 2 ** 33 + 2 ** 20):
        x = np.full((1, 8), 0.3, np.float64)
        x[0, 0] = 1.0                                        # s = 1/7: every other element sits at 2.1, frac 0.1
        cfg = oracle.Config(format=INT4, granularity=PER_TENSOR, rounding=SR)
        w, _ = oracle.quantize(cfg, x, seed=seed, step=step, tensor_id=tid, index_base=base)
        for i in range(1, 8):
            pos = base + i                                   # the counter written out here, not asked of the oracle
            word = int(oracle.philox4x32_10([(pos >> 2) & 0xFFFFFFFF, tid, step & 0xFFFFFFFF, step >> 32],
                                            [seed & 0xFFFFFFFF, seed >> 32])[pos & 3])
            up = (word >> 8) < (np.float64(0.3) * (7.0 / 1.0) - 2.0) * 2 ** 24
            assert code_of(INT4, w, i)[0] == (3 if up else 2), (base, i)
