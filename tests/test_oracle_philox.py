"""Pins of the oracle's Philox4x32-10 against a library generator (cuRAND's host
Philox4_32_10 generator, which runs on the CPU) and against what the published
construction fixes (Weyl constants, bijectivity, avalanche)."""
import ctypes
import glob
import math
import os

import numpy as np
import pytest

import oracle


def _find_curand():
    pats = ["/usr/local/cuda/targets/x86_64-linux/lib/libcurand.so.10",
            "/usr/local/cuda*/targets/x86_64-linux/lib/libcurand.so*",
            "/usr/local/cuda*/lib64/libcurand.so*"]
    try:
        import nvidia.curand  # type: ignore
        pats.append(os.path.join(os.path.dirname(nvidia.curand.__file__), "lib", "libcurand.so*"))
    except Exception:
        pass
    for p in pats:
        for f in sorted(glob.glob(p)):
            if "stubs" not in f:
                return f
    return None


def _curand_host_philox(seed: int, n_words: int) -> np.ndarray:
    path = _find_curand()
    if path is None:
        pytest.skip("libcurand not found")
    cr = ctypes.CDLL(path)
    gen = ctypes.c_void_p()
    CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
    assert cr.curandCreateGeneratorHost(ctypes.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) == 0
    assert cr.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    out = np.zeros(n_words, dtype=np.uint32)
    assert cr.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n_words)) == 0
    cr.curandDestroyGenerator(gen)
    return out


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF])
def test_philox_matches_library_generator(seed):
    """The library's stream is made of 4-word Philox outputs for key = seed and
    counters (c0, 0, c2, 0); every oracle output for such a counter must occur in
    it as an aligned group (the order in which the library walks the counters is
    its own business)."""
    n_groups = 3 * 65536
    stream = _curand_host_philox(seed, 4 * n_groups).reshape(n_groups, 4)
    index = {tuple(int(x) for x in g): i for i, g in enumerate(stream)}
    assert len(index) == n_groups
    key = [seed & 0xFFFFFFFF, seed >> 32]
    first = tuple(int(x) for x in oracle.philox4x32_10([0, 0, 0, 0], key))
    assert index.get(first) == 0
    found = 0
    for c0 in range(3):
        for c2 in (0, 1, 2, 77, 4095, 65535):
            got = tuple(int(x) for x in oracle.philox4x32_10([c0, 0, c2, 0], key))
            assert got in index, (c0, c2)
            found += 1
    assert found == 18


def test_weyl_constants_are_the_published_irrationals():
    """The key schedule adds floor(2^32 (phi - 1)) and floor(2^32 (sqrt(3) - 1)).  With an all-zero
    counter the first round leaves (0 ^ 0 ^ k0, 0, 0 ^ 0 ^ k1, 0); feeding two keys that differ by
    the Weyl constants must therefore reproduce a 9-round tail -- checked through the public
    10-round function on counters built from that identity."""
    from decimal import Decimal, getcontext
    getcontext().prec = 50
    w0 = int(((Decimal(5).sqrt() + 1) / 2 - 1) * 2 ** 32)
    w1 = int((Decimal(3).sqrt() - 1) * 2 ** 32)
    assert (w0, w1) == (0x9E3779B9, 0xBB67AE85)
    # one Philox round on counter (0,0,0,0) and key (a,b) gives counter (a,0,b,0) and key (a+w0, b+w1):
    # so philox10(ctr=0, key=(a,b)) == philox9 applied to ((a,0,b,0), key (a+w0,b+w1)).
    # Compare two 10-round evaluations that must agree on that 9-round tail after one more round.
    a, b = 0x12345678, 0x9ABCDEF0
    full = oracle.philox4x32_10([0, 0, 0, 0], [a, b])
    # 10 rounds from (a,0,b,0) with the bumped key = the 9-round tail plus one extra round;
    # undo nothing: instead check the extra round explicitly with big-int arithmetic.
    ext = oracle.philox4x32_10([a, 0, b, 0], [(a + w0) & 0xFFFFFFFF, (b + w1) & 0xFFFFFFFF])
    k0 = (a + 10 * w0) & 0xFFFFFFFF
    k1 = (b + 10 * w1) & 0xFFFFFFFF
    p0 = 0xD2511F53 * int(full[0])
    p1 = 0xCD9E8D57 * int(full[2])
    one_more = [(p1 >> 32) ^ int(full[1]) ^ k0, p1 & 0xFFFFFFFF, (p0 >> 32) ^ int(full[3]) ^ k1, p0 & 0xFFFFFFFF]
    assert [int(x) for x in ext] == one_more


def test_philox_counter_bijection_and_avalanche():
    rng = np.random.default_rng(5)
    key = [0xDEADBEEF, 0x0BADF00D]
    outs = set()
    for c in range(4096):
        outs.add(tuple(int(x) for x in oracle.philox4x32_10([c & 15, (c >> 4) & 15, (c >> 8) & 15, 0], key)))
    assert len(outs) == 4096
    flips = []
    for _ in range(400):
        ctr = rng.integers(0, 2 ** 32, 4, dtype=np.uint32)
        k = rng.integers(0, 2 ** 32, 2, dtype=np.uint32)
        base = oracle.philox4x32_10(ctr, k)
        which = int(rng.integers(0, 6))
        bit = np.uint32(1 << int(rng.integers(0, 32)))
        c2, k2 = ctr.copy(), k.copy()
        if which < 4:
            c2[which] ^= bit
        else:
            k2[which - 4] ^= bit
        other = oracle.philox4x32_10(c2, k2)
        flips.append(sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(base, other)))
    mean = float(np.mean(flips))
    assert abs(mean - 64) < 4 * math.sqrt(32) / math.sqrt(len(flips)) * 4  # 128 output bits, half flip


def test_element_word_layout():
    """Element i takes word i mod 4 of counter (i div 4, tensor_id, step lo, step hi), key = seed."""
    seed, step, tid = 0xEC0ABCDEF1234, (7 << 32) | 99, 4242
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for i in (0, 1, 2, 3, 4, 5, 1023, 2 ** 32 + 6, 2 ** 34 - 1):
        blk = oracle.philox4x32_10([(i >> 2) & 0xFFFFFFFF, tid, step & 0xFFFFFFFF, step >> 32], key)
        assert oracle.element_random_word(seed, step, tid, i) == int(blk[i & 3])
    # uniformity of the 24 bits that decide stochastic rounding
    u = np.array([oracle.element_random_word(1, 1, 0, i) >> 8 for i in range(40000)], dtype=np.float64) / 2 ** 24
    assert abs(u.mean() - 0.5) < 5 * math.sqrt(1 / 12 / u.size)
    assert abs((u < 0.1).mean() - 0.1) < 5 * math.sqrt(0.09 / u.size)
