"""Pins for the oracle's Philox4x32-10 and its keying (no GPU needed)."""
import ctypes
import ctypes.util
import math
import os

import numpy as np
import pytest

import oracle

M32 = 0xFFFFFFFF


def _weyl_constants():
    # closed forms given with the generator's definition: floor(2^32 / golden ratio) and
    # floor(2^32 (sqrt(3) - 1)), in exact integer arithmetic
    s5 = math.isqrt(5 << 128)            # sqrt(5) * 2^64
    golden = ((s5 - (1 << 64)) << 31) >> 64   # (sqrt5 - 1)/2 * 2^32
    s3 = math.isqrt(3 << 128)
    w1 = ((s3 - (1 << 64)) << 32) >> 64
    return golden, w1


def _philox_bigint(ctr, key):
    """Restatement with Python integers; Weyl constants from their closed forms."""
    w0, w1 = _weyl_constants()
    c = [int(x) for x in ctr]
    k = [int(x) for x in key]
    for r in range(10):
        if r:
            k = [(k[0] + w0) & M32, (k[1] + w1) & M32]
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & M32, (p0 >> 32) ^ c[3] ^ k[1], p0 & M32]
    return c


def test_weyl_constants_closed_form():
    assert _weyl_constants() == (0x9E3779B9, 0xBB67AE85)


def test_philox_matches_bigint_restatement_on_random_inputs():
    rng = np.random.default_rng(1234)
    for _ in range(3000):
        ctr = rng.integers(0, 1 << 32, 4, dtype=np.uint64)
        key = rng.integers(0, 1 << 32, 2, dtype=np.uint64)
        assert oracle.philox4x32_10(ctr, key) == _philox_bigint(ctr, key)
    # edge words
    for ctr in ([0, 0, 0, 0], [M32] * 4, [1, 0, 0, 0], [0, 0, 0, 1]):
        for key in ([0, 0], [M32, M32]):
            assert oracle.philox4x32_10(ctr, key) == _philox_bigint(ctr, key)


def _curand():
    for name in ("libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so.10", ctypes.util.find_library("curand")):
        if not name:
            continue
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF, 0xDEADBEEF00000000])
def test_philox_matches_curand_host_generator(seed):
    """cuRAND's HOST Philox4_32_10 generator (a CPU routine of the CUDA toolkit, no GPU
    involved) emits, as its g-th group of four 32-bit outputs, the Philox block of
    counter (g >> 16, 0, g & 0xFFFF, 0) under key (seed_lo, seed_hi).  That fixes the
    round function, both multipliers, both Weyl constants, the key schedule and the
    order of the output words independently of this repository."""
    cu = _curand()
    if cu is None:
        pytest.skip("libcurand not found")
    gen = ctypes.c_void_p()
    assert cu.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0   # CURAND_RNG_PSEUDO_PHILOX4_32_10
    try:
        assert cu.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        n_groups = 3 * 65536 + 17
        out = (ctypes.c_uint32 * (4 * n_groups))()
        assert cu.curandGenerate(gen, out, ctypes.c_size_t(4 * n_groups)) == 0
        got = np.frombuffer(out, dtype=np.uint32).reshape(n_groups, 4)
    finally:
        cu.curandDestroyGenerator(gen)
    key = [seed & M32, seed >> 32]
    rng = np.random.default_rng(seed & 0xFFFF)
    groups = np.concatenate([np.arange(64), rng.integers(0, n_groups, 1500), [65535, 65536, 65537, n_groups - 1]])
    for g in groups:
        g = int(g)
        assert oracle.philox4x32_10([g >> 16, 0, g & 0xFFFF, 0], key) == [int(x) for x in got[g]], g


def test_philox_is_a_bijection_on_counters():
    key = [0xCAFEF00D, 0x12345678]
    seen = set()
    for g in range(1 << 15):
        for ctr in ([g, 0, 0, 0], [0, g, 0, 0], [0, 0, g, 0], [0, 0, 0, g]):
            if g == 0 and ctr != [0, 0, 0, 0] and tuple(ctr) == (0, 0, 0, 0):
                continue
            seen.add(tuple(oracle.philox4x32_10(ctr, key)))
    assert len(seen) == 4 * (1 << 15) - 3      # counter 0 appears four times


def test_philox_bits_look_uniform():
    words = np.array([oracle.philox4x32_10([i, 7, 0, 0], [42, 0]) for i in range(1 << 14)], dtype=np.uint32)
    bits = np.unpackbits(words.view(np.uint8))
    n = bits.size
    assert abs(bits.sum() - n / 2) < 5 * math.sqrt(n / 4)
    counts = np.bincount(words.view(np.uint8).ravel(), minlength=256)
    exp = counts.sum() / 256
    chi2 = ((counts - exp) ** 2 / exp).sum()
    assert chi2 < 255 + 5 * math.sqrt(2 * 255)


def test_keying_of_mask_and_permutation_streams():
    seed, step, t = 0x1122334455667788, (5 << 32) | 99, 17
    key = [seed & M32, seed >> 32]
    for i in (0, 1, 2, 3, 4, 5, 1023, (1 << 32) - 1):
        blk = oracle.philox4x32_10([i >> 2, t, step & M32, ((step >> 32) << 8) | 0], key)
        assert oracle.mask_word(seed, step, t, i) == blk[i & 3]
        for m in range(0, 11):
            blk = oracle.philox4x32_10([i, t, step & M32, ((step >> 32) << 8) | (1 + (m >> 2))], key)
            assert oracle.perm_word(seed, step, t, i, m) == blk[m & 3]
    # the two streams never share a counter: the low byte of counter word 3 is 0 for the
    # mask and >= 1 for permutations
    assert oracle.mask_word(seed, step, t, 0) != oracle.perm_word(seed, step, t, 0, 0)


def test_threshold_rule():
    assert oracle.threshold(0.0) == 0
    assert oracle.threshold(1.0) == 1 << 32
    assert oracle.threshold(0.5) == 1 << 31
    assert oracle.threshold(0.001) == math.floor(0.001 * 2 ** 32)
    assert oracle.threshold(2.0 ** -33) == 0
