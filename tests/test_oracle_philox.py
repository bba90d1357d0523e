"""Pins for the oracle's Philox4x32-10 core (CPU only).

Three things other than the oracle itself fix it: a second implementation in
Python big integers written from the published round function, the inverse
cipher (each round is a bijection given the key), and the cuRAND *host*
generator CURAND_RNG_PSEUDO_PHILOX4_32_10, a library routine that runs on the
CPU.  Plus bit-frequency statistics.
"""
import ctypes
import ctypes.util
import os
import random

import numpy as np
import pytest

from oracle import flora_oracle as orc

M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def philox_bigint(ctr, key):
    c = list(ctr)
    k0, k1 = key
    for _ in range(10):
        p0 = M0 * c[0]
        p1 = M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k0, p1 & MASK, (p0 >> 32) ^ c[3] ^ k1, p0 & MASK]
        k0 = (k0 + W0) & MASK
        k1 = (k1 + W1) & MASK
    return c


def philox_inverse(out, key):
    inv0 = pow(M0, -1, 1 << 32)
    inv1 = pow(M1, -1, 1 << 32)
    keys = [((key[0] + i * W0) & MASK, (key[1] + i * W1) & MASK) for i in range(10)]
    n = list(out)
    for k0, k1 in reversed(keys):
        c2 = (n[1] * inv1) & MASK
        c0 = (n[3] * inv0) & MASK
        c1 = n[0] ^ ((M1 * c2) >> 32) ^ k0
        c3 = n[2] ^ ((M0 * c0) >> 32) ^ k1
        n = [c0, c1, c2, c3]
    return n


def _rand_inputs(count, seed):
    rnd = random.Random(seed)
    edge = [0, 1, MASK, 0x80000000, 0x7FFFFFFF]
    for i in range(count):
        if i < 25:
            yield [edge[i % 5], edge[(i // 5) % 5], edge[(i * 3) % 5], edge[(i * 7) % 5]], [edge[(i + 1) % 5], edge[(i + 2) % 5]]
        else:
            yield [rnd.getrandbits(32) for _ in range(4)], [rnd.getrandbits(32) for _ in range(2)]


def test_matches_independent_bigint_implementation():
    for ctr, key in _rand_inputs(20000, 1):
        assert list(map(int, orc.philox4x32_10(ctr, key))) == philox_bigint(ctr, key)


def test_cipher_is_invertible():
    for ctr, key in _rand_inputs(3000, 2):
        out = list(map(int, orc.philox4x32_10(ctr, key)))
        assert philox_inverse(out, key) == ctr


def _curand_host():
    for name in ("libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so.10", ctypes.util.find_library("curand")):
        if not name:
            continue
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


def test_matches_curand_host_generator():
    """cuRAND's Philox4_32_10 *host* generator (runs on the CPU): the key is the 64-bit seed and
    output block i (four words, found by probing the public API) is the Philox block with
    counter (i >> 16, 0, i & 0xFFFF, 0)."""
    lib = _curand_host()
    if lib is None:
        pytest.skip("libcurand not present")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:
        pytest.skip("cuRAND host generator unavailable")
    rnd = random.Random(3)
    try:
        for i in range(400):
            seed = rnd.getrandbits(64) if i else 0
            block = rnd.getrandbits(rnd.choice([4, 17, 30, 47])) if i else 0
            assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
            assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(4 * block)) == 0
            out = np.zeros(4, dtype=np.uint32)
            assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(4)) == 0
            mine = orc.philox4x32_10([block >> 16, 0, block & 0xFFFF, 0], [seed & MASK, seed >> 32])
            assert list(map(int, out)) == list(map(int, mine)), (seed, block)
    finally:
        lib.curandDestroyGenerator(gen)


def test_bit_and_byte_frequencies():
    # 2^16 blocks = 2^18 words: every bit position within 5 sigma of 1/2, byte histogram chi-square sane
    words = []
    for q in range(1 << 14):
        words.extend(int(x) for x in orc.philox4x32_10([q, 5, 0, 0], [0xDEADBEEF, 0x12345678]))
    w = np.array(words, dtype=np.uint32)
    n = w.size
    for bit in range(32):
        ones = int(((w >> bit) & 1).sum())
        assert abs(ones - n / 2) < 5 * (n ** 0.5) / 2
    hist = np.bincount(w.view(np.uint8), minlength=256).astype(np.float64)
    expected = 4 * n / 256
    chi2 = ((hist - expected) ** 2 / expected).sum()
    assert abs(chi2 - 255) < 6 * (2 * 255) ** 0.5


def test_counter_and_key_words_all_matter():
    base = list(map(int, orc.philox4x32_10([1, 2, 3, 4], [5, 6])))
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] ^= 1
        assert list(map(int, orc.philox4x32_10(c, [5, 6]))) != base
    assert list(map(int, orc.philox4x32_10([1, 2, 3, 4], [4, 6]))) != base
    assert list(map(int, orc.philox4x32_10([1, 2, 3, 4], [5, 7]))) != base
