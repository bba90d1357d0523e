"""Pins for the oracle's normal transform and for the seed -> A addressing (CPU only).

The paper fixes the law of A (i.i.d. N(0, 1/r), Algorithm 1) and that A is a function of the
seed alone; these tests check the transform against the textbook Box-Muller formula evaluated
with libm in double precision, and the samples against the normal law."""
import math
import random

import numpy as np
import pytest
from scipy import stats

from oracle import flora_oracle as orc


def _textbook(xa, xb):
    u1, u2 = orc.pair_uniforms(xa, xb)
    rho = math.sqrt(-2.0 * math.log(u1))
    return rho * math.cos(2 * math.pi * u2), rho * math.sin(2 * math.pi * u2)


def _check(xa, xb):
    zc, zs = orc.normal_pair(xa, xb)
    tc, ts = _textbook(xa, xb)
    assert abs(zc - tc) <= 2e-6 * max(1.0, abs(tc)), (hex(xa), hex(xb), zc, tc)
    assert abs(zs - ts) <= 2e-6 * max(1.0, abs(ts)), (hex(xa), hex(xb), zs, ts)


def test_uniform_ranges():
    assert orc.pair_uniforms(0, 0) == (2.0 ** -24, 0.0)
    u1, u2 = orc.pair_uniforms(0xFFFFFFFF, 0xFFFFFFFF)
    assert u1 == 1.0 and u2 == 1.0 - 2.0 ** -24
    # the low 8 bits of each word are unused
    assert orc.pair_uniforms(0x12345600, 0xABCDEF00) == orc.pair_uniforms(0x123456FF, 0xABCDEFFF)


def test_transform_matches_textbook_box_muller_random():
    rnd = random.Random(11)
    for _ in range(150000):
        _check(rnd.getrandbits(32), rnd.getrandbits(32))


def test_transform_matches_textbook_box_muller_edges():
    # u1 at both ends and around every power of two (exponent split), u2 around every octant edge
    k1s = [1, 2, 3, (1 << 24) - 1, 1 << 24]
    for e in range(1, 24):
        k1s += [(1 << e) - 1, 1 << e, (1 << e) + 1, int((1 << e) * 4 / 3), int((1 << e) * 4 / 3) + 1, int((1 << e) * 4 / 3) - 1]
    k2s = [0, 1, (1 << 24) - 1]
    for o in range(1, 8):
        k2s += [(o << 21) - 1, o << 21, (o << 21) + 1, (o << 21) + (1 << 20)]
    for k1 in k1s:
        for k2 in k2s:
            _check(((k1 - 1) << 8) | 0x5A, (k2 << 8) | 0xC3)


def test_largest_and_zero_radius():
    zc, zs = orc.normal_pair(0, 0)              # u1 = 2^-24: the largest radius, angle 0
    assert zc == pytest.approx(math.sqrt(2 * 24 * math.log(2)), rel=1e-6) and zs == 0.0
    zc, zs = orc.normal_pair(0xFFFFFFFF, 0x40000000)   # u1 = 1: radius exactly zero
    assert zc == 0.0 and zs == 0.0


def test_exact_quarter_turns():
    xa = 0x80000000
    rho = orc.normal_pair(xa, 0)[0]
    assert orc.normal_pair(xa, 0x40000000)[1] == pytest.approx(rho, rel=1e-6)     # angle pi/2
    assert orc.normal_pair(xa, 0x80000000)[0] == pytest.approx(-rho, rel=1e-6)    # angle pi
    assert orc.normal_pair(xa, 0xC0000000)[1] == pytest.approx(-rho, rel=1e-6)    # angle 3pi/2
    c, s = orc.normal_pair(xa, 0x20000000)                                         # angle pi/4
    assert c == pytest.approx(s, rel=1e-6) and c > 0


@pytest.fixture(scope="module")
def big_sample():
    return orc.materialize_A(0x1234ABCD5678EF01, 1, 1 << 22)[0].astype(np.float64)   # r = 1: A = z


def test_moments_of_standard_normal(big_sample):
    z = big_sample
    n = z.size
    assert abs(z.mean()) <= 6 / math.sqrt(n)
    assert abs(z.var() - 1) <= 6 * math.sqrt(2 / n)
    assert abs((z ** 3).mean()) <= 6 * math.sqrt(15 / n)
    assert abs((z ** 4).mean() - 3) <= 6 * math.sqrt(96 / n)


def test_kolmogorov_smirnov_against_phi(big_sample):
    z = big_sample[: 1 << 20]
    d = stats.kstest(z, "norm").statistic
    assert d < 1.95 / math.sqrt(z.size)       # 0.1 % critical value of the KS statistic


def test_elements_of_a_pair_and_neighbours_are_uncorrelated(big_sample):
    z = big_sample
    n = z.size // 2
    for a, b in ((z[0::2], z[1::2]), (z[:-1:2], z[1::2] ** 2 - 1), (z[0:-2:2], z[2::2])):
        m = min(a.size, b.size)
        assert abs(np.mean(a[:m] * b[:m])) <= 6 * math.sqrt(2.0 / n)


def test_variance_is_one_over_r():
    for r in (2, 8, 32, 256):
        A = orc.materialize_A(99 + r, r, 65536 // r * 4).astype(np.float64)
        n = A.size
        assert abs(A.var() * r - 1) <= 6 * math.sqrt(2 / n)
        assert abs(A.mean()) * math.sqrt(r) <= 6 / math.sqrt(n)


def test_element_depends_only_on_seed_row_column():
    seed = 0xFEEDFACE12345678
    big = orc.materialize_A(seed, 16, 203)
    # a prefix in the columns (including a count that is not a multiple of 4) and in the rows
    assert np.array_equal(orc.materialize_A(seed, 16, 77), big[:, :77])
    z1 = orc.materialize_A(seed, 1, 203)                      # scale 1: the standard normals of row 0
    z4 = orc.materialize_A(seed, 4, 203)                      # scale 1/2 exactly
    assert np.array_equal(z4[0], z1[0] * np.float32(0.5))
    s16 = np.float32(1.0) / np.sqrt(np.float32(16))
    assert np.array_equal(big[:4], orc.materialize_A(seed, 4, 203) * np.float32(2.0) * s16)
    assert not np.array_equal(orc.materialize_A(seed + 1, 16, 203), big)
    assert not np.array_equal(orc.materialize_A(seed ^ (1 << 40), 16, 203), big)
    assert not np.array_equal(big[0], big[1])


def test_element_layout_against_the_block_function():
    # column 4q+t of row j comes from Philox block (q, j, 0, 0): words (0,1) -> t = 0 (cos), 1 (sin);
    # words (2,3) -> t = 2, 3; key = (low, high) half of the seed
    seed = 0x0123456789ABCDEF
    r, m = 3, 10
    A = orc.materialize_A(seed, r, m)
    scale = np.float32(1.0) / np.sqrt(np.float32(r))
    for j in range(r):
        for q in range(3):
            x = orc.philox4x32_10([q, j, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
            z = orc.normal_pair(int(x[0]), int(x[1])) + orc.normal_pair(int(x[2]), int(x[3]))
            for t in range(4):
                if 4 * q + t < m:
                    assert A[j, 4 * q + t] == np.float32(z[t]) * scale


def test_bf16_rounding_is_nearest_even_against_torch():
    import torch
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(200000).astype(np.float32),
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 1.0, 3.3895314e38 / 2], dtype=np.float32)])
    vals, bits = orc.round_to_bf16(x)
    t = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits, t.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(vals, t.to(torch.float32).numpy())
    assert np.array_equal(orc.bf16_bits_to_f32(bits), vals)


def test_double_to_bf16_rounds_once():
    from fractions import Fraction
    rnd = random.Random(8)

    def exact(v):
        # nearest bf16 (8 significant bits) to the rational v, ties to even, by exact arithmetic
        if v == 0:
            return 0.0
        s = -1 if v < 0 else 1
        a = Fraction(abs(v))
        e = math.floor(math.log2(a))
        while Fraction(2) ** e > a:
            e -= 1
        while Fraction(2) ** (e + 1) <= a:
            e += 1
        ulp = Fraction(2) ** (e - 7)
        k = a / ulp
        lo = math.floor(k)
        frac = k - lo
        if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1):
            lo += 1
        return s * float(lo * ulp)

    cases = [1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 - 2.0 ** -40,
             -(1.0 + 2.0 ** -8 + 2.0 ** -30), 0.0, 1.0, -2.5]
    cases += [rnd.gauss(0, 1) * 10 ** rnd.uniform(-6, 6) for _ in range(20000)]
    # double values that sit just beside a float32 rounding boundary and a bf16 tie at once
    cases += [float(np.float32(1.0 + k * 2.0 ** -8)) + d for k in range(1, 40, 2) for d in (2.0 ** -26, -2.0 ** -26, 2.0 ** -50)]
    for v in cases:
        got = float(orc.bf16_bits_to_f32(np.array([orc.double_to_bf16_bits(v)], dtype=np.uint16))[0])
        assert got == exact(v), v
