"""Pins for the oracle's contractions (CPU only): brute force written from Algorithms 1 and 2,
float64 library matmul on the explicit A, and the identities the paper states (linearity of
Eq. (rp), E[A^T A] = I behind Theorem 2.4, row-norm preservation of Lemma 2.3, the momentum
recursion and the transfer M A A'^T of Algorithm 2)."""
import math

import numpy as np
import pytest

from oracle import flora_oracle as orc


def _rng(seed):
    return np.random.default_rng(seed)


def _bf16(x):
    return orc.round_to_bf16(x)          # (values, bits)


# ----------------------------------------------------------------------------- brute force
def test_compress_then_decompress_brute_force_python_loops():
    n, m, r = 5, 11, 3
    rng = _rng(0)
    G = rng.standard_normal((n, m)).astype(np.float32)
    W = rng.standard_normal((n, m)).astype(np.float32)
    A = orc.materialize_A(17, r, m)
    C = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate(G, A, C)
    Cb = [[sum(float(G[i, k]) * float(A[j, k]) for k in range(m)) for j in range(r)] for i in range(n)]
    for i in range(n):
        for j in range(r):
            assert C[i, j] == np.float32(Cb[i][j])
    lr, scale = 0.37, 0.25
    W2 = W.copy()
    orc.decompress_apply(W2, C, A, lr, scale)
    step = float(np.float32(lr)) * float(np.float32(scale))
    for i in range(n):
        for k in range(m):
            upd = sum(float(C[i, j]) * float(A[j, k]) for j in range(r))
            assert W2[i, k] == np.float32(float(W[i, k]) - step * upd)


def test_second_accumulation_adds_to_the_first():
    n, m, r = 4, 9, 2
    rng = _rng(1)
    G1 = rng.standard_normal((n, m)).astype(np.float32)
    G2 = rng.standard_normal((n, m)).astype(np.float32)
    A = orc.materialize_A(5, r, m)
    C = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate(G1, A, C)
    C1 = C.copy()
    orc.compress_accumulate(G2, A, C)
    for i in range(n):
        for j in range(r):
            inc = sum(float(G2[i, k]) * float(A[j, k]) for k in range(m))
            assert C[i, j] == np.float32(float(C1[i, j]) + inc)


# ----------------------------------------------------------------------------- library matmul
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_against_float64_matmul(dtype):
    n, m, r = 37, 130, 8
    rng = _rng(2)
    G = rng.standard_normal((n, m)).astype(np.float32)
    W = rng.standard_normal((n, m)).astype(np.float32)
    A = orc.projection(21, r, m, dtype)
    if dtype == "bf16":
        Gv, Gs = _bf16(G)
        Wv, Ws = _bf16(W)
    else:
        Gv, Gs, Wv, Ws = G, G, W, W.copy()
    C = rng.standard_normal((n, r)).astype(np.float32)
    C0 = C.copy()
    orc.compress_accumulate(Gs, A, C)
    ref = C0.astype(np.float64) + Gv.astype(np.float64) @ A.astype(np.float64).T
    assert np.allclose(C, ref, rtol=1e-6, atol=1e-6)
    assert np.max(np.abs(C - ref.astype(np.float32))) <= np.spacing(np.abs(ref).max().astype(np.float32))
    Wt = Ws.copy()
    orc.decompress_apply(Wt, C, A, 0.5, 0.125)
    refw = Wv.astype(np.float64) - 0.0625 * (C.astype(np.float64) @ A.astype(np.float64))
    got = orc.bf16_bits_to_f32(Wt) if dtype == "bf16" else Wt
    tol = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -23
    assert np.all(np.abs(got - refw) <= tol * np.abs(refw) + 1e-30)


def test_leading_dimensions_are_respected():
    n, m, r = 6, 10, 4
    rng = _rng(3)
    Gbig = rng.standard_normal((n, m + 7)).astype(np.float32)
    Cbig = np.zeros((n, r + 3), dtype=np.float32)
    A = orc.materialize_A(1, r, m)
    orc.compress_accumulate(Gbig[:, :m], A, Cbig[:, :r])
    C = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate(np.ascontiguousarray(Gbig[:, :m]), A, C)
    assert np.array_equal(Cbig[:, :r], C) and np.all(Cbig[:, r:] == 0)


# ----------------------------------------------------------------------------- Eq. (rp): linearity
def test_compression_is_linear_in_the_gradient():
    n, m, r = 16, 64, 8
    rng = _rng(4)
    G1 = rng.standard_normal((n, m)).astype(np.float32)
    G2 = rng.standard_normal((n, m)).astype(np.float32)
    A = orc.materialize_A(77, r, m)
    alpha = 0.75                                             # exact in binary
    Cs = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate((alpha * G1 + G2).astype(np.float32), A, Cs)
    C1 = np.zeros((n, r), dtype=np.float32)
    C2 = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate(G1, A, C1)
    orc.compress_accumulate(G2, A, C2)
    assert np.allclose(Cs, alpha * C1 + C2, rtol=0, atol=2e-5)


def test_tau_step_accumulation_equals_compression_of_the_sum():
    n, m, r, tau = 8, 48, 4, 6
    rng = _rng(5)
    Gs = [np.round(rng.standard_normal((n, m)) * 64).astype(np.float32) / 64 for _ in range(tau)]
    A = orc.materialize_A(3, r, m)
    C = np.zeros((n, r), dtype=np.float32)
    for G in Gs:
        orc.compress_accumulate(G, A, C)
    Csum = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate(sum(Gs).astype(np.float32), A, Csum)       # the sum is exact in fp32
    assert np.allclose(C, Csum, rtol=0, atol=1e-4)
    # and the decompressed mean uses scale = 1/tau
    W1 = np.zeros((n, m), dtype=np.float32)
    orc.decompress_apply(W1, C, A, 1.0, 1.0 / tau)
    ref = -(C.astype(np.float64) @ A.astype(np.float64)) * float(np.float32(1.0 / tau))
    assert np.allclose(W1, ref, rtol=1e-6, atol=1e-6)


# ----------------------------------------------------------------------------- Theorem 2.4 / Lemma 2.3
def test_expectation_of_AtA_is_identity():
    m, r, S = 16, 8, 4096
    acc = np.zeros((m, m))
    for s in range(S):
        A = orc.materialize_A(1000 + s, r, m).astype(np.float64)
        acc += A.T @ A
    acc /= S
    diag = np.diag(acc)
    off = acc - np.diag(diag)
    assert np.max(np.abs(diag - 1)) <= 6 * math.sqrt(2 / (r * S))
    assert np.max(np.abs(off)) <= 6 * math.sqrt(1 / (r * S))


def test_decompressed_compression_is_unbiased():
    n, m, r, S = 3, 24, 4, 6000
    rng = _rng(6)
    G = rng.standard_normal((n, m)).astype(np.float32)
    mean = np.zeros((n, m))
    for s in range(S):
        A = orc.materialize_A(50000 + s, r, m)
        C = np.zeros((n, r), dtype=np.float32)
        orc.compress_accumulate(G, A, C)
        W = np.zeros((n, m), dtype=np.float32)
        orc.decompress_apply(W, C, A, -1.0, 1.0)              # W = + C A
        mean += W
    mean /= S
    var = ((G.astype(np.float64) ** 2).sum(axis=1, keepdims=True) + G.astype(np.float64) ** 2) / r
    assert np.all(np.abs(mean - G) <= 6 * np.sqrt(var / S))


def test_theorem_2_4_entrywise_bound_single_draw():
    delta = 1e-3
    for r, m in ((64, 128), (256, 64), (8, 32)):
        A = orc.materialize_A(4242 + r, r, m).astype(np.float64)
        t = math.log(2 * m / delta)
        bound = 4 * math.sqrt(2 * t / r) + 8 * t / r
        assert np.max(np.abs(A.T @ A - np.eye(m))) <= bound


def test_row_norms_are_preserved_in_expectation():
    n, m, r, S = 4, 40, 8, 3000
    rng = _rng(7)
    G = rng.standard_normal((n, m)).astype(np.float32)
    ratios = np.zeros((S, n))
    for s in range(S):
        A = orc.materialize_A(9000 + s, r, m)
        C = np.zeros((n, r), dtype=np.float32)
        orc.compress_accumulate(G, A, C)
        ratios[s] = (C.astype(np.float64) ** 2).sum(axis=1) / (G.astype(np.float64) ** 2).sum(axis=1)
    # each ratio is chi^2_r / r: mean 1, variance 2/r
    assert np.all(np.abs(ratios.mean(axis=0) - 1) <= 6 * math.sqrt(2 / r / S))
    assert np.all(np.abs(ratios.var(axis=0) - 2 / r) <= 6 * math.sqrt((8 / r ** 2 + 48 / r ** 3) / S) + 0.01)


# ----------------------------------------------------------------------------- Algorithm 2: momentum
def test_momentum_special_cases_and_closed_form():
    n, m, r = 7, 33, 5
    rng = _rng(8)
    A = orc.materialize_A(31337, r, m)
    G = rng.standard_normal((n, m)).astype(np.float32)
    M0 = rng.standard_normal((n, r)).astype(np.float32)
    M = M0.copy()
    orc.momentum_step(G, A, 0.0, M)                            # beta = 0: plain compression
    C = np.zeros((n, r), dtype=np.float32)
    orc.compress_accumulate(G, A, C)
    assert np.array_equal(M, C)
    M = M0.copy()
    orc.momentum_step(G, A, 1.0, M)                            # beta = 1: state untouched
    assert np.array_equal(M, M0)
    beta, T = 0.875, 5
    Gs = [rng.standard_normal((n, m)).astype(np.float32) for _ in range(T)]
    M = np.zeros((n, r), dtype=np.float32)
    for G in Gs:
        orc.momentum_step(G, A, beta, M)
    closed = sum((1 - beta) * beta ** (T - 1 - t) * (Gs[t].astype(np.float64) @ A.astype(np.float64).T) for t in range(T))
    assert np.allclose(M, closed, rtol=0, atol=1e-5)


def test_momentum_brute_force():
    n, m, r = 3, 7, 2
    rng = _rng(9)
    A = orc.materialize_A(2, r, m)
    G = rng.standard_normal((n, m)).astype(np.float32)
    M0 = rng.standard_normal((n, r)).astype(np.float32)
    M = M0.copy()
    beta = 0.9
    orc.momentum_step(G, A, beta, M)
    b = float(np.float32(beta))
    for i in range(n):
        for j in range(r):
            acc = sum(float(G[i, k]) * float(A[j, k]) for k in range(m))
            assert M[i, j] == np.float32(b * float(M0[i, j]) + (1.0 - b) * acc)


# ----------------------------------------------------------------------------- Algorithm 2: transfer
def test_transfer_brute_force_in_printed_order():
    n, m, r = 4, 13, 3
    rng = _rng(10)
    M0 = rng.standard_normal((n, r)).astype(np.float32)
    Ao = orc.materialize_A(100, r, m)
    An = orc.materialize_A(101, r, m)
    M = M0.copy()
    orc.resample_transfer(M, Ao, An)
    for i in range(n):
        P = [sum(float(M0[i, j]) * float(Ao[j, k]) for j in range(r)) for k in range(m)]
        for j in range(r):
            assert M[i, j] == np.float32(sum(P[k] * float(An[j, k]) for k in range(m)))
    ref = (M0.astype(np.float64) @ Ao.astype(np.float64)) @ An.astype(np.float64).T
    assert np.allclose(M, ref, rtol=1e-6, atol=1e-6)


def test_transferred_momentum_decompresses_to_the_old_one_in_expectation():
    n, m, r, S = 2, 12, 4, 6000
    rng = _rng(11)
    M0 = rng.standard_normal((n, r)).astype(np.float32)
    Ao = orc.materialize_A(7, r, m)
    target = M0.astype(np.float64) @ Ao.astype(np.float64)          # M A_old, n x m
    mean = np.zeros((n, m))
    for s in range(S):
        An = orc.materialize_A(70000 + s, r, m)
        M = M0.copy()
        orc.resample_transfer(M, Ao, An)
        mean += M.astype(np.float64) @ An.astype(np.float64)
    mean /= S
    var = ((target ** 2).sum(axis=1, keepdims=True) + target ** 2) / r
    assert np.all(np.abs(mean - target) <= 6 * np.sqrt(var / S))


def test_same_seed_transfer_scales_by_m_over_r_on_average():
    m, r = 4096, 4
    A = orc.materialize_A(5, r, m)
    M = np.eye(r, dtype=np.float32)
    orc.resample_transfer(M, A, A)                                  # = A A^T
    assert np.allclose(np.diag(M), m / r, rtol=6 * math.sqrt(2 / m))
    assert np.max(np.abs(M - np.diag(np.diag(M)))) <= 6 * math.sqrt(m) / r


def test_transfer_axpby_composes_accumulation_with_momentum():
    # Algorithm 1 returns G~ = (1/tau) C A_acc; Algorithm 2 consumes it: M <- beta M + (1-beta) G~ A_mom^T
    n, m, r, tau, beta = 5, 21, 3, 4, 0.75
    rng = _rng(12)
    C = rng.standard_normal((n, r)).astype(np.float32)
    M0 = rng.standard_normal((n, r)).astype(np.float32)
    Aacc = orc.materialize_A(1, r, m)
    Amom = orc.materialize_A(2, r, m)
    M = M0.copy()
    orc.transfer_axpby(M, C, Aacc, Amom, (1 - beta) / tau, beta)
    Gt = np.zeros((n, m), dtype=np.float64) + (C.astype(np.float64) @ Aacc.astype(np.float64)) / tau
    ref = beta * M0.astype(np.float64) + (1 - beta) * (Gt @ Amom.astype(np.float64).T)
    assert np.allclose(M, ref, rtol=1e-6, atol=1e-6)


# ----------------------------------------------------------------------------- apply
def test_apply_with_zero_lr_is_identity_and_is_linear_in_the_step():
    n, m, r = 9, 20, 4
    rng = _rng(13)
    A = orc.projection(8, r, m, "bf16")
    C = rng.standard_normal((n, r)).astype(np.float32)
    Wv, Wb = _bf16(rng.standard_normal((n, m)).astype(np.float32))
    W = Wb.copy()
    orc.decompress_apply(W, C, A, 0.0, 1.0)
    assert np.array_equal(W, Wb)
    Z1 = np.zeros((n, m), dtype=np.float32)
    Z2 = np.zeros((n, m), dtype=np.float32)
    orc.decompress_apply(Z1, C, A, 0.5, 0.5)
    orc.decompress_apply(Z2, C, A, 1.0, 1.0)
    assert np.allclose(4 * Z1, Z2, rtol=1e-6, atol=1e-7)


def test_state_is_a_fraction_r_over_m_of_the_matrix():
    # Section 2.4: O(nm) -> O(nr); the paper's GPT-3 example: r = 256 of d_model 12288 is 2.08 %
    assert round(100 * 256 / 12288, 2) == 2.08
    from paper_2402_03293_b200 import workloads as wl
    w = wl.WORKLOADS["gpt2_small_set"]
    state = sum(n * w.r for n, _ in w.shapes)
    assert state * 4 == 8257536 and w.elements == 84934656


def test_resampled_momentum_step_is_the_closed_form_of_algorithm_2():
    """beta (M A_old A_new^T) + (1 - beta) G A_new^T with materialised projections, in float64."""
    n, m, r, beta = 5, 21, 4, 0.8
    rng = _rng(12)
    G = rng.standard_normal((n, m)).astype(np.float32)
    M0 = rng.standard_normal((n, r)).astype(np.float32)
    Ao, An = orc.materialize_A(300, r, m), orc.materialize_A(301, r, m)
    M = M0.copy()
    orc.momentum_step_resampled(G, Ao, An, beta, M)
    g, m0, ao, an = (x.astype(np.float64) for x in (G, M0, Ao, An))
    ref = beta * (m0 @ ao @ an.T) + (1.0 - beta) * (g @ an.T)
    assert np.allclose(M, ref, rtol=2e-6, atol=2e-6)
    # the two special cases: beta = 1 is the transfer alone, beta = 0 forgets the old state altogether
    M = M0.copy()
    orc.momentum_step_resampled(G, Ao, An, 1.0, M)
    T = M0.copy()
    orc.resample_transfer(T, Ao, An)
    assert np.array_equal(M, T)
    M = M0.copy()
    orc.momentum_step_resampled(G, Ao, An, 0.0, M)
    C = np.zeros_like(M0)
    orc.compress_accumulate(G, An, C)
    assert np.array_equal(M, C)
