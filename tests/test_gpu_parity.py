"""GPU parity: every operation of the C ABI against the CPU oracle on the same stored inputs.

Bit-exact for the generated projection; max |x-ref| / max |ref| <= 1e-5 (fp32) or 2e-2 (bf16
inputs, fp32 accumulation) for the contractions."""
import numpy as np
import pytest
import torch

from oracle import flora_oracle as orc
from paper_2402_03293_b200 import binding as fb
from paper_2402_03293_b200 import workloads as wl
from tests.parity_util import (TOL, oracle_compress, oracle_decompress, oracle_transfer, rel_err, sample_rows, values)

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(autouse=True)
def _auto_path():
    fb.flora_debug_force_path(0)
    yield
    fb.flora_debug_force_path(0)
    torch.cuda.synchronize()
    assert fb.flora_device_status() == 0


def _g(n, m, dtype, seed, var=1e-2):
    return wl.gaussian_matrix(n, m, var, dtype, seed).to(DEV)


# --------------------------------------------------------------------------------------- generator
@pytest.mark.parametrize("seed,r,m", [(42, 8, 512), (0, 1, 1), (2 ** 64 - 1, 3, 7), (0x123456789ABCDEF0, 32, 770),
                                      (7, 256, 1030), (99, 64, 4097)])
def test_generated_projection_is_bit_exact(seed, r, m):
    ref = orc.materialize_A(seed, r, m)
    out = torch.full((r, m + 5), 7.0, device=DEV, dtype=torch.float32)
    fb.flora_materialize_A(out[:, :m], seed)
    got = out.cpu().numpy()
    assert np.array_equal(got[:, :m].view(np.uint32), ref.view(np.uint32))
    assert np.all(got[:, m:] == 7.0)
    outb = torch.zeros((r, m), device=DEV, dtype=torch.bfloat16)
    fb.flora_materialize_A(outb, seed)
    assert np.array_equal(wl.as_numpy(outb), orc.round_to_bf16(ref)[1])


# --------------------------------------------------------------------------------------- contractions
SHAPES = [(1, 1, 1), (5, 7, 3), (33, 100, 8), (130, 257, 17), (64, 512, 32), (300, 1000, 64), (129, 200, 256),
          # eligible for the tensor-core kernels (bf16, 16-byte aligned rows, n >= 128, m >= 64), ragged tiles and tails
          (128, 64, 16), (256, 1024, 32), (1000, 2056, 8), (384, 4104, 32), (515, 1288, 128), (200, 776, 96),
          (700, 1600, 256), (1030, 520, 1), (2100, 1088, 256), (1600, 1600, 200)]


@pytest.mark.parametrize("force_simt", [0, 1])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,m,r", SHAPES)
def test_compress_and_momentum(n, m, r, dtype, force_simt):
    fb.flora_debug_force_path(force_simt)
    G = _g(n, m, dtype, 1)
    S0 = torch.randn(n, r, device=DEV)
    C = S0.clone()
    fb.flora_compress_accumulate(G, C, 1234, r)
    assert rel_err(C.cpu().numpy(), oracle_compress(G, S0, 1234)) <= TOL[dtype]
    M = S0.clone()
    fb.flora_momentum_step(G, M, 0.9, 77)
    assert rel_err(M.cpu().numpy(), oracle_compress(G, S0, 77, a=1.0 - float(np.float32(0.9)), b=0.9)) <= TOL[dtype]
    # beta = 1 leaves the state alone; beta = 0 ignores what was there (even NaN)
    M = S0.clone()
    fb.flora_momentum_step(G, M, 1.0, 77)
    assert rel_err(M.cpu().numpy(), S0.cpu().numpy()) <= 1e-6
    M = torch.full((n, r), float("nan"), device=DEV)
    fb.flora_momentum_step(G, M, 0.0, 77)
    assert rel_err(M.cpu().numpy(), oracle_compress(G, torch.zeros(n, r), 77)) <= TOL[dtype]


@pytest.mark.parametrize("force_simt", [0, 1])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,m,r", SHAPES)
def test_decompress_apply(n, m, r, dtype, force_simt):
    fb.flora_debug_force_path(force_simt)
    W0 = _g(n, m, dtype, 2, var=4e-4)
    C = torch.randn(n, r, device=DEV)
    W = W0.clone()
    lr, scale = 0.5, 0.25                       # the update is as large as W: rounding of W does not hide it
    fb.flora_decompress_apply(W, C, 555, lr, scale)
    ref = oracle_decompress(W0, C, 555, lr, scale)
    assert rel_err(values(wl.as_numpy(W)), values(ref)) <= TOL[dtype]
    w0 = values(wl.as_numpy(W0)).astype(np.float64)
    assert rel_err(values(wl.as_numpy(W)) - w0, values(ref) - w0) <= TOL[dtype]
    W = W0.clone()
    fb.flora_decompress_apply(W, C, 555, 0.0, 1.0)          # lr = 0: bit-identical weights
    assert torch.equal(W, W0)


@pytest.mark.parametrize("operand", ["f32", "bf16"])
@pytest.mark.parametrize("n,m,r", [(1, 1, 1), (9, 33, 4), (100, 515, 32), (257, 1024, 64), (40, 300, 256), (300, 11008, 200),
                                   (64, 4097, 130), (1000, 64, 8), (33, 70, 17), (64, 20000, 64), (40, 40010, 16)])
def test_transfer(n, m, r, operand):
    M0 = torch.randn(n, r, device=DEV)
    M = M0.clone()
    fb.flora_resample_transfer(M, m, operand, 10, 11)
    assert rel_err(M.cpu().numpy(), oracle_transfer(M0, M0, m, operand, 10, 11, 1.0, 0.0)) <= TOL[operand]
    src = torch.randn(n, r, device=DEV)
    dst = M0.clone()
    fb.flora_transfer_axpby(dst, src, m, operand, 3, 4, 0.0125, 0.9)
    assert rel_err(dst.cpu().numpy(), oracle_transfer(M0, src, m, operand, 3, 4, 0.0125, 0.9)) <= TOL[operand]


@pytest.mark.parametrize("n,m,r", [(70, 200, 16), (300, 1000, 20), (384, 2048, 200)])     # SIMT path; tensor-core paths with ragged tiles
def test_strided_views_are_honoured(n, m, r):
    Gbig = _g(n, m + 24, "bf16", 3)
    Cbig = torch.zeros(n, r + 8, device=DEV)
    fb.flora_compress_accumulate(Gbig[:, :m], Cbig[:, :r], 9, r)
    ref = oracle_compress(Gbig[:, :m].contiguous(), torch.zeros(n, r), 9)
    assert rel_err(Cbig[:, :r].cpu().numpy(), ref) <= TOL["bf16"]
    assert torch.all(Cbig[:, r:] == 0)
    Wbig = _g(n, m + 24, "bf16", 4)
    W0 = Wbig.clone()
    fb.flora_decompress_apply(Wbig[:, :m], Cbig[:, :r], 9, 1.0, 1.0)
    refw = oracle_decompress(W0[:, :m].contiguous(), Cbig[:, :r].contiguous(), 9, 1.0, 1.0)
    assert rel_err(values(wl.as_numpy(Wbig[:, :m].contiguous())), values(refw)) <= TOL["bf16"]
    assert torch.equal(Wbig[:, m:], W0[:, m:])
    # momentum (read-modify-write of the strided sketch) and the transfer leave the columns beside the view alone
    Mbig = torch.randn(n, r + 8, device=DEV)
    M0 = Mbig.clone()
    fb.flora_momentum_step(Gbig[:, :m], Mbig[:, :r], 0.9, 9)
    ref = oracle_compress(Gbig[:, :m].contiguous(), M0[:, :r].contiguous(), 9, a=0.1, b=0.9)
    assert rel_err(Mbig[:, :r].cpu().numpy(), ref) <= TOL["bf16"]
    fb.flora_resample_transfer(Mbig[:, :r], m, "bf16", 9, 10)
    assert torch.equal(Mbig[:, r:], M0[:, r:])


def test_empty_inputs():
    z = torch.zeros(0, 16, device=DEV)
    fb.flora_compress_accumulate(z, torch.zeros(0, 4, device=DEV), 1, 4)
    C = torch.ones(8, 4, device=DEV)
    fb.flora_compress_accumulate(torch.zeros(8, 0, device=DEV), C, 1, 4)
    assert torch.all(C == 1)
    fb.flora_decompress_apply(torch.zeros(8, 0, device=DEV), C, 1, 1.0, 1.0)
    fb.flora_resample_transfer(torch.zeros(0, 4, device=DEV), 16, "f32", 1, 2)
    M = torch.ones(3, 4, device=DEV)
    fb.flora_resample_transfer(M, 0, "f32", 1, 2)              # A has no columns: A A'^T = 0
    assert torch.all(M == 0)


# --------------------------------------------------------------------------------------- configs
def test_config_single_f32_accumulation_cycle():
    w = wl.WORKLOADS["single_f32_512"]
    n, m = w.shapes[0]
    seedA = 42
    C = torch.zeros(n, w.r, device=DEV)
    Cref = np.zeros((n, w.r), dtype=np.float32)
    A = orc.projection(seedA, w.r, m, "f32")
    for i in range(w.tau):
        G = wl.gradient(w, 0, i)
        fb.flora_compress_accumulate(G.to(DEV), C, seedA, w.r)
        orc.compress_accumulate(wl.as_numpy(G), A, Cref)
    assert rel_err(C.cpu().numpy(), Cref) <= TOL["f32"]
    W0 = wl.weight(w, 0)
    W = W0.to(DEV)
    fb.flora_decompress_apply(W, C, seedA, w.lr, 1.0 / w.tau)
    Wref = wl.as_numpy(W0).copy()
    orc.decompress_apply(Wref, Cref, A, w.lr, 1.0 / w.tau)
    assert rel_err(W.cpu().numpy(), Wref) <= TOL["f32"]
    # the update itself (about 1e-3 of |W|): W is stored in fp32, so each side carries up to half an ulp of W
    w0 = wl.as_numpy(W0).astype(np.float64)
    upd_ref, upd_got = Wref - w0, W.cpu().numpy() - w0
    ulp = float(np.spacing(np.float32(np.abs(Wref).max())))
    assert np.abs(upd_got - upd_ref).max() <= TOL["f32"] * np.abs(upd_ref).max() + ulp


def _small_set(dtype, r, shapes):
    G = [_g(n, m, dtype, 100 + i, var=1e-3) for i, (n, m) in enumerate(shapes)]
    W = [_g(n, m, dtype, 200 + i, var=4e-4) for i, (n, m) in enumerate(shapes)]
    S = [torch.zeros(n, r, device=DEV) for n, _ in shapes]
    return G, W, S


@pytest.mark.parametrize("force_simt", [0, 1])
def test_set_accumulation_cycle_and_momentum(force_simt):
    fb.flora_debug_force_path(force_simt)
    shapes = [(96, 288), (96, 96), (96, 384), (384, 96), (130, 200)]
    r, tau = 32, 3
    G, W, S = _small_set("bf16", r, shapes)
    W0 = [w.clone() for w in W]
    fset = fb.FloraSet(G, W, S)
    seeds = [fb.flora_derive_seed(1, i, 0) for i in range(len(shapes))]
    Sref = [np.zeros((n, r), dtype=np.float32) for n, _ in shapes]
    for step in range(tau):
        Gs = [_g(n, m, "bf16", 1000 * step + i, var=1e-3) for i, (n, m) in enumerate(shapes)]
        fset.rebind_gradients(Gs)
        fset.compress_accumulate(seeds)
        for i in range(len(shapes)):
            Sref[i] = oracle_compress(Gs[i], torch.from_numpy(Sref[i]), seeds[i])
    for i in range(len(shapes)):
        assert rel_err(S[i].cpu().numpy(), Sref[i]) <= TOL["bf16"], i
    fset.decompress_apply(seeds, 30.0, 1.0 / tau)
    for i in range(len(shapes)):
        ref = oracle_decompress(W0[i], S[i], seeds[i], 30.0, 1.0 / tau)
        assert rel_err(values(wl.as_numpy(W[i])), values(ref)) <= TOL["bf16"], i
    # momentum with a transfer
    new = [fb.flora_derive_seed(1, i, 1) for i in range(len(shapes))]
    Sbefore = [s.clone() for s in S]
    fset.resample_transfer(seeds, new)
    for i, (n, m) in enumerate(shapes):
        assert rel_err(S[i].cpu().numpy(), oracle_transfer(Sbefore[i], Sbefore[i], m, "bf16", seeds[i], new[i], 1.0, 0.0)) <= TOL["bf16"]
    Sbefore = [s.clone() for s in S]
    fset.momentum_step(0.9, new)
    for i in range(len(shapes)):
        assert rel_err(S[i].cpu().numpy(), oracle_compress(fset.G[i], Sbefore[i], new[i], a=1.0 - float(np.float32(0.9)), b=0.9)) <= TOL["bf16"]
    fset.zero_state()
    assert all(torch.all(s == 0) for s in S)
    fset.close()


def test_set_on_tensor_core_eligible_shapes():
    shapes = [(256, 576), (384, 128), (128, 1088), (640, 320), (200, 264), (1536, 2048)]
    r = 32
    G, W, S = _small_set("bf16", r, shapes)
    S0 = [torch.randn_like(s) for s in S]
    for s, s0 in zip(S, S0):
        s.copy_(s0)
    fset = fb.FloraSet(G, W, S)
    seeds = [fb.flora_derive_seed(9, i, 0) for i in range(len(shapes))]
    fset.compress_accumulate(seeds)
    for i in range(len(shapes)):
        assert rel_err(S[i].cpu().numpy(), oracle_compress(G[i], S0[i], seeds[i])) <= TOL["bf16"], i
    S1 = [s.clone() for s in S]
    fset.momentum_step(0.5, seeds)
    for i in range(len(shapes)):
        assert rel_err(S[i].cpu().numpy(), oracle_compress(G[i], S1[i], seeds[i], a=0.5, b=0.5)) <= TOL["bf16"], i
    W0 = [w.clone() for w in W]
    fset.decompress_apply(seeds, 0.01, 1.0)
    for i in range(len(shapes)):
        ref = oracle_decompress(W0[i], S[i], seeds[i], 0.01, 1.0)
        assert rel_err(values(wl.as_numpy(W[i])), values(ref)) <= TOL["bf16"], i
    fset.close()


@pytest.mark.parametrize("r", [130, 200, 256])
def test_set_decompress_on_cta_pairs_many_short_items(r):
    """Ranks above 128 decompress on CTA pairs whose two MMA-issuing threads take tile iterations in turn across item
    boundaries: a set with more column slabs than there are pairs, of matrices with 1 to 7 row tiles (odd and even
    counts, ragged last tiles, a last slab of 8 to 72 live columns), compared element by element with the oracle."""
    rng = np.random.default_rng(77)
    shapes = [(int(rng.integers(1, 8)) * 128 - int(rng.integers(0, 120)), int(rng.integers(2, 7)) * 128 + int(rng.choice([8, 64, 72, 128])))
              for _ in range(64)]
    G, W, S = _small_set("bf16", r, shapes)
    for i, s_ in enumerate(S):
        s_.copy_(torch.from_numpy(np.random.default_rng(500 + i).standard_normal(tuple(s_.shape)).astype(np.float32)))
    W0 = [w.clone() for w in W]
    fset = fb.FloraSet(G, W, S)
    seeds = [fb.flora_derive_seed(21, i, 0) for i in range(len(shapes))]
    fset.decompress_apply(seeds, 0.02, 1.0)
    torch.cuda.synchronize()
    for i in range(len(shapes)):
        ref = oracle_decompress(W0[i], S[i], seeds[i], 0.02, 1.0)
        w0 = values(wl.as_numpy(W0[i])).astype(np.float64)
        assert rel_err(values(wl.as_numpy(W[i])), values(ref)) <= TOL["bf16"], (i, shapes[i])
        assert rel_err(values(wl.as_numpy(W[i])) - w0, values(ref) - w0) <= TOL["bf16"], (i, shapes[i])
    fset.close()


def test_host_to_device_entry_points():
    shapes = [(64, 160), (40, 72)]
    r = 8
    G, W, S = _small_set("bf16", r, shapes)
    fset = fb.FloraSet(G, W, S)
    hostG = [wl.gaussian_matrix(n, m, 1e-3, "bf16", 50 + i).pin_memory() for i, (n, m) in enumerate(shapes)]
    seeds = [5, 6]
    fset.compress_accumulate_from_host(hostG, seeds)
    torch.cuda.synchronize()
    for i in range(2):
        assert torch.equal(G[i].cpu(), hostG[i])
        assert rel_err(S[i].cpu().numpy(), oracle_compress(hostG[i], torch.zeros(shapes[i][0], r), seeds[i])) <= TOL["bf16"]
    hostW = [torch.empty(n, m, dtype=torch.bfloat16).pin_memory() for n, m in shapes]
    fset.read_weights_to_host(hostW)
    torch.cuda.synchronize()
    assert all(torch.equal(hostW[i], W[i].cpu()) for i in range(2))
    fset.close()


# --------------------------------------------------------------------------------------- full-size configs, sampled rows
@pytest.mark.parametrize("name", ["gpt2_small_set"])
def test_full_size_set_sampled_rows(name):
    """The benchmark's step at full size and in its launch configuration: tau gradient sets bound to one set of weights
    and sketches, tau compressions, one decompress-apply with scale 1/tau, the reset of C; sampled rows replayed on the oracle."""
    w = wl.WORKLOADS[name]
    count = len(w.shapes)
    G = [[wl.gradient(w, i, k, device=DEV) for i in range(count)] for k in range(w.tau)]
    W = [wl.weight(w, i, device=DEV, std=0.02) for i in range(count)]
    W0 = [x.clone() for x in W]
    S = [torch.zeros(n, w.r, device=DEV) for n, _ in w.shapes]
    sets = [fb.FloraSet(G[k], W, S) for k in range(w.tau)]
    seeds = [fb.flora_derive_seed(3, i, 0) for i in range(count)]
    for k in range(w.tau):
        sets[k].compress_accumulate(seeds)
    Sacc = [x.clone() for x in S]
    sets[0].decompress_apply(seeds, 4.0, 1.0 / w.tau)
    sets[0].zero_state()
    torch.cuda.synchronize()
    assert fb.flora_device_status() == 0
    for i in range(0, count, 5):
        n, m = w.shapes[i]
        rows = sample_rows(n, 24, i)
        idx = torch.from_numpy(rows).to(DEV)
        c = np.zeros((len(rows), w.r), dtype=np.float32)
        for k in range(w.tau):
            c = oracle_compress(G[k][i][idx].cpu(), torch.from_numpy(c), seeds[i])
        got = Sacc[i].cpu().numpy()[rows]
        assert rel_err(got, c) <= TOL["bf16"], i
        ref = oracle_decompress(W0[i][idx].cpu(), torch.from_numpy(got), seeds[i], 4.0, 1.0 / w.tau)
        assert rel_err(values(wl.as_numpy(W[i])[rows]), values(ref)) <= TOL["bf16"], i
        assert not S[i].any()                                                      # C is zero again for the next cycle
    for s_ in sets:
        s_.close()


# --------------------------------------------------------------------------------------- robustness
def test_more_matrices_than_one_launch_carries_seeds_for():
    """460 matrices: the set is cut into two launches (seeds travel as a kernel parameter, 448 per launch)."""
    count, n, m, r = 460, 128, 128, 16
    torch.manual_seed(1)
    Gbig = (torch.randn(count, n, m, device=DEV) * 0.03).to(torch.bfloat16)
    Wbig = (torch.randn(count, n, m, device=DEV) * 0.02).to(torch.bfloat16)
    Sbig = torch.zeros(count, n, r, device=DEV)
    G, W, S = [Gbig[i] for i in range(count)], [Wbig[i] for i in range(count)], [Sbig[i] for i in range(count)]
    W0 = Wbig.clone()
    fset = fb.FloraSet(G, W, S)
    seeds = [fb.flora_derive_seed(2, i, 0) for i in range(count)]
    fset.compress_accumulate(seeds)
    fset.momentum_step(0.5, seeds)
    fset.decompress_apply(seeds, 2.0, 1.0)
    torch.cuda.synchronize()
    for i in (0, 1, 447, 448, 449, 459):
        c1 = oracle_compress(G[i], torch.zeros(n, r), seeds[i])
        c2 = oracle_compress(G[i], torch.from_numpy(c1), seeds[i], a=0.5, b=0.5)
        assert rel_err(S[i].cpu().numpy(), c2) <= TOL["bf16"], i
        ref = oracle_decompress(W0[i], S[i], seeds[i], 2.0, 1.0)
        assert rel_err(values(wl.as_numpy(W[i])), values(ref)) <= TOL["bf16"], i
    fset.close()


def test_bounded_wait_gives_up_and_reports_a_timeout():
    """A wait that can never be satisfied returns after its limit, the status says so, and the device keeps working."""
    assert fb.flora_debug_wait_timeout_selftest() == 7                 # FLORA_ERR_TIMEOUT
    assert fb.flora_device_status() == 7                               # the error word was raised ...
    assert fb.flora_device_status() == 0                               # ... and reading it cleared it
    C = torch.zeros(256, 8, device=DEV)
    G = _g(256, 512, "bf16", 3)
    fb.flora_compress_accumulate(G, C, 5, 8)
    assert rel_err(C.cpu().numpy(), oracle_compress(G, torch.zeros(256, 8), 5)) <= TOL["bf16"]


@pytest.mark.parametrize("n,m,r", [(2048, 2304, 32), (4096, 1024, 128), (1600, 1600, 256), (768, 3072, 64)])
def test_repeated_launches_are_bit_identical(n, m, r):
    """Race detector: the same call, repeated, must give the same bits wherever the arithmetic fixes the order of
    the additions (decompression always; compression when every row of the sketch has a single owner)."""
    G = _g(n, m, "bf16", 11)
    items, _ = fb.flora_debug_plan([(n, m)], r, "compress")
    owned = all(it[5] == 1 for it in items)
    first_c = first_m = first_w = None
    W0 = (torch.randn(n, m, device=DEV) * 0.02).to(torch.bfloat16)
    S = torch.randn(n, r, device=DEV)
    for it in range(25):
        C = torch.zeros(n, r, device=DEV)
        fb.flora_compress_accumulate(G, C, 9, r)
        M = torch.ones(n, r, device=DEV)
        fb.flora_momentum_step(G, M, 0.75, 9)
        W = W0.clone()
        fb.flora_decompress_apply(W, S, 9, 0.5, 1.0)
        if it == 0:
            first_c, first_m, first_w = C, M, W
        else:
            assert torch.equal(W, first_w)
            if owned:
                assert torch.equal(C, first_c) and torch.equal(M, first_m)
            else:
                assert rel_err(C.cpu().numpy(), first_c.cpu().numpy()) <= 1e-5
    assert fb.flora_device_status() == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,m,r", [(9, 33, 4), (300, 1024, 32), (256, 4096, 128), (1000, 515, 17)])
def test_resampled_momentum_step(n, m, r, dtype):
    """Algorithm 2 at a resampling step as one call, against the oracle's transfer followed by its momentum step."""
    G = _g(n, m, dtype, 21)
    M0 = torch.randn(n, r, device=DEV)
    M = M0.clone()
    fb.flora_momentum_step_resampled(G, M, 0.9, 40, 41)
    ref = wl.as_numpy(M0).copy()
    orc.momentum_step_resampled(wl.as_numpy(G), orc.projection(40, r, m, dtype), orc.projection(41, r, m, dtype), 0.9, ref)
    assert rel_err(M.cpu().numpy(), ref) <= TOL[dtype]
    # and the set-level call over several matrices
    shapes = [(256, 512), (384, 1024), (128, 64)]
    Gs = [_g(a, b, "bf16", 30 + i) for i, (a, b) in enumerate(shapes)]
    Ms = [torch.randn(a, r, device=DEV) for a, _ in shapes]
    M0s = [x.clone() for x in Ms]
    fset = fb.FloraSet(Gs, None, Ms)
    old, new = [50, 51, 52], [60, 61, 62]
    fset.momentum_step_resampled(0.5, old, new)
    for i, (a, b) in enumerate(shapes):
        ref = wl.as_numpy(M0s[i]).copy()
        orc.momentum_step_resampled(wl.as_numpy(Gs[i]), orc.projection(old[i], r, b, "bf16"), orc.projection(new[i], r, b, "bf16"), 0.5, ref)
        assert rel_err(Ms[i].cpu().numpy(), ref) <= TOL["bf16"], i
    fset.close()


@pytest.mark.parametrize("case", range(14))
def test_random_sets_against_oracle(case):
    """Seeded random weight sets (shapes on both sides of every eligibility rule of the tensor-core path, ranks that are
    and are not multiples of 4, 16, 64), run through every set-level operation and compared with the oracle."""
    rng = np.random.default_rng(1000 + case)
    r = int(rng.choice([1, 4, 8, 17, 32, 48, 64, 100, 128, 200, 256]))
    count = int(rng.integers(1, 5))
    eligible = case % 3 != 0                     # two thirds of the cases: every matrix large and aligned enough for tcgen05
    shapes = []
    for _ in range(count):
        if eligible:
            shapes.append((int(rng.integers(128, 700)), int(rng.integers(8, 300)) * 8))
        else:
            shapes.append((int(rng.integers(1, 300)), int(rng.integers(1, 700))))
    G = [_g(n, m, "bf16", 100 * case + i) for i, (n, m) in enumerate(shapes)]
    W = [(torch.randn(n, m, device=DEV) * 0.02).to(torch.bfloat16) for n, m in shapes]
    W0 = [x.clone() for x in W]
    S = [torch.zeros(n, r, device=DEV) for n, _ in shapes]
    fset = fb.FloraSet(G, W, S)
    s0 = [int(x) for x in rng.integers(1, 2 ** 62, size=count)]
    s1 = [int(x) for x in rng.integers(1, 2 ** 62, size=count)]
    fset.compress_accumulate(s0)
    fset.compress_accumulate(s0)
    fset.momentum_step(0.7, s0)
    fset.momentum_step_resampled(0.6, s0, s1)
    fset.decompress_apply(s1, 0.5, 0.25)
    torch.cuda.synchronize()
    assert fb.flora_device_status() == 0
    for i, (n, m) in enumerate(shapes):
        A0, A1 = orc.projection(s0[i], r, m, "bf16"), orc.projection(s1[i], r, m, "bf16")
        g = wl.as_numpy(G[i])
        ref = np.zeros((n, r), dtype=np.float32)
        orc.compress_accumulate(g, A0, ref)
        orc.compress_accumulate(g, A0, ref)
        orc.momentum_step(g, A0, 0.7, ref)
        orc.momentum_step_resampled(g, A0, A1, 0.6, ref)
        assert rel_err(S[i].cpu().numpy(), ref) <= TOL["bf16"], (case, i, "sketch")
        w = wl.as_numpy(W0[i]).copy()
        orc.decompress_apply(w, S[i].cpu().numpy(), A1, 0.5, 0.25)
        assert rel_err(values(wl.as_numpy(W[i])), values(w)) <= TOL["bf16"], (case, i, "weights")
    fset.close()
