"""GPU tests of what lives across calls: sets of different footprint alive together, bit-reproducible mode,
resuming from saved state, and how close the tensor-core compression really is to the oracle."""
import numpy as np
import pytest
import torch

from oracle import flora_oracle as orc
from paper_2402_03293_b200 import binding as fb
from paper_2402_03293_b200 import hostlogic
from paper_2402_03293_b200 import workloads as wl
from tests.parity_util import TOL, oracle_compress, oracle_decompress, rel_err, values

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(autouse=True)
def _clean():
    fb.flora_debug_force_path(0)
    fb.flora_set_deterministic(False)
    yield
    fb.flora_set_deterministic(False)
    torch.cuda.synchronize()
    assert fb.flora_device_status() == 0


def _g(n, m, seed, var=1e-2):
    return wl.gaussian_matrix(n, m, var, "bf16", seed).to(DEV)


def test_sets_of_different_shared_memory_footprint_stay_usable_together():
    """The limit on a kernel's dynamic shared memory belongs to the kernel, not to a launch: a set that needs little
    must not lower it for a live set that needs all of it.  A rank-256 set, then a rank-8 set and single-matrix calls,
    then the first set again, all against the oracle."""
    big_shapes, small_shapes = [(512, 1024), (384, 640)], [(256, 512)]
    Gb = [_g(n, m, 1 + i) for i, (n, m) in enumerate(big_shapes)]
    Wb = [(torch.randn(n, m, device=DEV) * 0.02).to(torch.bfloat16) for n, m in big_shapes]
    Cb = [torch.zeros(n, 256, device=DEV) for n, _ in big_shapes]
    big = fb.FloraSet(Gb, Wb, Cb)
    big.compress_accumulate([5, 6])
    Gs = [_g(n, m, 9) for n, m in small_shapes]
    Ws = [(torch.randn(n, m, device=DEV) * 0.02).to(torch.bfloat16) for n, m in small_shapes]
    Cs = [torch.zeros(n, 8, device=DEV) for n, _ in small_shapes]
    small = fb.FloraSet(Gs, Ws, Cs)
    small.compress_accumulate([7])
    small.decompress_apply([7], 0.5, 1.0)
    one_c = torch.zeros(256, 8, device=DEV)
    fb.flora_compress_accumulate(Gs[0], one_c, 7, 8)                     # single-matrix calls plan a set of their own
    one_w = Ws[0].clone()
    fb.flora_decompress_apply(one_w, one_c, 7, 0.25, 1.0)
    W0 = [w.clone() for w in Wb]
    big.compress_accumulate([5, 6])                                      # the rank-256 set again, at its full footprint
    big.decompress_apply([5, 6], 0.5, 0.5)
    torch.cuda.synchronize()
    for i in range(2):
        want = np.zeros(Cb[i].shape, dtype=np.float32)
        A = orc.projection(5 + i, 256, big_shapes[i][1], "bf16")
        for _ in range(2):
            orc.compress_accumulate(wl.as_numpy(Gb[i]), A, want)
        assert rel_err(Cb[i].cpu().numpy(), want) <= TOL["bf16"]
        wref = oracle_decompress(W0[i], Cb[i], 5 + i, 0.5, 0.5)
        assert rel_err(values(wl.as_numpy(Wb[i])), values(wref)) <= TOL["bf16"]
    assert rel_err(one_c.cpu().numpy(), oracle_compress(Gs[0], torch.zeros_like(one_c), 7)) <= TOL["bf16"]
    big.close()
    small.close()


@pytest.mark.parametrize("n,m,r", [(256, 8192, 32), (512, 16384, 256), (384, 12288, 128)])
def test_deterministic_mode_gives_the_same_bits_every_time(n, m, r):
    """Few rows and many columns: by default the planner splits such a matrix over column ranges whose partial sums
    are added in arrival order.  With flora_set_deterministic every row of the sketch has one owner, and the r x r
    product of the transfer is summed by one CTA: 25 repeats must agree bit for bit, and still match the oracle."""
    items, _ = fb.flora_debug_plan([(n, m)], r, "compress")
    assert any(it[5] == 0 for it in items), "the default plan was expected to split this shape over columns"
    fb.flora_set_deterministic(True)
    items, _ = fb.flora_debug_plan([(n, m)], r, "compress")
    assert all(it[5] == 1 for it in items)
    G = _g(n, m, 3)
    M0 = torch.randn(n, r, device=DEV)
    first = None
    for it in range(25):
        C = torch.zeros(n, r, device=DEV)
        fset = fb.FloraSet([G], None, [C])
        fset.compress_accumulate([11])
        fset.momentum_step(0.9, [11])
        fset.close()
        M = M0.clone()
        fb.flora_resample_transfer(M, m, "bf16", 11, 12)
        if first is None:
            first = (C, M)
        else:
            assert torch.equal(C, first[0]) and torch.equal(M, first[1])
    want = np.zeros((n, r), dtype=np.float32)
    A = orc.projection(11, r, m, "bf16")
    orc.compress_accumulate(wl.as_numpy(G), A, want)
    orc.momentum_step(wl.as_numpy(G), A, 0.9, want)
    assert rel_err(first[0].cpu().numpy(), want) <= TOL["bf16"]


def test_resuming_from_saved_state_gives_identical_bits():
    """The state of the method is {sketches, seeds, step counters} (Section 2.4: store the seed, not the projection).
    2k steps in one go, against k steps, a copy of the state into fresh tensors and a fresh set, and k more."""
    fb.flora_set_deterministic(True)
    shapes, r, k = [(384, 1024), (256, 640), (1600, 1600)], 128, 3
    count = len(shapes)

    def grads(t):
        return [_g(n, m, 100 * t + i) for i, (n, m) in enumerate(shapes)]

    def fresh():
        W = [wl.gaussian_matrix(n, m, 4e-4, "bf16", 50 + i).to(DEV) for i, (n, m) in enumerate(shapes)]
        M = [torch.zeros(n, r, device=DEV) for n, _ in shapes]
        return W, M

    # momentum with resampling (Algorithm 2), kappa = 2
    W, M = fresh()
    fset = fb.FloraSet(grads(0), W, M)
    mom = hostlogic.MomentumState(fset, count, 0.9, 2, base_seed=4)
    for t in range(2 * k):
        fset.rebind_gradients(grads(t))
        mom.step(0.5)
    torch.cuda.synchronize()
    fset.close()
    W2, M2 = fresh()
    fset2 = fb.FloraSet(grads(0), W2, M2)
    mom2 = hostlogic.MomentumState(fset2, count, 0.9, 2, base_seed=4)
    for t in range(k):
        fset2.rebind_gradients(grads(t))
        mom2.step(0.5)
    torch.cuda.synchronize()
    saved = {"W": [w.cpu() for w in W2], "M": [x.cpu() for x in M2], "t": mom2.t, "epoch": mom2.epoch}
    fset2.close()
    W3, M3 = [w.to(DEV) for w in saved["W"]], [x.to(DEV) for x in saved["M"]]
    fset3 = fb.FloraSet(grads(0), W3, M3)
    mom3 = hostlogic.MomentumState(fset3, count, 0.9, 2, base_seed=4)
    mom3.t, mom3.epoch = saved["t"], saved["epoch"]
    for t in range(k, 2 * k):
        fset3.rebind_gradients(grads(t))
        mom3.step(0.5)
    torch.cuda.synchronize()
    for i in range(count):
        assert torch.equal(M[i], M3[i]) and torch.equal(W[i], W3[i]), i
    fset3.close()

    # accumulation cycles (Algorithm 1), tau = 2: stop in the middle of a cycle
    def run(cycles_then_micro, state=None):
        W, _ = fresh()
        C = [torch.zeros(n, r, device=DEV) for n, _ in shapes]
        if state:
            W, C = [w.to(DEV) for w in state["W"]], [c.to(DEV) for c in state["C"]]
        s = fb.FloraSet(grads(0), W, C)
        cyc = hostlogic.AccumulationCycle(s, count, 2, base_seed=8)
        if state:
            cyc.epoch, cyc.micro_step = state["epoch"], state["micro"]
        first, last = cycles_then_micro
        for t in range(first, last):
            s.rebind_gradients(grads(t))
            if cyc.accumulate():
                cyc.apply(0.5)
        torch.cuda.synchronize()
        out = {"W": [w.cpu() for w in W], "C": [c.cpu() for c in C], "epoch": cyc.epoch, "micro": cyc.micro_step}
        s.close()
        return out

    whole = run((0, 5))
    part = run((3, 5), state=run((0, 3)))
    for i in range(count):
        assert torch.equal(whole["W"][i], part["W"][i]) and torch.equal(whole["C"][i], part["C"][i]), i


@pytest.mark.parametrize("n,m,r", [(512, 4096, 32), (1600, 6400, 256), (4096, 11008, 128)])
def test_compression_is_far_closer_to_the_oracle_than_the_tolerance_asks(n, m, r):
    """Both sides multiply the same bf16-rounded G and A, whose products are exact in fp32, so all that separates the
    tensor-core sum from the oracle's double-precision sum is fp32 accumulation over m terms: a bound of
    m * 2^-24 * sum|g a| per element, far inside 2e-2.  A dropped or doubled 8-column chunk would show up here.
    Checked on sampled rows, normwise and relative to sum_k |G_ik| |A_jk| per element."""
    G = _g(n, m, 17, var=1e-3)
    C = torch.zeros(n, r, device=DEV)
    fb.flora_compress_accumulate(G, C, 23, r)
    torch.cuda.synchronize()
    rows = np.unique(np.linspace(0, n - 1, 24).astype(np.int64))
    Gn = np.ascontiguousarray(wl.as_numpy(G)[rows])
    A = orc.projection(23, r, m, "bf16")
    want = np.zeros((len(rows), r), dtype=np.float32)
    orc.compress_accumulate(Gn, A, want)
    got = C.cpu().numpy()[rows]
    normwise = rel_err(got, want)
    mags = np.abs(orc.bf16_bits_to_f32(Gn).astype(np.float64)) @ np.abs(A.astype(np.float64)).T
    componentwise = float((np.abs(got.astype(np.float64) - want) / mags).max())
    print(f"compress {n}x{m} r={r}: normwise {normwise:.2e}, componentwise {componentwise:.2e}")
    assert normwise <= 2e-5
    assert componentwise <= m * 2.0 ** -24


@pytest.mark.parametrize("r", [32, 256])
def test_first_compression_of_a_cycle_overwrites_whatever_the_sketch_held(r):
    """Algorithm 1 starts a cycle from C = 0; the host classes fold that into the first compression (C <- G A^T).  The
    result must not depend on what C held before (here NaN and huge values) and must equal zeroing followed by an
    accumulating compression: to the bit where every row of a sketch has one writer, to rounding where a wide matrix is
    split along its columns and partial sums are added in whatever order they arrive."""
    shapes = [(384, 1024), (130, 200), (128, 16384), (1600, 1600)]
    G = [_g(n, m, 40 + i) for i, (n, m) in enumerate(shapes)]
    W = [torch.zeros(n, m, device=DEV, dtype=torch.bfloat16) for n, m in shapes]
    S = [torch.full((n, r), float("nan"), device=DEV) for n, _ in shapes]
    S[0].fill_(3e38)
    fset = fb.FloraSet(G, W, S)
    seeds = [fb.flora_derive_seed(4, i, 0) for i in range(len(shapes))]
    fset.compress_overwrite(seeds)
    first = [s.clone() for s in S]
    fset.zero_state()
    fset.compress_accumulate(seeds)
    torch.cuda.synchronize()
    for i, (n, m) in enumerate(shapes):
        assert torch.isfinite(first[i]).all(), i
        assert rel_err(first[i].cpu().numpy(), S[i].cpu().numpy()) <= 1e-6, i
        assert rel_err(first[i].cpu().numpy(), oracle_compress(G[i], torch.zeros(n, r), seeds[i])) <= TOL["bf16"], i
    assert torch.equal(first[1], S[1])          # a small matrix has one owner per row in either schedule
    # the host class uses it: a second cycle starts from the first cycle's leftovers without a zeroing call
    cyc = hostlogic.AccumulationCycle(fset, len(shapes), tau=2, base_seed=6)
    for _ in range(2):
        cyc.accumulate()
        cyc.accumulate()
        s_used = cyc.seeds()
        cyc.apply(0.0)
    for i, (n, m) in enumerate(shapes):
        two = oracle_compress(G[i], torch.from_numpy(oracle_compress(G[i], torch.zeros(n, r), s_used[i])), s_used[i])
        assert rel_err(S[i].cpu().numpy(), two) <= TOL["bf16"], i
    fset.close()
