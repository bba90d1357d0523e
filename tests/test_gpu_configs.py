"""Full-size parity on the paper-shaped configurations, in the launch configuration that is timed.

The oracle cannot afford whole matrices at these sizes, but every row of a sketch and of a weight matrix depends
only on the same row of the gradient, the seed(s) and (for the transfer) the r x r product, so replaying the
whole sequence of operations on a sample of rows of a sample of matrices is an exact check of those rows."""
import numpy as np
import pytest
import torch

from oracle import flora_oracle as orc
from paper_2402_03293_b200 import binding as fb
from paper_2402_03293_b200 import hostlogic
from paper_2402_03293_b200 import workloads as wl
from tests.parity_util import TOL, rel_err, sample_rows, values

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(autouse=True)
def _clean():
    fb.flora_debug_force_path(0)
    yield
    torch.cuda.synchronize()
    assert fb.flora_device_status() == 0


def _rows_of(t, rows):
    return t[torch.from_numpy(rows).to(t.device)].cpu()


class _Replay:
    """The oracle's copy of a few rows of one matrix: replays the calls the set makes."""

    def __init__(self, rows, r, m, dtype, W0):
        self.rows, self.r, self.m, self.dtype = rows, r, m, dtype
        self.S = np.zeros((len(rows), r), dtype=np.float32)
        self.W = wl.as_numpy(_rows_of(W0, rows)).copy()

    def A(self, seed):
        return orc.projection(seed, self.r, self.m, self.dtype)

    def compress(self, G, seed):
        orc.compress_accumulate(wl.as_numpy(_rows_of(G, self.rows)), self.A(seed), self.S)

    def momentum(self, G, beta, seed):
        orc.momentum_step(wl.as_numpy(_rows_of(G, self.rows)), self.A(seed), beta, self.S)

    def transfer(self, s_old, s_new):
        orc.resample_transfer(self.S, self.A(s_old), self.A(s_new))

    def decompress(self, seed, lr, scale):
        orc.decompress_apply(self.W, self.S, self.A(seed), lr, scale)


class _Mirror:
    """Stands between the host sequencing and the set: forwards every call and replays it on the oracle rows."""

    def __init__(self, fset, replays, current_G):
        self.fset, self.replays, self.G = fset, replays, current_G

    def compress_accumulate(self, seeds, stream=None):
        self.fset.compress_accumulate(seeds, stream)
        for i, rp in self.replays.items():
            rp.compress(self.G()[i], seeds[i])

    def compress_overwrite(self, seeds, stream=None):
        self.fset.compress_overwrite(seeds, stream)
        for i, rp in self.replays.items():                        # Algorithm 1 as printed: C <- 0, then C += G A^T
            rp.S[:] = 0
            rp.compress(self.G()[i], seeds[i])

    def momentum_step(self, beta, seeds, stream=None):
        self.fset.momentum_step(beta, seeds, stream)
        for i, rp in self.replays.items():
            rp.momentum(self.G()[i], beta, seeds[i])

    def resample_transfer(self, old, new, stream=None):
        self.fset.resample_transfer(old, new, stream)
        for i, rp in self.replays.items():
            rp.transfer(old[i], new[i])

    def momentum_step_resampled(self, beta, old, new, stream=None):
        self.fset.momentum_step_resampled(beta, old, new, stream)
        for i, rp in self.replays.items():                        # the oracle takes Algorithm 2's two steps in order
            rp.transfer(old[i], new[i])
            rp.momentum(self.G()[i], beta, new[i])

    def transfer_axpby_from(self, src, old, new, a, b, stream=None):
        self.fset.transfer_axpby_from(src.fset, old, new, a, b, stream)
        for i, rp in self.replays.items():
            orc.transfer_axpby(rp.S, src.replays[i].S, rp.A(old[i]), rp.A(new[i]), float(np.float32(a)), float(np.float32(b)))

    def decompress_apply(self, seeds, lr, scale, stream=None):
        self.fset.decompress_apply(seeds, lr, scale, stream)
        for i, rp in self.replays.items():
            rp.decompress(seeds[i], lr, scale)

    def zero_state(self, stream=None):
        self.fset.zero_state(stream)
        for rp in self.replays.values():
            rp.S[:] = 0


def _check(replays, S, W, dtype, what):
    for i, rp in replays.items():
        assert rel_err(S[i].cpu().numpy()[rp.rows], rp.S) <= TOL[dtype], (what, "sketch", i)
        assert rel_err(values(wl.as_numpy(W[i])[rp.rows]), values(rp.W)) <= TOL[dtype], (what, "weights", i)


def test_t5_large_set_momentum_with_transfer():
    w = wl.WORKLOADS["t5_large_set"]
    count = len(w.shapes)
    W = [wl.weight(w, i, device=DEV, std=0.02) for i in range(count)]
    M = [torch.zeros(n, w.r, device=DEV) for n, _ in w.shapes]
    G = [wl.gradient(w, i, 0, device=DEV) for i in range(count)]
    picked = list(range(0, count, 37)) + [count - 1]
    replays = {i: _Replay(sample_rows(w.shapes[i][0], 12, i), w.r, w.shapes[i][1], w.dtype, W[i]) for i in picked}
    fset = fb.FloraSet(G, W, M)
    cur = [G]
    mom = hostlogic.MomentumState(_Mirror(fset, replays, lambda: cur[0]), count, w.beta, kappa=2, base_seed=3)
    for t in range(3):                               # t = 2 resamples: transfer, then update and yield with the new projection
        if t:
            cur[0] = [wl.gradient(w, i, t, device=DEV) for i in range(count)]
            fset.rebind_gradients(cur[0])
        mom.step(lr=2.0)
    torch.cuda.synchronize()
    _check(replays, M, W, w.dtype, "t5_large_set")
    fset.close()


@pytest.mark.parametrize("r", [8, 32, 128, 256])
def test_single_bf16_matrix_rank_sweep_resample_every_step(r):
    w = wl.WORKLOADS["single_bf16_4096x11008"]
    n, m = w.shapes[0]
    W = [wl.weight(w, 0, device=DEV, std=0.02)]
    M = [torch.zeros(n, r, device=DEV)]
    G = [wl.gradient(w, 0, 0, device=DEV)]
    replays = {0: _Replay(sample_rows(n, 16, r), r, m, w.dtype, W[0])}
    fset = fb.FloraSet(G, W, M)
    cur = [G]
    mom = hostlogic.MomentumState(_Mirror(fset, replays, lambda: cur[0]), 1, w.beta, kappa=1, base_seed=r,
                                  skip_transfer_of_zero_state=False)
    for t in range(2):
        if t:
            cur[0] = [wl.gradient(w, 0, t, device=DEV)]
            fset.rebind_gradients(cur[0])
        mom.step(lr=0.5 if t == 0 else 0.5 * r / m)          # the transfer scales the state by about sqrt(m/r)
    torch.cuda.synchronize()
    _check(replays, M, W, w.dtype, ("single", r))
    fset.close()


def test_gpt2_xl_set_accumulation_into_momentum_with_outliers():
    w = wl.WORKLOADS["gpt2_xl_set"]
    count, tau = len(w.shapes), 2                    # two of the sixteen micro-steps keep the test short
    W = [wl.weight(w, i, device=DEV, std=0.02) for i in range(count)]
    # C holds leftovers (here NaN): a cycle's first compression overwrites it, which stands for Algorithm 1's C <- 0
    C = [torch.full((n, w.r), float("nan"), device=DEV) for n, _ in w.shapes]
    M = [torch.randn(n, w.r, device=DEV) * 0.01 for n, _ in w.shapes]
    picked = list(range(1, count, 29)) + [count - 1]
    rows = {i: sample_rows(w.shapes[i][0], 8, i) for i in picked}
    rep_c = {i: _Replay(rows[i], w.r, w.shapes[i][1], w.dtype, W[i]) for i in picked}
    rep_m = {i: _Replay(rows[i], w.r, w.shapes[i][1], w.dtype, W[i]) for i in picked}
    for i in picked:
        rep_m[i].S[:] = M[i].cpu().numpy()[rows[i]]
    G = [wl.gradient(w, i, 0, device=DEV) for i in range(count)]
    acc, mom = fb.FloraSet(G, None, C), fb.FloraSet(None, W, M)
    cur = [G]
    # Algorithm 1's output G~ = (1/tau) C A_acc is Algorithm 2's gradient: M <- beta M + (1-beta)/tau C A_acc A_mom^T,
    # sequenced by the host class that the benchmark uses
    both = hostlogic.AccumulatedMomentum(_Mirror(acc, rep_c, lambda: cur[0]), _Mirror(mom, rep_m, None), count, tau, w.beta, w.kappa, base_seed=5)
    for k in range(tau):
        if k:
            cur[0] = [wl.gradient(w, i, k, device=DEV) for i in range(count)]
            acc.rebind_gradients(cur[0])
        both.accumulate()
    torch.cuda.synchronize()
    for i in picked:
        assert rel_err(C[i].cpu().numpy()[rows[i]], rep_c[i].S) <= TOL[w.dtype], ("accumulated sketch", i)
    both.apply(50.0)
    torch.cuda.synchronize()
    _check(rep_m, M, W, w.dtype, "gpt2_xl_set")
    assert both.micro_step == 0 and both.t == 1      # the cycle ended; the next one's first compression overwrites C
    acc.close()
    mom.close()
