"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, rejects bad
arguments before touching a device, and the host sequencing follows Algorithms 1 and 2."""
import ctypes
import os
import re

import pytest

from paper_2402_03293_b200 import binding as fb
from paper_2402_03293_b200 import hostlogic

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "flora.h")).read()
    declared = set(re.findall(r"\b(flora_[a-zA-Z_0-9]+)\s*\(", header))
    assert declared == set(fb.EXPORTS)
    lib = fb.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert fb.flora_version() >= 100


def _m(rows, cols, ld=None, dtype=fb.FLORA_F32, data=0x1000):
    return fb.flora_mat(data, rows, cols, cols if ld is None else ld, dtype)


def _st(name):
    return {v: k for k, v in fb.STATUS_NAMES.items()}[name]


def test_argument_validation_happens_before_any_launch():
    lib = fb.load()
    G, C = _m(8, 16), _m(8, 4)
    by = ctypes.byref
    assert lib.flora_compress_accumulate(None, by(C), 1, 4, None) == _st("FLORA_ERR_NULL")
    assert lib.flora_compress_accumulate(by(G), by(C), 1, 5, None) == _st("FLORA_ERR_RANK")
    assert lib.flora_compress_accumulate(by(G), by(_m(8, 0)), 1, 0, None) == _st("FLORA_ERR_RANK")
    assert lib.flora_compress_accumulate(by(G), by(_m(8, 300)), 1, 300, None) == _st("FLORA_ERR_RANK")
    assert lib.flora_compress_accumulate(by(G), by(_m(7, 4)), 1, 4, None) == _st("FLORA_ERR_SHAPE")
    assert lib.flora_compress_accumulate(by(_m(8, 16, ld=15)), by(C), 1, 4, None) == _st("FLORA_ERR_SHAPE")
    assert lib.flora_compress_accumulate(by(_m(-1, 16)), by(C), 1, 4, None) == _st("FLORA_ERR_SHAPE")
    assert lib.flora_compress_accumulate(by(_m(8, 16, dtype=7)), by(C), 1, 4, None) == _st("FLORA_ERR_DTYPE")
    assert lib.flora_compress_accumulate(by(G), by(_m(8, 4, dtype=fb.FLORA_BF16)), 1, 4, None) == _st("FLORA_ERR_DTYPE")
    assert lib.flora_compress_accumulate(by(_m(8, 16, data=0x1002)), by(C), 1, 4, None) == _st("FLORA_ERR_ALIGN")
    assert lib.flora_compress_accumulate(by(_m(8, 16, data=None)), by(C), 1, 4, None) == _st("FLORA_ERR_NULL")
    assert lib.flora_momentum_step(by(G), by(_m(9, 4)), 0.9, 1, None) == _st("FLORA_ERR_SHAPE")
    assert lib.flora_decompress_apply(by(G), by(_m(8, 257)), 1, 0.1, 1.0, None) == _st("FLORA_ERR_RANK")
    assert lib.flora_resample_transfer(by(C), -5, fb.FLORA_F32, 1, 2, None) == _st("FLORA_ERR_SHAPE")
    assert lib.flora_resample_transfer(by(C), 16, 9, 1, 2, None) == _st("FLORA_ERR_DTYPE")
    assert lib.flora_transfer_axpby(by(C), by(_m(8, 5)), 16, fb.FLORA_F32, 1, 2, 1.0, 0.0, None) == _st("FLORA_ERR_RANK")
    assert lib.flora_materialize_A(by(_m(300, 16)), 1, None) == _st("FLORA_ERR_RANK")
    # empty problems are accepted and launch nothing
    before = fb.flora_launch_count()
    assert lib.flora_compress_accumulate(by(_m(0, 16, data=None)), by(_m(0, 4, data=None)), 1, 4, None) == 0
    assert lib.flora_compress_accumulate(by(_m(8, 0, data=None)), by(C), 1, 4, None) == 0
    assert lib.flora_decompress_apply(by(_m(8, 0, data=None)), by(C), 1, 0.1, 1.0, None) == 0
    assert fb.flora_launch_count() == before
    handle = ctypes.c_void_p()
    arrG = (fb.flora_mat * 2)(_m(8, 16), _m(8, 16))
    arrS = (fb.flora_mat * 2)(_m(8, 4), _m(8, 5))
    assert lib.flora_set_create(2, arrG, None, arrS, by(handle)) == _st("FLORA_ERR_RANK")
    assert lib.flora_set_create(2, None, None, arrS, by(handle)) == _st("FLORA_ERR_NULL")
    for s in range(10):
        assert fb.status_string(s) != "unknown status"


def test_seed_derivation_is_a_64_bit_mix():
    seen = set()
    for base in (0, 1, 2 ** 63):
        for mtx in range(20):
            for epoch in range(20):
                seen.add(fb.flora_derive_seed(base, mtx, epoch))
    assert len(seen) == 3 * 20 * 20
    assert all(0 <= s < 2 ** 64 for s in seen)
    # high and low halves (the two Philox key words) both vary
    assert len({s >> 32 for s in seen}) > 1190 and len({s & 0xFFFFFFFF for s in seen}) > 1190
    assert fb.flora_derive_seed(5, 6, 7) == fb.flora_derive_seed(5, 6, 7)


def test_resampling_schedule():
    assert [t for t in range(10) if fb.flora_resamples_at(t, 4)] == [0, 4, 8]
    assert [t for t in range(4) if fb.flora_resamples_at(t, 1)] == [0, 1, 2, 3]
    assert not any(fb.flora_resamples_at(t, 0) for t in range(5))


class _Recorder:
    def __init__(self):
        self.calls = []

    def __getattr__(self, name):
        def f(*args):
            self.calls.append((name,) + tuple(a for a in args if a is not None))
        return f


def test_accumulation_cycle_order_algorithm_1():
    ops = _Recorder()
    cyc = hostlogic.AccumulationCycle(ops, count=3, tau=4, base_seed=11)
    s0 = cyc.seeds()
    for i in range(4):
        full = cyc.accumulate()
        assert full == (i == 3)
    with pytest.raises(RuntimeError):
        cyc.accumulate()
    cyc.apply(0.5)
    # the first compression of a cycle overwrites C (zeroing folded into it), the others add
    assert [c[0] for c in ops.calls] == ["compress_overwrite"] + ["compress_accumulate"] * 3 + ["decompress_apply"]
    assert all(c[1] == s0 for c in ops.calls[:5])                 # one projection for the whole cycle
    assert ops.calls[4][2:] == (0.5, 0.25)                        # arithmetic mean over tau steps
    s1 = cyc.seeds()
    assert s1 != s0 and len(set(s0 + s1)) == 6                    # resampled once the cycle ends
    with pytest.raises(RuntimeError):
        cyc.apply(0.5)


def test_momentum_order_algorithm_2():
    ops = _Recorder()
    mom = hostlogic.MomentumState(ops, count=2, beta=0.9, kappa=3, base_seed=5, fuse_transfer=False)
    for _ in range(7):
        mom.step(0.1)
    names = [c[0] for c in ops.calls]
    # t = 0: resample (transfer of the zero state skipped); t = 3, 6: transfer old -> new, then update and yield with new
    assert names == ["momentum_step", "decompress_apply"] * 3 + \
        ["resample_transfer", "momentum_step", "decompress_apply"] + ["momentum_step", "decompress_apply"] * 2 + \
        ["resample_transfer", "momentum_step", "decompress_apply"]
    tr = ops.calls[6]
    assert tr[1] == ops.calls[4][2] and tr[2] == ops.calls[7][2] == ops.calls[8][1]
    assert ops.calls[0][1] == 0.9 and ops.calls[1][2:] == (0.1, 1.0)
    ops2 = _Recorder()
    mom2 = hostlogic.MomentumState(ops2, count=1, beta=0.5, kappa=1, skip_transfer_of_zero_state=False, fuse_transfer=False)
    mom2.step(1.0)
    assert [c[0] for c in ops2.calls] == ["resample_transfer", "momentum_step", "decompress_apply"]
    # by default a resampling step is one call that carries both seed lists
    ops3 = _Recorder()
    mom3 = hostlogic.MomentumState(ops3, count=2, beta=0.9, kappa=3, base_seed=5)
    for _ in range(4):
        mom3.step(0.1)
    assert [c[0] for c in ops3.calls] == ["momentum_step", "decompress_apply"] * 3 + ["momentum_step_resampled", "decompress_apply"]
    fused = ops3.calls[6]
    assert fused[1] == 0.9 and fused[2] == ops3.calls[4][2] and fused[3] == ops3.calls[7][1]


def test_accumulation_feeding_momentum_order():
    acc, mom = _Recorder(), _Recorder()
    both = hostlogic.AccumulatedMomentum(acc, mom, count=2, tau=3, beta=0.75, kappa=2, base_seed=9)
    for step in range(3):
        s_acc = both.acc_seeds()
        for k in range(3):
            assert both.accumulate() == (k == 2)
        with pytest.raises(RuntimeError):
            both.accumulate()
        both.apply(0.5)
        assert both.acc_seeds() != s_acc                           # a fresh accumulation projection per cycle
    assert [c[0] for c in acc.calls] == (["compress_overwrite"] + ["compress_accumulate"] * 2) * 3
    names = [c[0] for c in mom.calls]
    # t = 0 resamples (nothing to carry), t = 1 keeps the projection, t = 2 resamples and carries M over first
    assert names == ["transfer_axpby_from", "decompress_apply"] * 2 + ["resample_transfer", "transfer_axpby_from", "decompress_apply"]
    ax0, ax1, tr, ax2 = mom.calls[0], mom.calls[2], mom.calls[4], mom.calls[5]
    assert ax0[1] is acc and ax0[2] == acc.calls[0][1]             # the sketches of `acc` with the cycle's accumulation seeds
    assert ax0[4:6] == (0.25 / 3, 0.75)                            # (1 - beta) / tau and beta
    assert ax0[3] == ax1[3] == mom.calls[1][1] == tr[1]            # one momentum projection until it is resampled
    assert tr[2] == ax2[3] == mom.calls[6][1] and tr[2] != tr[1]
    assert mom.calls[1][2:] == (0.5, 1.0)
    with pytest.raises(RuntimeError):
        both.apply(0.5)
