"""flora_resample_transfer_static, the entry point for callers that cannot allocate device memory.

Some users of this library run with every byte of device memory already assigned (a fixed memory plan) or
from a place where calling the allocator is not allowed, so the r x r scratch of the momentum transfer cannot
come from cudaMallocAsync there.  The static variant keeps that scratch in a fixed array inside the library.
This file checks, through the C ABI, that it gives the same result as flora_resample_transfer, twice in a
row (the second call finds the array dirty from the first), and that it refuses what does not fit.

The file name sorts last on purpose: a run that stops at the first failure has by then run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2402_03293_b200 import binding as fb
from tests.parity_util import TOL, oracle_transfer, rel_err

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_the_allocating_one_twice_in_a_row():
    dev = "cuda"
    torch.manual_seed(0)
    cases = [(300, 1000, 64, "bf16", 11, 12), (129, 515, 256, "f32", 21, 22)]   # the second leaves a larger, dirty scratch behind
    for rep in range(2):
        for n, m, r, operand, s_old, s_new in cases + cases[:1]:
            M0 = torch.randn(n, r, device=dev)
            ref = M0.clone()
            fb.flora_resample_transfer(ref, m, operand, s_old + rep, s_new + rep)
            got = M0.clone()
            fb.flora_resample_transfer_static(got, m, operand, s_old + rep, s_new + rep)
            torch.cuda.synchronize()
            assert rel_err(got.cpu().numpy(), ref.cpu().numpy()) <= TOL[operand], (rep, n, m, r)
            # and against the CPU oracle, which evaluates (M A_old) A_new^T in the printed order
            want = oracle_transfer(M0, M0, m, operand, s_old + rep, s_new + rep, 1.0, 0.0)
            assert rel_err(got.cpu().numpy(), want) <= TOL[operand], ("oracle", rep, n, m, r)
    assert fb.flora_device_status() == 0


def test_static_scratch_variant_leaves_device_memory_as_it_found_it():
    # a caller whose device memory is fully planned must see the same amount of free memory before and after the
    # call, from the driver's point of view (an allocation that was freed again into a pool would still show here)
    dev = "cuda"
    for n, m, r, operand in [(384, 1024, 128, "bf16"), (200, 300, 48, "f32")]:
        M = torch.randn(n, r, device=dev)
        fb.flora_resample_transfer_static(M, m, operand, 5, 6)      # first use of these kernels: module loading may allocate
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        for k in range(3):
            fb.flora_resample_transfer_static(M, m, operand, 7 + k, 8 + k)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, (operand, free_before, free_after)


def test_static_scratch_variant_rejects_what_does_not_fit():
    dev = "cuda"
    lib = fb.load()
    too_wide = fb.flora_mat(0x1000, 8, 257, 257, fb.FLORA_F32)
    assert lib.flora_resample_transfer_static(ctypes.byref(too_wide), 64, fb.FLORA_F32, 1, 2, None) == 5   # FLORA_ERR_RANK
    M = torch.randn(64, 32, device=dev)
    fb.flora_resample_transfer_static(M, 256, "f32", 1, 2)          # set-up call for this device
    for _ in range(3):
        fb.flora_resample_transfer_static(M, 256, "f32", 3, 4)
    torch.cuda.synchronize()
    assert np.isfinite(M.cpu().numpy()).all()
