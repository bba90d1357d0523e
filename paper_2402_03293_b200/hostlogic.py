"""Host sequencing of Algorithms 1 and 2: which call happens when, with which seed.

Nothing here computes on matrices; the classes drive an object with the methods of
:class:`paper_2402_03293_b200.binding.FloraSet` and ask the library for seeds
(``flora_derive_seed``) and for the resampling schedule (``flora_resamples_at``).
"""
from __future__ import annotations

from typing import List

from . import binding


def _derived(cache: dict, base_seed: int, count: int, epoch: int):
    """The seeds of one epoch, derived once (they are asked for at every micro-step)."""
    if epoch not in cache:
        if len(cache) > 4:
            cache.clear()
        cache[epoch] = binding.SeedList(binding.flora_derive_seed(base_seed, i, epoch) for i in range(count))
    return cache[epoch]


class AccumulationCycle:
    """Algorithm 1: tau compressions into C with one projection per matrix, then one decompression
    with scale 1/tau; after that C starts from zero again and the projection is resampled (Section 2.4).
    The zeroing is folded into the first compression of the next cycle, which overwrites C instead of adding to it."""

    def __init__(self, ops, count: int, tau: int, base_seed: int = 0):
        if tau < 1:
            raise ValueError("tau must be positive")
        self.ops, self.count, self.tau, self.base_seed = ops, count, tau, base_seed
        self.epoch = 0
        self.micro_step = 0
        self._seeds = {}

    def seeds(self) -> List[int]:
        return _derived(self._seeds, self.base_seed, self.count, self.epoch)

    def accumulate(self, stream=None) -> bool:
        """Compress the gradients currently bound to the set; True when the cycle is full."""
        if self.micro_step >= self.tau:
            raise RuntimeError("cycle is full: call apply() first")
        if self.micro_step == 0:
            self.ops.compress_overwrite(self.seeds(), stream)         # C <- G A^T: stands for "C <- 0" and the first "C += G A^T"
        else:
            self.ops.compress_accumulate(self.seeds(), stream)
        self.micro_step += 1
        return self.micro_step == self.tau

    def apply(self, lr: float, stream=None) -> None:
        """Decompress the mean of the cycle into the weights, then start the next cycle."""
        if self.micro_step != self.tau:
            raise RuntimeError("cycle is not full")
        self.ops.decompress_apply(self.seeds(), lr, 1.0 / self.tau, stream)
        self.epoch += 1
        self.micro_step = 0


class MomentumState:
    """Algorithm 2: at steps t = 0 mod kappa the projection is resampled and M is carried over by
    M <- M A_old A_new^T; then M <- beta M + (1-beta) G A_new^T and the update M A_new is applied."""

    def __init__(self, ops, count: int, beta: float, kappa: int, base_seed: int = 0, skip_transfer_of_zero_state: bool = True,
                 fuse_transfer: bool = True):
        self.ops, self.count, self.beta, self.kappa, self.base_seed = ops, count, beta, kappa, base_seed
        self.t = 0
        self.epoch = 0
        self.skip0 = skip_transfer_of_zero_state
        self.fuse = fuse_transfer                        # transfer and update of a resampling step as one call
        self._seeds = {}

    def seeds(self, epoch: int) -> List[int]:
        return _derived(self._seeds, self.base_seed, self.count, epoch)

    def step(self, lr: float, stream=None) -> None:
        fused = False
        if binding.flora_resamples_at(self.t, self.kappa):
            old, new = self.seeds(self.epoch), self.seeds(self.epoch + 1)
            if not (self.t == 0 and self.skip0):          # M = 0 at t = 0: the transfer of zeros is zeros
                if self.fuse:
                    self.ops.momentum_step_resampled(self.beta, old, new, stream)   # transfer and update in one call
                    fused = True
                else:
                    self.ops.resample_transfer(old, new, stream)
            self.epoch += 1
        cur = self.seeds(self.epoch)
        if not fused:
            self.ops.momentum_step(self.beta, cur, stream)
        self.ops.decompress_apply(cur, lr, 1.0, stream)
        self.t += 1


class AccumulatedMomentum:
    """Algorithm 1 feeding Algorithm 2: tau micro-steps are compressed into C with the accumulation
    projections; at the end of the cycle the mean gradient G~ = C A_acc / tau is Algorithm 2's gradient, so
    M <- beta M + (1-beta)/tau C (A_acc A_mom^T) without ever forming G~, the update M A_mom is applied, C is
    zeroed and the accumulation projections are resampled (Section 2.4).  Every kappa optimizer steps the
    momentum projections are resampled too and M is carried over first (Algorithm 2's resampling branch).

    `acc` holds the gradients and C, `mom` holds the weights and M (objects with the methods of
    :class:`paper_2402_03293_b200.binding.FloraSet`)."""

    def __init__(self, acc, mom, count: int, tau: int, beta: float, kappa: int, base_seed: int = 0):
        if tau < 1:
            raise ValueError("tau must be positive")
        self.acc, self.mom, self.count, self.tau, self.beta, self.kappa = acc, mom, count, tau, beta, kappa
        self.base_seed = base_seed
        self.t = 0                      # optimizer steps done
        self.micro_step = 0
        self.acc_epoch = 0
        self.mom_epoch = 0
        self._acc, self._mom = {}, {}

    def acc_seeds(self) -> List[int]:
        return _derived(self._acc, self.base_seed, self.count, self.acc_epoch)

    def mom_seeds(self, epoch: int) -> List[int]:
        return _derived(self._mom, self.base_seed ^ 0x5DEECE66D, self.count, epoch)

    def accumulate(self, stream=None) -> bool:
        """Compress the gradients currently bound to `acc`; True when the cycle is full."""
        if self.micro_step >= self.tau:
            raise RuntimeError("cycle is full: call apply() first")
        if self.micro_step == 0:
            self.acc.compress_overwrite(self.acc_seeds(), stream)     # C <- G A^T: stands for "C <- 0" and the first "C += G A^T"
        else:
            self.acc.compress_accumulate(self.acc_seeds(), stream)
        self.micro_step += 1
        return self.micro_step == self.tau

    def apply(self, lr: float, stream=None) -> None:
        if self.micro_step != self.tau:
            raise RuntimeError("cycle is not full")
        if binding.flora_resamples_at(self.t, self.kappa):
            if self.t > 0:              # M = 0 at t = 0: nothing to carry over
                self.mom.resample_transfer(self.mom_seeds(self.mom_epoch), self.mom_seeds(self.mom_epoch + 1), stream)
            self.mom_epoch += 1
        cur = self.mom_seeds(self.mom_epoch)
        self.mom.transfer_axpby_from(self.acc, self.acc_seeds(), cur, (1.0 - self.beta) / self.tau, self.beta, stream)
        self.mom.decompress_apply(cur, lr, 1.0, stream)
        self.acc_epoch += 1
        self.micro_step = 0
        self.t += 1
