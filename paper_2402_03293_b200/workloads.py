"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds shapes and input generators only: no projection, no
contraction, nothing of the method's arithmetic.  The same stored bytes are fed
to the CUDA library and to whatever checks it.

The paper applies the projection to the attention and feed-forward weight
matrices of T5 / GPT-2 models (Section 3, "Competing methods") and uses ranks
r in 8..512, tau = 16 accumulation steps and kappa = 1000 (Section 3.1); real
gradients need its datasets and checkpoints, so Gaussian matrices of the same
shapes stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    shapes: Tuple[Tuple[int, int], ...]       # (n, m) per weight matrix
    dtype: str                                # "f32" or "bf16"
    r: int
    grad_var: float                           # gradient entries ~ N(0, grad_var)
    mode: str                                 # "accumulate", "momentum", "accumulate+momentum"
    tau: int = 1
    beta: float = 0.0
    kappa: int = 0
    lr: float = 1e-3
    outlier_frac: float = 0.0                 # Bernoulli mask multiplying entries by outlier_gain
    outlier_gain: float = 1.0
    r_sweep: Tuple[int, ...] = field(default_factory=tuple)

    @property
    def elements(self) -> int:
        return sum(n * m for n, m in self.shapes)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


def _gpt2_block(d: int) -> List[Tuple[int, int]]:
    return [(d, 3 * d), (d, d), (d, 4 * d), (4 * d, d)]


def _t5_large() -> List[Tuple[int, int]]:
    # gated feed-forward with d_ff = 2816: two d_model x d_ff and one d_ff x d_model matrix
    d, ff = 1024, 2816
    ffn = [(d, ff), (d, ff), (ff, d)]
    enc = [(d, d)] * 4 + ffn
    dec = [(d, d)] * 8 + ffn
    return enc * 24 + dec * 24


WORKLOADS = {
    "single_f32_512": Workload("single_f32_512", ((512, 512),), "f32", 8, 1e-2, "accumulate", tau=4, lr=1e-3),
    "gpt2_small_set": Workload("gpt2_small_set", tuple(_gpt2_block(768) * 12), "bf16", 32, 1e-3,
                               "accumulate", tau=8),
    "t5_large_set": Workload("t5_large_set", tuple(_t5_large()), "bf16", 64, 1e-3, "momentum",
                             beta=0.9, kappa=200),
    "single_bf16_4096x11008": Workload("single_bf16_4096x11008", ((4096, 11008),), "bf16", 256, 1e-3,
                                       "momentum", beta=0.9, kappa=1, r_sweep=(8, 32, 128, 256)),
    "gpt2_xl_set": Workload("gpt2_xl_set", tuple(_gpt2_block(1600) * 48), "bf16", 256, 1e-3,
                            "accumulate+momentum", tau=16, beta=0.9, kappa=1000,
                            outlier_frac=0.01, outlier_gain=100.0),
}
CONFIG_ORDER = ["single_f32_512", "gpt2_small_set", "t5_large_set", "single_bf16_4096x11008", "gpt2_xl_set"]


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def gaussian_matrix(n: int, m: int, var: float, dtype: str, seed: int, device: str = "cpu",
                    outlier_frac: float = 0.0, outlier_gain: float = 1.0) -> torch.Tensor:
    """n x m entries ~ N(0, var), optionally with a Bernoulli(outlier_frac) mask of entries
    multiplied by outlier_gain, stored in `dtype`.  Deterministic for (seed, device type)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    x = torch.randn((n, m), generator=gen, device=device, dtype=torch.float32) * (var ** 0.5)
    if outlier_frac > 0.0:
        mask = torch.rand((n, m), generator=gen, device=device) < outlier_frac
        x = torch.where(mask, x * outlier_gain, x)
    return x.to(torch_dtype(dtype)).contiguous()


def gradient(wl: Workload, matrix: int, micro_step: int, device: str = "cpu", base_seed: int = 0) -> torch.Tensor:
    n, m = wl.shapes[matrix]
    seed = base_seed * 1_000_003 + micro_step * 10_007 + matrix
    return gaussian_matrix(n, m, wl.grad_var, wl.dtype, seed, device, wl.outlier_frac, wl.outlier_gain)


def weight(wl: Workload, matrix: int, device: str = "cpu", std: float = 1.0, base_seed: int = 7) -> torch.Tensor:
    n, m = wl.shapes[matrix]
    return gaussian_matrix(n, m, std * std, wl.dtype, 900_001 + base_seed * 1_000_003 + matrix, device)


def as_numpy(t: torch.Tensor):
    """Stored bytes of a CPU/GPU tensor as numpy: float32 as is, bf16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view("uint16")
    return t.numpy()
