"""Shared helpers of the GPU parity tests: run the oracle on the stored bytes of torch tensors."""
import numpy as np
import torch

from oracle import flora_oracle as orc
from paper_2402_03293_b200 import workloads as wl

TOL = {"f32": 1e-5, "bf16": 2e-2}     # max |x - ref| / max |ref| per output tensor


def operand_of(t: torch.Tensor) -> str:
    return "bf16" if t.dtype == torch.bfloat16 else "f32"


def rel_err(x: np.ndarray, ref: np.ndarray) -> float:
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    denom = np.abs(ref).max() if ref.size else 0.0
    if denom == 0.0:
        return float(np.abs(x).max()) if x.size else 0.0
    return float(np.abs(x - ref).max() / denom)


def values(a: np.ndarray) -> np.ndarray:
    return orc.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a


def oracle_compress(G: torch.Tensor, S0: torch.Tensor, seed: int, a: float = 1.0, b: float = 1.0, rows=None):
    """b*S0 + a*G A^T on the CPU oracle (a=b=1: Algorithm 1; a=1-beta, b=beta: Algorithm 2)."""
    Gn, Sn = wl.as_numpy(G), wl.as_numpy(S0).copy()
    if rows is not None:
        Gn, Sn = np.ascontiguousarray(Gn[rows]), np.ascontiguousarray(Sn[rows])
    A = orc.projection(seed, Sn.shape[1], Gn.shape[1], operand_of(G))
    if a == 1.0 and b == 1.0:
        orc.compress_accumulate(Gn, A, Sn)
    else:
        assert abs((1.0 - b) - a) < 1e-6
        orc.momentum_step(Gn, A, b, Sn)
    return Sn


def oracle_decompress(W0: torch.Tensor, C: torch.Tensor, seed: int, lr: float, scale: float, rows=None):
    Wn, Cn = wl.as_numpy(W0).copy(), wl.as_numpy(C)
    if rows is not None:
        Wn, Cn = np.ascontiguousarray(Wn[rows]), np.ascontiguousarray(Cn[rows])
    A = orc.projection(seed, Cn.shape[1], Wn.shape[1], operand_of(W0))
    orc.decompress_apply(Wn, Cn, A, lr, scale)
    return Wn


def oracle_transfer(dst0: torch.Tensor, src: torch.Tensor, m: int, operand: str, s_old: int, s_new: int, a: float, b: float):
    d, s = wl.as_numpy(dst0).copy(), wl.as_numpy(src)
    r = d.shape[1]
    orc.transfer_axpby(d, s, orc.projection(s_old, r, m, operand), orc.projection(s_new, r, m, operand), a, b)
    return d


def sample_rows(n: int, count: int, seed: int) -> np.ndarray:
    if n <= count:
        return np.arange(n)
    rng = np.random.default_rng(seed)
    picks = set(rng.choice(n, size=count - 3, replace=False).tolist()) | {0, n - 1, n // 2}
    return np.array(sorted(picks))
