"""ctypes front end of the CPU oracle in ``flora_oracle.c``.

TEST INFRASTRUCTURE.  Only the test-suite, the smoke check and the CPU-baseline
timing may import this module; the CUDA library never does, and this module
never touches the CUDA library.  All arithmetic lives in the C file (triple
loops, double accumulation); this file only builds it with gcc, marshals numpy
arrays and names the operations after Algorithms 1 and 2 of the paper.

bf16 matrices travel as ``numpy.uint16`` arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flora_oracle.c")
_LIB = os.path.join(_HERE, "libflora_oracle.so")
F32, BF16 = 0, 1
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no contraction of a*b+c into fma)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               _SRC, "-o", _LIB + ".tmp", "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.flora_oracle_max_threads.restype = ctypes.c_int
        _lib.flora_oracle_transfer_axpby.restype = ctypes.c_int
        _lib.flora_oracle_resample_transfer.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("matrix must be float32, or uint16 holding bf16 bits")


def _check2d(a: np.ndarray, name: str):
    if a.ndim != 2 or a.strides[1] != a.itemsize or a.strides[0] % a.itemsize:
        raise ValueError(f"{name} must be a row-major 2-D array")
    return a.strides[0] // a.itemsize


def set_threads(t: int) -> None:
    lib().flora_oracle_set_threads(ctypes.c_int(t))


def max_threads() -> int:
    return int(lib().flora_oracle_max_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().flora_oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def normal_pair(xa: int, xb: int):
    zc, zs = ctypes.c_float(), ctypes.c_float()
    lib().flora_oracle_normal_pair(ctypes.c_uint32(xa), ctypes.c_uint32(xb),
                                   ctypes.byref(zc), ctypes.byref(zs))
    return zc.value, zs.value


def pair_uniforms(xa: int, xb: int):
    u1, u2 = ctypes.c_double(), ctypes.c_double()
    lib().flora_oracle_pair_uniforms(ctypes.c_uint32(xa), ctypes.c_uint32(xb),
                                     ctypes.byref(u1), ctypes.byref(u2))
    return u1.value, u2.value


def materialize_A(seed: int, r: int, m: int) -> np.ndarray:
    """The explicit r x m fp32 projection A ~ N_seed(0, 1/r)."""
    A = np.zeros((r, m), dtype=np.float32)
    if r and m:
        lib().flora_oracle_materialize_A(ctypes.c_uint64(seed), ctypes.c_int(r),
                                         ctypes.c_int64(m), _p(A), ctypes.c_int64(m))
    return A


def round_to_bf16(x: np.ndarray):
    """(values as float32 on the bf16 grid, raw uint16 bits), round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    vals = np.empty_like(x)
    bits = np.empty(x.shape, dtype=np.uint16)
    lib().flora_oracle_round_to_bf16(_p(x), ctypes.c_int64(x.size), _p(vals), _p(bits))
    return vals, bits


def double_to_bf16_bits(v: float) -> int:
    """One correctly rounded (nearest-even) step from a double to bf16 bits."""
    f = lib().flora_oracle_double_to_bf16
    f.restype = ctypes.c_uint16
    return int(f(ctypes.c_double(v)))


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def projection(seed: int, r: int, m: int, operand: str) -> np.ndarray:
    """A as the contraction sees it: fp32 values, or those values rounded to bf16."""
    A = materialize_A(seed, r, m)
    if operand == "bf16":
        A = round_to_bf16(A)[0]
    elif operand != "f32":
        raise ValueError(operand)
    return A


def compress_accumulate(G: np.ndarray, A: np.ndarray, C: np.ndarray) -> None:
    """Algorithm 1: C <- C + G A^T (in place on C)."""
    n, m = G.shape
    r = A.shape[0]
    assert A.shape == (r, m) and C.shape == (n, r) and C.dtype == np.float32 and A.dtype == np.float32
    lib().flora_oracle_compress_accumulate(
        _p(G), ctypes.c_int(_dtype_code(G)), ctypes.c_int64(n), ctypes.c_int64(m),
        ctypes.c_int64(_check2d(G, "G")), _p(A), ctypes.c_int(r), ctypes.c_int64(_check2d(A, "A")),
        _p(C), ctypes.c_int64(_check2d(C, "C")))


def momentum_step(G: np.ndarray, A: np.ndarray, beta: float, M: np.ndarray) -> None:
    """Algorithm 2: M <- beta M + (1 - beta) G A^T (in place on M)."""
    n, m = G.shape
    r = A.shape[0]
    assert A.shape == (r, m) and M.shape == (n, r) and M.dtype == np.float32 and A.dtype == np.float32
    lib().flora_oracle_momentum_step(
        _p(G), ctypes.c_int(_dtype_code(G)), ctypes.c_int64(n), ctypes.c_int64(m),
        ctypes.c_int64(_check2d(G, "G")), _p(A), ctypes.c_int(r), ctypes.c_int64(_check2d(A, "A")),
        ctypes.c_float(beta), _p(M), ctypes.c_int64(_check2d(M, "M")))


def decompress_apply(W: np.ndarray, C: np.ndarray, A: np.ndarray, lr: float, scale: float) -> None:
    """Algorithm 1 reconstruction used as an update: W <- W - lr*scale*(C A) (in place on W)."""
    n, m = W.shape
    r = A.shape[0]
    assert A.shape == (r, m) and C.shape == (n, r) and C.dtype == np.float32 and A.dtype == np.float32
    lib().flora_oracle_decompress_apply(
        _p(W), ctypes.c_int(_dtype_code(W)), ctypes.c_int64(n), ctypes.c_int64(m),
        ctypes.c_int64(_check2d(W, "W")), _p(C), ctypes.c_int(r), ctypes.c_int64(_check2d(C, "C")),
        _p(A), ctypes.c_int64(_check2d(A, "A")), ctypes.c_float(lr), ctypes.c_float(scale))


def resample_transfer(M: np.ndarray, A_old: np.ndarray, A_new: np.ndarray) -> None:
    """Algorithm 2: M <- (M A_old) A_new^T, evaluated in that order (in place on M)."""
    n, r = M.shape
    m = A_old.shape[1]
    assert A_old.shape == (r, m) and A_new.shape == (r, m) and M.dtype == np.float32
    rc = lib().flora_oracle_resample_transfer(
        _p(M), ctypes.c_int64(_check2d(M, "M")), ctypes.c_int64(n), ctypes.c_int(r), ctypes.c_int64(m),
        _p(A_old), ctypes.c_int64(_check2d(A_old, "A_old")), _p(A_new), ctypes.c_int64(_check2d(A_new, "A_new")))
    if rc:
        raise MemoryError("oracle transfer")


def momentum_step_resampled(G: np.ndarray, A_old: np.ndarray, A_new: np.ndarray, beta: float, M: np.ndarray) -> None:
    """Algorithm 2 at a resampling step, in the paper's order: first M <- (M A_old) A_new^T, then
    M <- beta M + (1 - beta) G A_new^T (in place on M)."""
    resample_transfer(M, A_old, A_new)
    momentum_step(G, A_new, beta, M)


def transfer_axpby(dst: np.ndarray, src: np.ndarray, A_old: np.ndarray, A_new: np.ndarray,
                   a: float, b: float) -> None:
    """dst <- b dst + a (src A_old) A_new^T: Algorithm 1's output fed to Algorithm 2's update."""
    n, r = src.shape
    m = A_old.shape[1]
    assert dst.shape == (n, r) and A_old.shape == (r, m) and A_new.shape == (r, m)
    assert dst.dtype == np.float32 and src.dtype == np.float32
    rc = lib().flora_oracle_transfer_axpby(
        _p(dst), ctypes.c_int64(_check2d(dst, "dst")), _p(src), ctypes.c_int64(_check2d(src, "src")),
        ctypes.c_int64(n), ctypes.c_int(r), ctypes.c_int64(m),
        _p(A_old), ctypes.c_int64(_check2d(A_old, "A_old")), _p(A_new), ctypes.c_int64(_check2d(A_new, "A_new")),
        ctypes.c_double(a), ctypes.c_double(b))
    if rc:
        raise MemoryError("oracle transfer")
