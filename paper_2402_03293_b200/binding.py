"""ctypes binding of libflora.so: same names as include/flora.h, argument marshalling only.

Every operation runs in the CUDA library; there is no fallback.  If the library has not been
built (``python -c "import __graft_entry__ as g; g.build()"`` or
``python paper_2402_03293_b200/_build.py``) loading it raises.  PyTorch is used here for device
memory (tensors) and streams only.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libflora.so")

FLORA_OK = 0
STATUS_NAMES = {0: "FLORA_OK", 1: "FLORA_ERR_NULL", 2: "FLORA_ERR_SHAPE", 3: "FLORA_ERR_DTYPE", 4: "FLORA_ERR_ALIGN",
                5: "FLORA_ERR_RANK", 6: "FLORA_ERR_CUDA", 7: "FLORA_ERR_TIMEOUT", 8: "FLORA_ERR_UNSUPPORTED",
                9: "FLORA_ERR_ALLOC"}
FLORA_F32, FLORA_BF16 = 0, 1

# every symbol include/flora.h declares
EXPORTS = [
    "flora_compress_accumulate", "flora_decompress_apply", "flora_momentum_step", "flora_momentum_step_resampled", "flora_resample_transfer",
    "flora_resample_transfer_static", "flora_transfer_axpby", "flora_materialize_A", "flora_set_create", "flora_set_destroy",
    "flora_set_rebind_gradients", "flora_set_compress_accumulate", "flora_set_momentum_step",
    "flora_set_decompress_apply", "flora_set_resample_transfer", "flora_set_transfer_axpby", "flora_set_momentum_step_resampled", "flora_set_zero_state", "flora_derive_seed",
    "flora_resamples_at", "flora_set_upload_gradients", "flora_set_compress_accumulate_from_host", "flora_set_read_weights_to_host",
    "flora_debug_force_path", "flora_set_deterministic", "flora_debug_plan", "flora_debug_wait_timeout_selftest", "flora_launch_count", "flora_device_status", "flora_status_string", "flora_version",
]


class FloraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({status_string(status)})")


class flora_mat(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("ld", ctypes.c_int64), ("dtype", ctypes.c_int32)]


_lib: Optional[ctypes.CDLL] = None


def load() -> ctypes.CDLL:
    """Load libflora.so; raises if it was not built (there is no other implementation to fall back to)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build the CUDA library first (__graft_entry__.build())")
        lib = ctypes.CDLL(LIB_PATH)
        P, U64, I64, I32, F = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
        MP = ctypes.POINTER(flora_mat)
        sig = {
            "flora_compress_accumulate": (I32, [MP, MP, U64, ctypes.c_int, P]),
            "flora_decompress_apply": (I32, [MP, MP, U64, F, F, P]),
            "flora_momentum_step": (I32, [MP, MP, F, U64, P]),
            "flora_resample_transfer": (I32, [MP, I64, I32, U64, U64, P]),
            "flora_momentum_step_resampled": (I32, [MP, MP, F, U64, U64, P]),
            "flora_resample_transfer_static": (I32, [MP, I64, I32, U64, U64, P]),
            "flora_transfer_axpby": (I32, [MP, MP, I64, I32, U64, U64, F, F, P]),
            "flora_materialize_A": (I32, [MP, U64, P]),
            "flora_set_create": (I32, [ctypes.c_int, MP, MP, MP, ctypes.POINTER(P)]),
            "flora_set_destroy": (I32, [P]),
            "flora_set_rebind_gradients": (I32, [P, MP, P]),
            "flora_set_compress_accumulate": (I32, [P, ctypes.POINTER(U64), P]),
            "flora_set_momentum_step": (I32, [P, F, ctypes.POINTER(U64), P]),
            "flora_set_decompress_apply": (I32, [P, ctypes.POINTER(U64), F, F, P]),
            "flora_set_resample_transfer": (I32, [P, ctypes.POINTER(U64), ctypes.POINTER(U64), P]),
            "flora_set_momentum_step_resampled": (I32, [P, F, ctypes.POINTER(U64), ctypes.POINTER(U64), P]),
            "flora_set_transfer_axpby": (I32, [P, P, ctypes.POINTER(U64), ctypes.POINTER(U64), F, F, P]),
            "flora_set_zero_state": (I32, [P, P]),
            "flora_derive_seed": (U64, [U64, U64, U64]),
            "flora_resamples_at": (ctypes.c_int, [I64, I64]),
            "flora_set_compress_accumulate_from_host": (I32, [P, ctypes.POINTER(P), ctypes.POINTER(U64), P]),
            "flora_set_read_weights_to_host": (I32, [P, ctypes.POINTER(P), P]),
            "flora_set_upload_gradients": (I32, [P, ctypes.POINTER(P), P]),
            "flora_debug_force_path": (None, [ctypes.c_int]),
            "flora_set_deterministic": (None, [ctypes.c_int]),
            "flora_debug_plan": (I32, [P, P, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, P, ctypes.c_int64, P, P]),
            "flora_debug_wait_timeout_selftest": (I32, [P]),
            "flora_launch_count": (U64, []),
            "flora_device_status": (I32, []),
            "flora_status_string": (ctypes.c_char_p, [I32]),
            "flora_version": (ctypes.c_int, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().flora_status_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != FLORA_OK:
        raise FloraError(status, where)


def mat(t: torch.Tensor) -> flora_mat:
    """A borrowed row-major view of a 2-D CUDA tensor (float32 or bfloat16)."""
    if t.dim() != 2:
        raise ValueError("expected a 2-D tensor")
    if t.numel() and t.stride(1) != 1:
        raise ValueError("expected unit stride along columns")
    if t.dtype == torch.float32:
        dt = FLORA_F32
    elif t.dtype == torch.bfloat16:
        dt = FLORA_BF16
    else:
        raise ValueError("expected float32 or bfloat16")
    if t.numel() and not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    ld = t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0) if t.numel() else 0)
    return flora_mat(t.data_ptr() if t.numel() else None, t.shape[0], t.shape[1], max(ld, t.shape[1]), dt)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _dt(dtype) -> int:
    if isinstance(dtype, int) and dtype in (FLORA_F32, FLORA_BF16):
        return dtype
    if dtype in (torch.float32, "f32"):
        return FLORA_F32
    if dtype in (torch.bfloat16, "bf16"):
        return FLORA_BF16
    raise ValueError(dtype)


# ---------------------------------------------------------------------------------- single-matrix calls
def flora_compress_accumulate(G: torch.Tensor, C: torch.Tensor, seed: int, r: int, stream=None) -> None:
    g, c = mat(G), mat(C)
    _check(load().flora_compress_accumulate(ctypes.byref(g), ctypes.byref(c), seed, r, _stream(stream)),
           "flora_compress_accumulate")


def flora_decompress_apply(W: torch.Tensor, C: torch.Tensor, seed: int, lr: float, scale: float, stream=None) -> None:
    w, c = mat(W), mat(C)
    _check(load().flora_decompress_apply(ctypes.byref(w), ctypes.byref(c), seed, lr, scale, _stream(stream)),
           "flora_decompress_apply")


def flora_momentum_step(G: torch.Tensor, M: torch.Tensor, beta: float, seed: int, stream=None) -> None:
    g, m_ = mat(G), mat(M)
    _check(load().flora_momentum_step(ctypes.byref(g), ctypes.byref(m_), beta, seed, _stream(stream)),
           "flora_momentum_step")


def flora_momentum_step_resampled(G: torch.Tensor, M: torch.Tensor, beta: float, seed_old: int, seed_new: int, stream=None) -> None:
    g, m_ = mat(G), mat(M)
    _check(load().flora_momentum_step_resampled(ctypes.byref(g), ctypes.byref(m_), beta, seed_old, seed_new, _stream(stream)),
           "flora_momentum_step_resampled")


def flora_resample_transfer(M: torch.Tensor, m: int, operand, seed_old: int, seed_new: int, stream=None) -> None:
    m_ = mat(M)
    _check(load().flora_resample_transfer(ctypes.byref(m_), m, _dt(operand), seed_old, seed_new, _stream(stream)),
           "flora_resample_transfer")


def flora_resample_transfer_static(M: torch.Tensor, m: int, operand, seed_old: int, seed_new: int, stream=None) -> None:
    """flora_resample_transfer without any allocation: the r x r scratch is a fixed 256 KB array inside the
    library (r <= 256).  Calls that can overlap on one GPU must be serialised by the caller."""
    m_ = mat(M)
    _check(load().flora_resample_transfer_static(ctypes.byref(m_), m, _dt(operand), seed_old, seed_new, _stream(stream)),
           "flora_resample_transfer_static")


def flora_transfer_axpby(dst: torch.Tensor, src: torch.Tensor, m: int, operand, seed_old: int, seed_new: int,
                         a: float, b: float, stream=None) -> None:
    d, s = mat(dst), mat(src)
    _check(load().flora_transfer_axpby(ctypes.byref(d), ctypes.byref(s), m, _dt(operand), seed_old, seed_new, a, b,
                                       _stream(stream)), "flora_transfer_axpby")


def flora_materialize_A(out: torch.Tensor, seed: int, stream=None) -> None:
    o = mat(out)
    _check(load().flora_materialize_A(ctypes.byref(o), seed, _stream(stream)), "flora_materialize_A")


# ---------------------------------------------------------------------------------- host helpers
def flora_derive_seed(base: int, matrix: int, epoch: int) -> int:
    return int(load().flora_derive_seed(base, matrix, epoch))


def flora_resamples_at(t: int, kappa: int) -> bool:
    return bool(load().flora_resamples_at(t, kappa))


def flora_debug_force_path(path: int) -> None:
    load().flora_debug_force_path(path)


def flora_set_deterministic(on: bool) -> None:
    load().flora_set_deterministic(1 if on else 0)


def flora_debug_plan(shapes, r: int, which: str):
    """Work items and launch parameters the library would use for bf16 matrices of these (rows, cols) shapes.

    which = "compress", "decompress" or "compress_slots" (the per-cluster unit lists of the persistent compression
    kernel that serves ranks above 64).  Returns (items, params): items as a list of tuples, params as a tuple of
    eight ints (see include/flora.h).  No kernel runs; usable without a GPU."""
    count = len(shapes)
    rows = (ctypes.c_int64 * max(count, 1))(*[int(n) for n, _ in shapes])
    cols = (ctypes.c_int64 * max(count, 1))(*[int(m) for _, m in shapes])
    w = {"compress": 0, "decompress": 1, "compress_slots": 2}[which]
    width = {0: 6, 1: 4, 2: 1}[w]
    n = ctypes.c_int64(0)
    params = (ctypes.c_int32 * 8)()
    _check(load().flora_debug_plan(rows, cols, count, r, w, None, 0, ctypes.byref(n), params), "flora_debug_plan")
    buf = (ctypes.c_int32 * max(1, n.value * width))()
    _check(load().flora_debug_plan(rows, cols, count, r, w, buf, n.value, ctypes.byref(n), params), "flora_debug_plan")
    items = [tuple(buf[i * width + j] for j in range(width)) for i in range(n.value)]
    return items, tuple(params)


def flora_debug_wait_timeout_selftest(stream=None) -> int:
    """Status of the bounded-wait self-test: FLORA_ERR_TIMEOUT (7) when the wait gave up as designed."""
    return int(load().flora_debug_wait_timeout_selftest(_stream(stream)))


def flora_launch_count() -> int:
    return int(load().flora_launch_count())


def flora_device_status() -> int:
    return int(load().flora_device_status())


def flora_version() -> int:
    return int(load().flora_version())


# ---------------------------------------------------------------------------------- weight sets
def _mat_array(ts: Optional[Sequence[torch.Tensor]]):
    if ts is None:
        return None
    arr = (flora_mat * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = mat(t)
    return arr


class SeedList(list):
    """A list of seeds that remembers its marshalled form, so that handing the same list to many calls costs nothing."""
    _marshalled = None


def _u64_array(vals):
    """Host array of 64-bit seeds; an array made by an earlier call is passed through unchanged."""
    if isinstance(vals, ctypes.Array):
        return vals
    if isinstance(vals, SeedList):
        if vals._marshalled is None or len(vals._marshalled) != len(vals):
            vals._marshalled = (ctypes.c_uint64 * len(vals))(*[int(v) & 0xFFFFFFFFFFFFFFFF for v in vals])
        return vals._marshalled
    return (ctypes.c_uint64 * len(vals))(*[int(v) & 0xFFFFFFFFFFFFFFFF for v in vals])


def seed_array(vals: Sequence[int]):
    """Marshal a list of seeds once, for reuse over several calls (the set calls accept the result)."""
    return _u64_array(vals)


class FloraSet:
    """flora_set_*: one launch per operation over all matrices of a model.

    Keeps the tensors alive for as long as the set exists (the library keeps their pointers)."""

    def __init__(self, G: Optional[List[torch.Tensor]], W: Optional[List[torch.Tensor]], S: List[torch.Tensor]):
        self.G, self.W, self.S = G, W, S
        self.count = len(S)
        handle = ctypes.c_void_p()
        _check(load().flora_set_create(self.count, _mat_array(G), _mat_array(W), _mat_array(S), ctypes.byref(handle)),
               "flora_set_create")
        self._h = handle

    def close(self) -> None:
        if self._h:
            load().flora_set_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def rebind_gradients(self, G: List[torch.Tensor], stream=None) -> None:
        _check(load().flora_set_rebind_gradients(self._h, _mat_array(G), _stream(stream)), "flora_set_rebind_gradients")
        self.G = G

    def compress_accumulate(self, seeds: Sequence[int], stream=None) -> None:
        _check(load().flora_set_compress_accumulate(self._h, _u64_array(seeds), _stream(stream)),
               "flora_set_compress_accumulate")

    def momentum_step(self, beta: float, seeds: Sequence[int], stream=None) -> None:
        _check(load().flora_set_momentum_step(self._h, beta, _u64_array(seeds), _stream(stream)),
               "flora_set_momentum_step")

    def compress_overwrite(self, seeds: Sequence[int], stream=None) -> None:
        """C <- G A^T: the first compression of an accumulation cycle, which makes zeroing C beforehand unnecessary
        (flora_set_momentum_step with beta = 0: the old sketch is neither read nor blended in)."""
        _check(load().flora_set_momentum_step(self._h, 0.0, _u64_array(seeds), _stream(stream)),
               "flora_set_momentum_step")

    def decompress_apply(self, seeds: Sequence[int], lr: float, scale: float, stream=None) -> None:
        _check(load().flora_set_decompress_apply(self._h, _u64_array(seeds), lr, scale, _stream(stream)),
               "flora_set_decompress_apply")

    def resample_transfer(self, seeds_old: Sequence[int], seeds_new: Sequence[int], stream=None) -> None:
        _check(load().flora_set_resample_transfer(self._h, _u64_array(seeds_old), _u64_array(seeds_new),
                                                  _stream(stream)), "flora_set_resample_transfer")

    def transfer_axpby_from(self, src: "FloraSet", seeds_old: Sequence[int], seeds_new: Sequence[int], a: float, b: float, stream=None) -> None:
        """self.S[i] <- b self.S[i] + a src.S[i] A(seeds_old[i]) A(seeds_new[i])^T for every matrix."""
        _check(load().flora_set_transfer_axpby(self._h, src._h, _u64_array(seeds_old), _u64_array(seeds_new), a, b, _stream(stream)),
               "flora_set_transfer_axpby")

    def momentum_step_resampled(self, beta: float, seeds_old: Sequence[int], seeds_new: Sequence[int], stream=None) -> None:
        _check(load().flora_set_momentum_step_resampled(self._h, beta, _u64_array(seeds_old), _u64_array(seeds_new),
                                                        _stream(stream)), "flora_set_momentum_step_resampled")

    def zero_state(self, stream=None) -> None:
        _check(load().flora_set_zero_state(self._h, _stream(stream)), "flora_set_zero_state")

    def upload_gradients(self, host_G: Sequence[torch.Tensor], stream=None) -> None:
        ptrs = (ctypes.c_void_p * self.count)(*[t.data_ptr() for t in host_G])
        _check(load().flora_set_upload_gradients(self._h, ptrs, _stream(stream)), "flora_set_upload_gradients")

    def compress_accumulate_from_host(self, host_G: Sequence[torch.Tensor], seeds: Sequence[int], stream=None) -> None:
        ptrs = (ctypes.c_void_p * self.count)(*[t.data_ptr() for t in host_G])
        _check(load().flora_set_compress_accumulate_from_host(self._h, ptrs, _u64_array(seeds), _stream(stream)),
               "flora_set_compress_accumulate_from_host")

    def read_weights_to_host(self, host_W: Sequence[torch.Tensor], stream=None) -> None:
        ptrs = (ctypes.c_void_p * self.count)(*[t.data_ptr() for t in host_W])
        _check(load().flora_set_read_weights_to_host(self._h, ptrs, _stream(stream)), "flora_set_read_weights_to_host")
