"""Thin ctypes binding over the C ABI in ``include/pop.h`` (same names, argument
marshalling only: every step of the path runs in the library's CUDA kernels).

PyTorch is used for device memory and streams.  There is no CPU fallback: if
``libpop.so`` has not been built, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Tuple

import numpy as np

POP_OK = 0
POP_ERR_INVALID_ARG = -1
POP_ERR_UNSUPPORTED = -2
POP_ERR_ALLOC = -3
POP_ERR_CUDA = -4
POP_ERR_TIMEOUT = -5
POP_MAX_BATCH = 8
POP_F32, POP_BF16 = 0, 1
POP_NOALLOC_MAX_N = 32768

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libpop.so")


class Ratios(C.Structure):
    _fields_ = [("retained", C.c_double), ("candidate", C.c_double), ("pruned", C.c_double)]


class Config(C.Structure):
    _fields_ = [("decode_kernel", C.c_int), ("launch_mode", C.c_int), ("wait_budget_us", C.c_uint),
                ("slab_cache_bytes", C.c_ulonglong)]


POP_DECODE_AUTO, POP_DECODE_FUSED, POP_DECODE_SIMPLE = 0, 1, 2
POP_LAUNCH_PDL, POP_LAUNCH_COOPERATIVE, POP_LAUNCH_PLAIN = 0, 1, 2


class PopError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = f"{where}: {status_string(status)}"
        if status in (POP_ERR_CUDA, POP_ERR_ALLOC, POP_ERR_TIMEOUT):
            msg += f" [{lib().pop_last_cuda_error().decode()}]"
        super().__init__(msg)


_lib = None

# name -> (restype, argtypes); mirrors include/pop.h
_P = C.c_void_p
SIGNATURES = {
    "pop_version": (C.c_char_p, []),
    "pop_status_string": (C.c_char_p, [C.c_int]),
    "pop_last_cuda_error": (C.c_char_p, []),
    "pop_kernel_launch_count": (C.c_ulonglong, []),
    "pop_get_config": (C.c_int, [C.POINTER(Config)]),
    "pop_set_config": (C.c_int, [C.POINTER(Config)]),
    "pop_release_cached_memory": (C.c_int, []),
    "pop_region_sizes": (C.c_int, [C.c_int, Ratios] + [C.POINTER(C.c_int)] * 4),
    "pop_prefill_partition": (C.c_int, [_P, C.c_int, C.c_int, _P, _P, _P, C.c_int, C.c_int, Ratios, _P,
                                        C.POINTER(_P)]),
    "pop_weights_prepare": (C.c_int, [_P, _P, _P, C.c_int, C.c_int, C.c_int, _P, C.POINTER(_P)]),
    "pop_prefill_partition_prepared": (C.c_int, [_P, C.c_int, _P, Ratios, _P, C.POINTER(_P)]),
    "pop_prefill_partition_probe": (C.c_int, [_P, C.c_int, C.c_int, _P, Ratios, _P, C.POINTER(_P)]),
    "pop_weights_destroy": (C.c_int, [_P]),
    "pop_prefill_partition_with_output": (C.c_int, [_P, C.c_int, _P, Ratios, C.c_int, _P, _P, C.POINTER(_P)]),
    "pop_partition_from_indices": (C.c_int, [_P, _P, _P, C.c_int, C.c_int, C.c_int, _P, C.c_int, _P, C.c_int,
                                             _P, C.POINTER(_P)]),
    "pop_partition_sizes": (C.c_int, [_P] + [C.POINTER(C.c_int)] * 3),
    "pop_partition_indices": (C.c_int, [_P] + [C.POINTER(_P)] * 3),
    "pop_partition_scores": (C.c_int, [_P, C.POINTER(_P)]),
    "pop_partition_score_bounds": (C.c_int, [_P, C.POINTER(_P)]),
    "pop_partition_streamed_scores": (C.c_int, [_P, C.POINTER(_P)]),
    "pop_partition_shape": (C.c_int, [_P, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "pop_partition_check": (C.c_int, [_P]),
    "pop_partition_destroy": (C.c_int, [_P]),
    "pop_decode_step": (C.c_int, [_P, _P, C.c_int, C.c_int, _P, _P, _P, _P]),
    "pop_prefill_scores_noalloc": (C.c_int, [_P, C.c_int, C.c_int, _P, _P, _P, C.c_int, C.c_int, _P, _P]),
}


def lib() -> C.CDLL:
    """Loads libpop.so (built by ``__graft_entry__.build()``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not built: run `python -c 'import __graft_entry__ as g; g.build()'`")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


def version() -> str:
    return lib().pop_version().decode()


def kernel_launch_count() -> int:
    return int(lib().pop_kernel_launch_count())


def status_string(status: int) -> str:
    return lib().pop_status_string(status).decode()


def _check(status: int, where: str):
    if status != POP_OK:
        raise PopError(status, where)


def get_config() -> Config:
    c = Config()
    _check(lib().pop_get_config(C.byref(c)), "pop_get_config")
    return c


def set_config(**fields) -> Config:
    """pop_set_config with the named fields replaced (decode_kernel, launch_mode, wait_budget_us, slab_cache_bytes);
    returns the settings that were in force before."""
    old = get_config()
    new = Config(old.decode_kernel, old.launch_mode, old.wait_budget_us, old.slab_cache_bytes)
    for k, v in fields.items():
        if k not in dict(Config._fields_):
            raise KeyError(k)
        setattr(new, k, v)
    _check(lib().pop_set_config(C.byref(new)), "pop_set_config")
    return old


def release_cached_memory():
    _check(lib().pop_release_cached_memory(), "pop_release_cached_memory")


def region_sizes(N: int, ratios) -> Tuple[int, int, int, int]:
    """(n_ret, n_cand, n_pruned, k_default) - host only."""
    out = [C.c_int() for _ in range(4)]
    _check(lib().pop_region_sizes(N, Ratios(*ratios), *[C.byref(o) for o in out]), "pop_region_sizes")
    return tuple(o.value for o in out)


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2602_06822_b200 needs a CUDA device (there is no CPU path)")
    return torch


def _dtype_code(t) -> int:
    torch = _torch()
    if t.dtype == torch.float32:
        return POP_F32
    if t.dtype == torch.bfloat16:
        return POP_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream_ptr(stream=None) -> int:
    torch = _torch()
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


class _DevView:
    """Minimal __cuda_array_interface__ carrier for a raw device pointer."""

    def __init__(self, ptr: int, n: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2, "strides": None}


class Partition:
    """Owner of a ``pop_partition_t*``."""

    def __init__(self, handle: int, device):
        self._h = C.c_void_p(handle)
        self.device = device
        n = [C.c_int() for _ in range(3)]
        _check(lib().pop_partition_sizes(self._h, *[C.byref(v) for v in n]), "pop_partition_sizes")
        self.n_ret, self.n_cand, self.n_pruned = (v.value for v in n)
        s = [C.c_int() for _ in range(3)]
        _check(lib().pop_partition_shape(self._h, *[C.byref(v) for v in s]), "pop_partition_shape")
        self.d, self.N, self.dtype_code = (v.value for v in s)

    @property
    def handle(self) -> C.c_void_p:
        if self._h is None:
            raise RuntimeError("partition destroyed")
        return self._h

    def _view(self, ptr: int, n: int, typestr: str):
        """torch view (no copy) of a device array owned by the partition."""
        torch = _torch()
        if n == 0:
            return torch.empty(0, device=self.device, dtype={"<i4": torch.int32, "<f8": torch.float64, "<f4": torch.float32}[typestr])
        return torch.as_tensor(_DevView(ptr, n, typestr), device=self.device)

    def indices_device(self):
        """(R, C, P) channel ids as int32 CUDA tensors that alias the partition's arrays."""
        p = [C.c_void_p() for _ in range(3)]
        _check(lib().pop_partition_indices(self.handle, *[C.byref(v) for v in p]), "pop_partition_indices")
        return (self._view(p[0].value, self.n_ret, "<i4"), self._view(p[1].value, self.n_cand, "<i4"),
                self._view(p[2].value, self.n_pruned, "<i4"))

    def indices(self) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """(R, C, P) channel ids as host int32 arrays (synchronises)."""
        return tuple(t.cpu().numpy() for t in self.indices_device())

    def scores(self) -> np.ndarray:
        """Prefill importance scores I_i as a host float64 array (synchronises)."""
        p = C.c_void_p()
        _check(lib().pop_partition_scores(self.handle, C.byref(p)), "pop_partition_scores")
        return self._view(p.value, self.N, "<f8").cpu().numpy()

    def score_bounds(self) -> np.ndarray:
        """Bound of |scores()[i] - exact I_i| per channel as a host float64 array (synchronises)."""
        p = C.c_void_p()
        _check(lib().pop_partition_score_bounds(self.handle, C.byref(p)), "pop_partition_score_bounds")
        return self._view(p.value, self.N, "<f8").cpu().numpy()

    def streamed_scores(self):
        """(score, bound) of every candidate as the streaming kernel's last step saw them: two host float32
        arrays (synchronises); raises PopError(POP_ERR_UNSUPPORTED) for partitions served by another kernel."""
        p = C.c_void_p()
        _check(lib().pop_partition_streamed_scores(self.handle, C.byref(p)), "pop_partition_streamed_scores")
        pairs = self._view(p.value, 2 * self.n_cand, "<f4").cpu().numpy().reshape(self.n_cand, 2)
        return pairs[:, 0].copy(), pairs[:, 1].copy()

    def check(self):
        _check(lib().pop_partition_check(self.handle), "pop_partition_check")

    def destroy(self):
        if self._h is not None:
            _torch().cuda.synchronize(self.device)
            lib().pop_partition_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def prefill_partition(X, Wg, Wu, Wd, ratios, stream=None) -> Partition:
    """pop_prefill_partition: X [L, d], Wg/Wu [N, d], Wd [d, N] CUDA tensors of one dtype."""
    for t in (X, Wg, Wu, Wd):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")
    L, d = X.shape
    N = Wg.shape[0]
    if tuple(Wg.shape) != (N, d) or tuple(Wu.shape) != (N, d) or tuple(Wd.shape) != (d, N):
        raise ValueError("shape mismatch")
    dt = _dtype_code(X)
    if any(_dtype_code(t) != dt for t in (Wg, Wu, Wd)):
        raise TypeError("dtype mismatch")
    out = C.c_void_p()
    _check(lib().pop_prefill_partition(X.data_ptr(), L, d, Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), N, dt,
                                       Ratios(*ratios), _stream_ptr(stream), C.byref(out)),
           "pop_prefill_partition")
    return Partition(out.value, X.device)


class Weights:
    """Owner of a ``pop_weights_t*`` (pop_weights_prepare).  Keeps references to the weight tensors, which the
    library reads again at every prefill that uses the object."""

    def __init__(self, Wg, Wu, Wd, stream=None):
        for t in (Wg, Wu, Wd):
            if not (t.is_cuda and t.is_contiguous()):
                raise ValueError("tensors must be contiguous CUDA tensors")
        N, d = Wg.shape
        if tuple(Wu.shape) != (N, d) or tuple(Wd.shape) != (d, N):
            raise ValueError("shape mismatch")
        dt = _dtype_code(Wg)
        if any(_dtype_code(t) != dt for t in (Wu, Wd)):
            raise TypeError("dtype mismatch")
        self.tensors = (Wg, Wu, Wd)
        self.device = Wg.device
        out = C.c_void_p()
        _check(lib().pop_weights_prepare(Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), N, d, dt, _stream_ptr(stream),
                                         C.byref(out)), "pop_weights_prepare")
        self._h = out

    def prefill_partition(self, X, ratios, stream=None) -> "Partition":
        """pop_prefill_partition_prepared: X [L, d] -> partition, with this weight set's statistics."""
        if not (X.is_cuda and X.is_contiguous()) or _dtype_code(X) != _dtype_code(self.tensors[0]):
            raise ValueError("X must be a contiguous CUDA tensor of the weights' dtype")
        if X.shape[1] != self.tensors[0].shape[1]:
            raise ValueError("shape mismatch")
        out = C.c_void_p()
        _check(lib().pop_prefill_partition_prepared(X.data_ptr(), X.shape[0], self._h, Ratios(*ratios), _stream_ptr(stream),
                                                    C.byref(out)), "pop_prefill_partition_prepared")
        return Partition(out.value, X.device)

    def prefill_partition_probe(self, X, ratios, token_stride: int, stream=None) -> "Partition":
        """pop_prefill_partition_probe: the partition from every token_stride-th row of X [L, d]."""
        if not (X.is_cuda and X.is_contiguous()) or _dtype_code(X) != _dtype_code(self.tensors[0]):
            raise ValueError("X must be a contiguous CUDA tensor of the weights' dtype")
        if X.shape[1] != self.tensors[0].shape[1]:
            raise ValueError("shape mismatch")
        out = C.c_void_p()
        _check(lib().pop_prefill_partition_probe(X.data_ptr(), X.shape[0], int(token_stride), self._h, Ratios(*ratios),
                                                 _stream_ptr(stream), C.byref(out)), "pop_prefill_partition_probe")
        return Partition(out.value, X.device)

    def prefill_partition_with_output(self, X, ratios, k: int, Y=None, stream=None):
        """pop_prefill_partition_with_output: (partition, Y [L, d]) - the partition and the prompt's own block output
        over Retained + the k best Candidates by prefill score."""
        torch = _torch()
        if not (X.is_cuda and X.is_contiguous()) or _dtype_code(X) != _dtype_code(self.tensors[0]):
            raise ValueError("X must be a contiguous CUDA tensor of the weights' dtype")
        if Y is None:
            Y = torch.empty_like(X)
        out = C.c_void_p()
        _check(lib().pop_prefill_partition_with_output(X.data_ptr(), X.shape[0], self._h, Ratios(*ratios), k, Y.data_ptr(),
                                                       _stream_ptr(stream), C.byref(out)), "pop_prefill_partition_with_output")
        return Partition(out.value, X.device), Y

    def destroy(self):
        if self._h is not None:
            _torch().cuda.synchronize(self.device)
            lib().pop_weights_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def partition_from_indices(Wg, Wu, Wd, ret: np.ndarray, cand: np.ndarray, stream=None) -> Partition:
    for t in (Wg, Wu, Wd):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")
    N, d = Wg.shape
    ret = np.ascontiguousarray(ret, dtype=np.int32)
    cand = np.ascontiguousarray(cand, dtype=np.int32)
    out = C.c_void_p()
    _check(lib().pop_partition_from_indices(Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), N, d, _dtype_code(Wg),
                                            ret.ctypes.data, ret.size, cand.ctypes.data, cand.size,
                                            _stream_ptr(stream), C.byref(out)),
           "pop_partition_from_indices")
    return Partition(out.value, Wg.device)


def decode_step(part: Partition, x, k: int, y=None, mask_out=None, sel_out=None, stream=None):
    """pop_decode_step: x [B, d] -> y [B, d]; optional mask_out uint8 [n_cand], sel_out int32 [k]."""
    torch = _torch()
    if x.dim() == 1:
        x = x.unsqueeze(0)
    if not (x.is_cuda and x.is_contiguous()):
        raise ValueError("x must be a contiguous CUDA tensor")
    B, d = x.shape
    if d != part.d or _dtype_code(x) != part.dtype_code:
        raise ValueError("x does not match the partition")
    if y is None:
        y = torch.empty_like(x)
    _check(lib().pop_decode_step(part.handle, x.data_ptr(), B, k, y.data_ptr(),
                                 None if mask_out is None else mask_out.data_ptr(),
                                 None if sel_out is None else sel_out.data_ptr(), _stream_ptr(stream)),
           "pop_decode_step")
    return y


def prefill_scores_noalloc(X, Wg, Wu, Wd, out, stream=None):
    """pop_prefill_scores_noalloc: the prefill scores I_i written into ``out`` (a float64 CUDA
    tensor of N elements that the caller already owns).  The library call allocates nothing: its
    temporaries live in a fixed array inside the library, shared by all calls on the device."""
    torch = _torch()
    for t in (X, Wg, Wu, Wd, out):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")
    L, d = X.shape
    N = Wg.shape[0]
    if out.dtype != torch.float64 or out.numel() != N:
        raise ValueError("out must be a float64 tensor of N elements")
    _check(lib().pop_prefill_scores_noalloc(X.data_ptr(), L, d, Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), N,
                                            _dtype_code(X), out.data_ptr(), _stream_ptr(stream)),
           "pop_prefill_scores_noalloc")
    return out
