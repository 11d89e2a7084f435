"""Thin ctypes binding over the C ABI of ``libkvq.so`` (``include/kvq.h``).

Argument marshalling only: every step of the quantizer runs in the library's CUDA
kernels.  PyTorch provides device memory and streams.  If the library has not
been built the binding raises; there is no other code path.

The functions carry the names of the C entry points: ``kvq_plan_create``,
``kvq_encode``, ``kvq_decode``, ``kvq_append`` ...  ``Plan`` is a small
convenience holder that frees the plan when collected.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvq.so")

KVQ_OK = 0
KVQ_ERR_INVALID_ARG = 1
KVQ_ERR_UNSUPPORTED_DIM = 2
KVQ_ERR_ALIGNMENT = 3
KVQ_ERR_CUDA = 4
KVQ_ERR_TIMEOUT = 5
KVQ_ERR_NOMEM = 6
KVQ_ERR_SCRATCH_LIMIT = 7
KVQ_ERR_RANGE = 8
KVQ_DEV_POSITION = 16   # bit of the device status word: kvq_append_at / kvq_flush_block_at met a position outside the cache

KVQ_F16 = 0
KVQ_BF16 = 1

KVQ_IMPL_AUTO = 0
KVQ_IMPL_FFT = 1
KVQ_IMPL_GEMM = 2
KVQ_IMPL_MATVEC = 3

# every symbol include/kvq.h declares
EXPORTS = (
    "kvq_plan_create", "kvq_plan_create_ex", "kvq_plan_set_rotation", "kvq_plan_clear_device_status", "kvq_plan_destroy", "kvq_plan_get_signs", "kvq_plan_describe", "kvq_plan_set_impl",
    "kvq_plan_device_status", "kvq_plan_prepare", "kvq_plan_set_wait_limit", "kvq_encode", "kvq_decode", "kvq_append", "kvq_decode_static", "kvq_calibrate_lambda", "kvq_flush_block", "kvq_append_at", "kvq_flush_block_at",
    "kvq_status_string",
    "kvq_launch_count",
)

_lib = None


class KvqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, status_string(status)))


def lib() -> ctypes.CDLL:
    """Loads libkvq.so (once).  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libkvq.so is missing at %s; build it with `python -m paper_2605_05699_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        i32, i64, u64, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p
        L.kvq_plan_create.restype = i32
        L.kvq_plan_create.argtypes = [i32, i32, u64, ctypes.POINTER(vp)]
        L.kvq_plan_clear_device_status.restype = i32
        L.kvq_plan_clear_device_status.argtypes = [vp]
        L.kvq_plan_set_rotation.restype = i32
        L.kvq_plan_set_rotation.argtypes = [vp, vp]
        L.kvq_plan_create_ex.restype = i32
        L.kvq_plan_create_ex.argtypes = [i32, i32, i32, u64, ctypes.POINTER(vp)]
        L.kvq_plan_destroy.restype = i32
        L.kvq_plan_destroy.argtypes = [vp]
        L.kvq_plan_get_signs.restype = i32
        L.kvq_plan_get_signs.argtypes = [vp, vp]
        L.kvq_plan_describe.restype = i32
        L.kvq_plan_describe.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_size_t)]
        L.kvq_plan_set_impl.restype = i32
        L.kvq_plan_set_impl.argtypes = [vp, i32, i32]
        L.kvq_plan_prepare.restype = i32
        L.kvq_plan_prepare.argtypes = [vp, i32]
        L.kvq_plan_set_wait_limit.restype = i32
        L.kvq_plan_set_wait_limit.argtypes = [vp, ctypes.c_uint32]
        L.kvq_plan_device_status.restype = i32
        L.kvq_plan_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
        L.kvq_encode.restype = i32
        L.kvq_encode.argtypes = [vp, vp, i32, i64, vp, i64, i64, vp, vp, vp]
        L.kvq_decode.restype = i32
        L.kvq_decode.argtypes = [vp, vp, vp, i64, vp, i64, i64, vp, i32, vp]
        L.kvq_append.restype = i32
        L.kvq_append.argtypes = [vp, vp, i32, i64, vp, i64, i64, vp, vp, i64, i64, vp]
        L.kvq_decode_static.restype = i32
        L.kvq_decode_static.argtypes = [vp, vp, vp, i64, vp, i64, i64, vp, i32, vp, vp]
        L.kvq_flush_block.restype = i32
        L.kvq_flush_block.argtypes = [vp, vp, i32, i64, i64, vp, i64, i64, vp, vp, vp, i64, i64, vp]
        L.kvq_append_at.restype = i32
        L.kvq_append_at.argtypes = [vp, vp, i32, i64, vp, i64, i64, vp, vp, i64, vp, vp]
        L.kvq_flush_block_at.restype = i32
        L.kvq_flush_block_at.argtypes = [vp, vp, i32, i64, i64, vp, i64, i64, vp, vp, vp, i64, vp, vp]
        L.kvq_calibrate_lambda.restype = i32
        L.kvq_calibrate_lambda.argtypes = [vp, vp, i32, i64, vp, vp]
        L.kvq_status_string.restype = ctypes.c_char_p
        L.kvq_status_string.argtypes = [i32]
        L.kvq_launch_count.restype = u64
        L.kvq_launch_count.argtypes = []
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().kvq_status_string(int(status)).decode()


def kvq_launch_count() -> int:
    return int(lib().kvq_launch_count())


def _check(status: int, where: str):
    if status != KVQ_OK:
        raise KvqError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return KVQ_F16
    if t.dtype == torch.bfloat16:
        return KVQ_BF16
    raise TypeError("expected a float16 or bfloat16 tensor, got %s" % t.dtype)


def _dev(t: torch.Tensor, what: str) -> int:
    if not t.is_cuda:
        raise ValueError("%s must live on a CUDA device" % what)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % what)
    return t.data_ptr()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream, device: torch.device = None) -> int:
    if stream is None:
        if _raw_stream is not None and device is not None and device.index is not None:
            return _raw_stream(device.index)   # the handle itself: no Stream object per call
        return torch.cuda.current_stream(device).cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


class _on_device:
    """Makes ``device`` current for the call (a plan's tables live on the device of its first use) and restores the
    previous one; costs one query when it already is current, which is the usual case."""
    __slots__ = ("idx", "prev")

    def __init__(self, device: torch.device):
        self.idx = device.index
        self.prev = -1

    def __enter__(self):
        if self.idx is not None:
            cur = torch.cuda.current_device()
            if cur != self.idx:
                self.prev = cur
                torch.cuda.set_device(self.idx)
        return self

    def __exit__(self, *exc):
        if self.prev >= 0:
            torch.cuda.set_device(self.prev)
        return False


# ---- C entry points, same names ---------------------------------------------------------

def kvq_plan_create(D: int, group: int, seed: int) -> int:
    h = ctypes.c_void_p()
    _check(lib().kvq_plan_create(D, group, ctypes.c_uint64(seed & (2**64 - 1)), ctypes.byref(h)), "kvq_plan_create")
    return h.value


def kvq_plan_create_ex(D: int, group: int, bits: int, seed: int) -> int:
    h = ctypes.c_void_p()
    _check(lib().kvq_plan_create_ex(D, group, bits, ctypes.c_uint64(seed & (2**64 - 1)), ctypes.byref(h)), "kvq_plan_create_ex")
    return h.value


def kvq_plan_set_rotation(plan: int, R, D: int) -> None:
    """R: host fp32 [D, D] (torch CPU tensor or numpy array) for a plan of head dimension D, or None to remove the
    rotation."""
    if R is None:
        _check(lib().kvq_plan_set_rotation(plan, None), "kvq_plan_set_rotation")
        return
    if isinstance(R, torch.Tensor):
        if R.is_cuda:
            raise ValueError("the rotation is a host matrix")
        R = R.detach().to(torch.float32).contiguous().numpy()
    import numpy as np

    R = np.ascontiguousarray(R, dtype=np.float32)
    if R.shape != (D, D):
        raise ValueError("the rotation must be [D, D]")
    _check(lib().kvq_plan_set_rotation(plan, R.ctypes.data_as(ctypes.c_void_p)), "kvq_plan_set_rotation")


def kvq_plan_destroy(plan: int) -> None:
    _check(lib().kvq_plan_destroy(plan), "kvq_plan_destroy")


def kvq_plan_get_signs(plan: int, D: int):
    import numpy as np

    s = np.empty(D, dtype=np.int8)
    _check(lib().kvq_plan_get_signs(plan, s.ctypes.data_as(ctypes.c_void_p)), "kvq_plan_get_signs")
    return s


def kvq_plan_describe(plan: int):
    r = (ctypes.c_int * 8)()
    n = ctypes.c_int()
    tb = ctypes.c_size_t()
    _check(lib().kvq_plan_describe(plan, r, ctypes.byref(n), ctypes.byref(tb)), "kvq_plan_describe")
    return list(r[: n.value]), int(tb.value)


def kvq_plan_set_impl(plan: int, encode_impl: int, decode_impl: int) -> None:
    _check(lib().kvq_plan_set_impl(plan, encode_impl, decode_impl), "kvq_plan_set_impl")


def kvq_plan_device_status(plan: int) -> int:
    w = ctypes.c_uint32()
    st = lib().kvq_plan_device_status(plan, ctypes.byref(w))
    # the codes that describe the word (bit 4, a position outside the cache, reads KVQ_ERR_INVALID_ARG) are not failures of the call
    if st not in (KVQ_OK, KVQ_ERR_TIMEOUT, KVQ_ERR_RANGE) and not (st == KVQ_ERR_INVALID_ARG and w.value & KVQ_DEV_POSITION):
        raise KvqError(st, "kvq_plan_device_status")
    return int(w.value)


def kvq_plan_prepare(plan: int, dtype: torch.dtype, device=None) -> None:
    """Allocates the plan's device tables and sets every kernel's launch attributes now, on ``device`` (default: the
    current one), so that later calls with tensors of ``dtype`` allocate nothing and never block."""
    code = KVQ_F16 if dtype == torch.float16 else KVQ_BF16 if dtype == torch.bfloat16 else -1
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with _on_device(dev):
        _check(lib().kvq_plan_prepare(plan, code), "kvq_plan_prepare")


def kvq_plan_set_wait_limit(plan: int, polls: int) -> None:
    _check(lib().kvq_plan_set_wait_limit(plan, polls), "kvq_plan_set_wait_limit")


def kvq_plan_clear_device_status(plan: int) -> None:
    _check(lib().kvq_plan_clear_device_status(plan), "kvq_plan_clear_device_status")


def kvq_encode(plan: int, x: torch.Tensor, lam: torch.Tensor, packed: torch.Tensor, scales: torch.Tensor,
               rows_per_lambda: int = 0, stream=None) -> None:
    D = x.shape[-1]
    N = x.numel() // D
    n_lambda = lam.numel() // D
    with _on_device(x.device):
        _check(lib().kvq_encode(plan, _dev(x, "x"), _dtype_code(x), N, _dev(lam, "lambda"), n_lambda,
                                rows_per_lambda, _dev(packed, "packed"), _dev(scales, "scales"), _stream(stream, x.device)),
               "kvq_encode")


def kvq_decode(plan: int, packed: torch.Tensor, scales: torch.Tensor, lam: torch.Tensor, out: torch.Tensor,
               rows_per_lambda: int = 0, stream=None) -> None:
    D = out.shape[-1]
    N = out.numel() // D
    n_lambda = lam.numel() // D
    with _on_device(out.device):
        _check(lib().kvq_decode(plan, _dev(packed, "packed"), _dev(scales, "scales"), N, _dev(lam, "lambda"),
                                n_lambda, rows_per_lambda, _dev(out, "out"), _dtype_code(out), _stream(stream, out.device)),
               "kvq_decode")


def kvq_append(plan: int, x_new: torch.Tensor, lam: torch.Tensor, packed_cache: torch.Tensor,
               scales_cache: torch.Tensor, pos: int, streams_per_lambda: int = 0, stream=None) -> None:
    D = x_new.shape[-1]
    S = x_new.numel() // D
    T_max = packed_cache.shape[-2]
    n_lambda = lam.numel() // D
    with _on_device(x_new.device):
        _check(lib().kvq_append(plan, _dev(x_new, "x_new"), _dtype_code(x_new), S, _dev(lam, "lambda"), n_lambda,
                                streams_per_lambda, _dev(packed_cache, "packed_cache"),
                                _dev(scales_cache, "scales_cache"), T_max, pos, _stream(stream, x_new.device)),
               "kvq_append")


def kvq_decode_static(plan: int, packed: torch.Tensor, scales: torch.Tensor, lam: torch.Tensor, out: torch.Tensor,
                      rows_per_lambda: int = 0, status_word: torch.Tensor | None = None, stream=None) -> None:
    """kvq_decode without any device allocation inside the library (D = 128, fp16 output only).

    For embedders that own all device memory themselves or cannot take an allocation in their decode
    loop: the kernel's table and status word live in a fixed block inside the library.  Calls must not
    overlap on the GPU; ``status_word`` is an optional int32 device tensor of one element."""
    D = out.shape[-1]
    N = out.numel() // D
    n_lambda = lam.numel() // D
    sw = None if status_word is None else _dev(status_word, "status_word")
    with _on_device(out.device):
        _check(lib().kvq_decode_static(plan, _dev(packed, "packed"), _dev(scales, "scales"), N, _dev(lam, "lambda"),
                                       n_lambda, rows_per_lambda, _dev(out, "out"), _dtype_code(out), sw,
                                       _stream(stream, out.device)),
               "kvq_decode_static")


def kvq_flush_block(plan: int, x_block: torch.Tensor, lam: torch.Tensor, packed_cache: torch.Tensor, scales_cache: torch.Tensor,
                    dq_cache: torch.Tensor, pos0: int, streams_per_lambda: int = 0, stream=None) -> None:
    S, rows, D = x_block.shape
    T_max = packed_cache.shape[-2]
    n_lambda = lam.numel() // D
    with _on_device(x_block.device):
        _check(lib().kvq_flush_block(plan, _dev(x_block, "x_block"), _dtype_code(x_block), S, rows, _dev(lam, "lambda"), n_lambda,
                                     streams_per_lambda, _dev(packed_cache, "packed_cache"), _dev(scales_cache, "scales_cache"),
                                     _dev(dq_cache, "dq_cache"), T_max, pos0, _stream(stream, x_block.device)),
               "kvq_flush_block")


def _pos_word(pos_device: torch.Tensor):
    if pos_device.dtype != torch.int64 or pos_device.numel() != 1:
        raise TypeError("the position word must be one int64 on the device")
    return _dev(pos_device, "pos_device")


def kvq_append_at(plan: int, x_new: torch.Tensor, lam: torch.Tensor, packed_cache: torch.Tensor, scales_cache: torch.Tensor,
                  pos_device: torch.Tensor, streams_per_lambda: int = 0, stream=None) -> None:
    """kvq_append with the row to write read from ``pos_device`` (one int64 on the device) when the kernel runs."""
    D = x_new.shape[-1]
    S = x_new.numel() // D
    T_max = packed_cache.shape[-2]
    n_lambda = lam.numel() // D
    with _on_device(x_new.device):
        _check(lib().kvq_append_at(plan, _dev(x_new, "x_new"), _dtype_code(x_new), S, _dev(lam, "lambda"), n_lambda,
                                   streams_per_lambda, _dev(packed_cache, "packed_cache"), _dev(scales_cache, "scales_cache"),
                                   T_max, _pos_word(pos_device), _stream(stream, x_new.device)),
               "kvq_append_at")


def kvq_flush_block_at(plan: int, x_block: torch.Tensor, lam: torch.Tensor, packed_cache: torch.Tensor, scales_cache: torch.Tensor,
                       dq_cache: torch.Tensor, pos0_device: torch.Tensor, streams_per_lambda: int = 0, stream=None) -> None:
    """kvq_flush_block with the first row to write read from ``pos0_device`` (one int64 on the device) when the kernel runs."""
    S, rows, D = x_block.shape
    T_max = packed_cache.shape[-2]
    n_lambda = lam.numel() // D
    with _on_device(x_block.device):
        _check(lib().kvq_flush_block_at(plan, _dev(x_block, "x_block"), _dtype_code(x_block), S, rows, _dev(lam, "lambda"), n_lambda,
                                        streams_per_lambda, _dev(packed_cache, "packed_cache"), _dev(scales_cache, "scales_cache"),
                                        _dev(dq_cache, "dq_cache"), T_max, _pos_word(pos0_device), _stream(stream, x_block.device)),
               "kvq_flush_block_at")


def kvq_calibrate_lambda(plan: int, x: torch.Tensor, lambda_out: torch.Tensor, stream=None) -> None:
    D = x.shape[-1]
    N = x.numel() // D
    with _on_device(x.device):
        _check(lib().kvq_calibrate_lambda(plan, _dev(x, "x"), _dtype_code(x), N, _dev(lambda_out, "lambda_out"), _stream(stream, x.device)),
               "kvq_calibrate_lambda")


class Plan:
    """Owns a ``kvq_plan_t`` handle: ``Plan(D, group, seed).handle`` goes to the kvq_* calls.  ``bits=8`` or
    ``group=D`` select the base variants (kvq_plan_create_ex)."""

    def __init__(self, D: int, group: int = 32, seed: int = 0, bits: int = 4):
        self.D, self.group, self.seed, self.bits = D, group, seed, bits
        self.handle = kvq_plan_create(D, group, seed) if bits == 4 and group == 32 else kvq_plan_create_ex(D, group, bits, seed)

    def signs(self):
        return kvq_plan_get_signs(self.handle, self.D)

    def set_rotation(self, R) -> None:
        kvq_plan_set_rotation(self.handle, R, self.D)

    def describe(self):
        """(radices of the length-D/2 complex FFT, bytes of device tables the plan holds: 0 until its first use on a device)"""
        return kvq_plan_describe(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            kvq_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    # allocation helpers for callers that do not bring their own buffers
    def empty_packed(self, N: int, device="cuda") -> torch.Tensor:
        return torch.empty(N, self.D * self.bits // 8, dtype=torch.uint8, device=device)

    def empty_scales(self, N: int, device="cuda") -> torch.Tensor:
        return torch.empty(N, self.D // self.group, dtype=torch.float16, device=device)
