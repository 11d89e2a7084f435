"""ctypes front end of the fp64 CPU oracle (``kvq_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It shares nothing with
the CUDA library and never imports the product package.

Every function takes and returns NumPy arrays on the host.  Half-precision
data travels as raw ``uint16`` bit patterns so that no conversion happens
outside the C file (``numpy.float16`` arrays are reinterpreted, bfloat16 is
always raw bits).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvq_oracle.c")
_LIB = os.path.join(_HERE, "libkvq_oracle.so")

F16 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=gnu11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, u64, p = ctypes.c_int64, ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p
        lib.kvqo_f16_to_f64.restype = ctypes.c_double
        lib.kvqo_f16_to_f64.argtypes = [ctypes.c_uint16]
        lib.kvqo_bf16_to_f64.restype = ctypes.c_double
        lib.kvqo_bf16_to_f64.argtypes = [ctypes.c_uint16]
        for name in ("kvqo_f64_to_f16", "kvqo_f64_to_f16_sat", "kvqo_f64_to_bf16"):
            getattr(lib, name).restype = ctypes.c_uint16
            getattr(lib, name).argtypes = [ctypes.c_double]
        lib.kvqo_splitmix64_mix.restype = u64
        lib.kvqo_splitmix64_mix.argtypes = [u64]
        lib.kvqo_signs.restype = None
        lib.kvqo_signs.argtypes = [i32, u64, p]
        lib.kvqo_srft_forward.restype = i32
        lib.kvqo_srft_forward.argtypes = [i32, p, p, p, i64]
        lib.kvqo_srft_inverse.restype = i32
        lib.kvqo_srft_inverse.argtypes = [i32, p, p, p, i64]
        lib.kvqo_calibrate_lambda.restype = i32
        lib.kvqo_calibrate_lambda.argtypes = [i32, p, p, i32, i64, p, p]
        lib.kvqo_pack_nibbles.restype = None
        lib.kvqo_pack_nibbles.argtypes = [p, i64, p]
        lib.kvqo_unpack_nibbles.restype = None
        lib.kvqo_unpack_nibbles.argtypes = [p, i64, p]
        lib.kvqo_encode_f64.restype = i32
        lib.kvqo_encode_f64.argtypes = [i32, i32, p, p, i64, p, i64, i64, p, p, p, p]
        lib.kvqo_encode.restype = i32
        lib.kvqo_encode.argtypes = [i32, i32, p, p, i32, i64, p, i64, i64, p, p, p, p]
        lib.kvqo_decode.restype = i32
        lib.kvqo_decode.argtypes = [i32, i32, p, p, p, i64, p, i64, i64, p, i32, p]
        lib.kvqo_encode_f64_br.restype = i32
        lib.kvqo_encode_f64_br.argtypes = [i32, i32, i32, p, p, p, i64, p, i64, i64, p, p, p, p]
        lib.kvqo_encode_br.restype = i32
        lib.kvqo_encode_br.argtypes = [i32, i32, i32, p, p, p, i32, i64, p, i64, i64, p, p, p, p]
        lib.kvqo_decode_br.restype = i32
        lib.kvqo_decode_br.argtypes = [i32, i32, i32, p, p, p, p, i64, p, i64, i64, p, i32, p]
        lib.kvqo_append.restype = i32
        lib.kvqo_append.argtypes = [i32, i32, p, p, i32, i64, p, i64, i64, p, p, i64, i64]
        lib.kvqo_num_threads.restype = i32
        lib.kvqo_num_threads.argtypes = []
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _raw16(x) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype == np.float16:
        x = x.view(np.uint16)
    if x.dtype != np.uint16:
        raise TypeError("half-precision data must be float16 or raw uint16 bits")
    return x


def _rot(rot, D):
    """None, or the rotation as a contiguous fp64 [D, D] array (row-major)."""
    if rot is None:
        return None
    rot = np.ascontiguousarray(rot, dtype=np.float64)
    if rot.shape != (D, D):
        raise ValueError("rotation must be [D, D]")
    return rot


def _lam(lam, D):
    lam = np.ascontiguousarray(lam, dtype=np.float32).reshape(-1, D)
    return lam, lam.shape[0]


def num_threads() -> int:
    return int(_load().kvqo_num_threads())


# ---- number formats -------------------------------------------------------

def f16_to_f64(bits) -> np.ndarray:
    lib = _load()
    b = np.asarray(bits, dtype=np.uint16)
    return np.array([lib.kvqo_f16_to_f64(int(v)) for v in b.ravel()], dtype=np.float64).reshape(b.shape)


def bf16_to_f64(bits) -> np.ndarray:
    lib = _load()
    b = np.asarray(bits, dtype=np.uint16)
    return np.array([lib.kvqo_bf16_to_f64(int(v)) for v in b.ravel()], dtype=np.float64).reshape(b.shape)


def f64_to_f16(v, saturate: bool = False) -> np.ndarray:
    lib = _load()
    f = lib.kvqo_f64_to_f16_sat if saturate else lib.kvqo_f64_to_f16
    a = np.asarray(v, dtype=np.float64)
    return np.array([f(float(t)) for t in a.ravel()], dtype=np.uint16).reshape(a.shape)


def f64_to_bf16(v) -> np.ndarray:
    lib = _load()
    a = np.asarray(v, dtype=np.float64)
    return np.array([lib.kvqo_f64_to_bf16(float(t)) for t in a.ravel()], dtype=np.uint16).reshape(a.shape)


def widen(raw, dtype: int) -> np.ndarray:
    """Exact fp64 value of raw half-precision bits (vectorised through NumPy views)."""
    raw = _raw16(raw)
    if dtype == F16:
        return raw.view(np.float16).astype(np.float64)
    return (raw.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ---- sign diagonal --------------------------------------------------------

def splitmix64_mix(z: int) -> int:
    return int(_load().kvqo_splitmix64_mix(ctypes.c_uint64(z & (2**64 - 1))))


def signs(D: int, seed: int) -> np.ndarray:
    s = np.empty(D, dtype=np.int8)
    _load().kvqo_signs(D, ctypes.c_uint64(seed & (2**64 - 1)), _ptr(s))
    return s


# ---- transform ------------------------------------------------------------

def srft_forward(x, sg) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    D = x.shape[-1]
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    z = np.empty_like(x)
    rc = _load().kvqo_srft_forward(D, _ptr(sg), _ptr(x), _ptr(z), x.size // D)
    if rc:
        raise ValueError("kvqo_srft_forward: rc=%d" % rc)
    return z


def srft_inverse(z, sg) -> np.ndarray:
    z = np.ascontiguousarray(z, dtype=np.float64)
    D = z.shape[-1]
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    x = np.empty_like(z)
    rc = _load().kvqo_srft_inverse(D, _ptr(sg), _ptr(z), _ptr(x), z.size // D)
    if rc:
        raise ValueError("kvqo_srft_inverse: rc=%d" % rc)
    return x


def calibrate_lambda(x_raw, dtype: int, sg):
    """Static lambda calibration (Sec. 7.1): lambda_c = 1 / max_n |SRFT(x_n)_c| over the rows of ``x_raw``
    (half-precision bit patterns).  Returns (lambda [D] float64, amax [D] float64)."""
    x = _raw16(x_raw)
    D = x.shape[-1]
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    lam = np.empty(D, dtype=np.float64)
    amax = np.empty(D, dtype=np.float64)
    rc = _load().kvqo_calibrate_lambda(D, _ptr(sg), _ptr(x), dtype, x.size // D, _ptr(lam), _ptr(amax))
    if rc:
        raise ValueError("kvqo_calibrate_lambda: rc=%d" % rc)
    return lam, amax


# ---- nibbles --------------------------------------------------------------

def pack_nibbles(q) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    out = np.empty(q.shape[:-1] + (q.shape[-1] // 2,), dtype=np.uint8)
    _load().kvqo_pack_nibbles(_ptr(q), q.size, _ptr(out))
    return out


def unpack_nibbles(b) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint8)
    out = np.empty(b.shape[:-1] + (b.shape[-1] * 2,), dtype=np.int8)
    _load().kvqo_unpack_nibbles(_ptr(b), out.size, _ptr(out))
    return out


# ---- quantizer ------------------------------------------------------------

def encode_f64(x, sg, lam, group: int, rows_per_lambda: int = 0, want_v: bool = False, bits: int = 4, rot=None):
    """Forward path on fp64 rows.  Returns dict(packed, scales, codes[, v]).  ``packed`` is [N, D/2] nibble pairs for
    bits = 4 and [N, D] two's-complement bytes for bits = 8."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    D = x.shape[-1]
    N = x.size // D
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    lam, nl = _lam(lam, D)
    packed = np.empty((N, D * bits // 8), dtype=np.uint8)
    scales = np.empty((N, D // group), dtype=np.uint16)
    codes = np.empty((N, D), dtype=np.int8)
    v = np.empty((N, D), dtype=np.float64) if want_v else None
    rot = _rot(rot, D)
    rc = _load().kvqo_encode_f64_br(D, group, bits, _ptr(rot), _ptr(sg), _ptr(x), N, _ptr(lam), nl, rows_per_lambda,
                                    _ptr(packed), _ptr(scales), _ptr(codes), _ptr(v))
    if rc:
        raise ValueError("kvqo_encode_f64: rc=%d" % rc)
    out = {"packed": packed, "scales": scales, "codes": codes}
    if want_v:
        out["v"] = v
    return out


def encode(x_raw, dtype: int, sg, lam, group: int, rows_per_lambda: int = 0, want_v: bool = False, bits: int = 4,
           rot=None):
    """Forward path on fp16 / bf16 rows given as raw bits.  Returns dict(packed, scales, codes[, v])."""
    x = _raw16(x_raw)
    D = x.shape[-1]
    N = x.size // D
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    lam, nl = _lam(lam, D)
    packed = np.empty((N, D * bits // 8), dtype=np.uint8)
    scales = np.empty((N, D // group), dtype=np.uint16)
    codes = np.empty((N, D), dtype=np.int8)
    v = np.empty((N, D), dtype=np.float64) if want_v else None
    rot = _rot(rot, D)
    rc = _load().kvqo_encode_br(D, group, bits, _ptr(rot), _ptr(sg), _ptr(x), dtype, N, _ptr(lam), nl, rows_per_lambda,
                                _ptr(packed), _ptr(scales), _ptr(codes), _ptr(v))
    if rc:
        raise ValueError("kvqo_encode: rc=%d" % rc)
    out = {"packed": packed, "scales": scales, "codes": codes}
    if want_v:
        out["v"] = v
    return out


def decode(packed, scales, sg, lam, group: int, dtype: int, rows_per_lambda: int = 0, want_f64: bool = False,
           bits: int = 4, rot=None):
    """Inverse path.  Returns raw bits of the rounded output, or (bits, fp64) if want_f64."""
    packed = np.ascontiguousarray(packed).view(np.uint8)
    D = packed.shape[-1] * 8 // bits
    N = packed.size // packed.shape[-1]
    scales = _raw16(scales)
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    lam, nl = _lam(lam, D)
    out = np.empty((N, D), dtype=np.uint16)
    o64 = np.empty((N, D), dtype=np.float64) if want_f64 else None
    rot = _rot(rot, D)
    rc = _load().kvqo_decode_br(D, group, bits, _ptr(rot), _ptr(sg), _ptr(packed), _ptr(scales), N, _ptr(lam), nl,
                                rows_per_lambda, _ptr(out), dtype, _ptr(o64))
    if rc:
        raise ValueError("kvqo_decode: rc=%d" % rc)
    return (out, o64) if want_f64 else out


def append(x_new_raw, dtype: int, sg, lam, group: int, packed_cache, scales_cache, pos: int,
           streams_per_lambda: int = 0):
    """Quantize S new rows and write them in place at row ``pos`` of [S,T_max,*] caches."""
    x = _raw16(x_new_raw)
    D = x.shape[-1]
    S = x.size // D
    if packed_cache.dtype != np.uint8 or not packed_cache.flags.c_contiguous:
        raise TypeError("packed_cache must be contiguous uint8")
    if scales_cache.dtype != np.uint16 or not scales_cache.flags.c_contiguous:
        raise TypeError("scales_cache must be contiguous uint16 bits")
    T_max = packed_cache.shape[1]
    sg = np.ascontiguousarray(sg, dtype=np.int8)
    lam, nl = _lam(lam, D)
    rc = _load().kvqo_append(D, group, _ptr(sg), _ptr(x), dtype, S, _ptr(lam), nl, streams_per_lambda,
                             _ptr(packed_cache), _ptr(scales_cache), T_max, pos)
    if rc:
        raise ValueError("kvqo_append: rc=%d" % rc)


def flush_block(x_block_raw, dtype: int, sg, lam, group: int, packed_cache, scales_cache, dq_cache, pos0: int,
                streams_per_lambda: int = 0):
    """Residual-window flush with a dequantized-prefix cache (Sec. 7.2), written as its definition: the block's rows
    are appended one token at a time, then the rows just stored are decoded into the same rows of ``dq_cache``
    ([S, T_max, D] raw 16-bit).  Nothing else in the three caches is written."""
    x = _raw16(x_block_raw)
    S, rows, D = x.shape
    if dq_cache.dtype != np.uint16 or not dq_cache.flags.c_contiguous:
        raise TypeError("dq_cache must be contiguous uint16 bits")
    T_max = packed_cache.shape[1]
    if pos0 < 0 or pos0 + rows > T_max:
        raise ValueError("block does not fit the cache")
    lam2, nl = _lam(lam, D)
    spl = streams_per_lambda if streams_per_lambda >= 1 else 1
    for t in range(rows):
        append(np.ascontiguousarray(x[:, t]), dtype, sg, lam, group, packed_cache, scales_cache, pos0 + t, streams_per_lambda)
    for s in range(S):
        row = lam2[s // spl if nl > 1 else 0]
        dq_cache[s, pos0:pos0 + rows] = decode(packed_cache[s, pos0:pos0 + rows], scales_cache[s, pos0:pos0 + rows], sg, row,
                                               group, dtype)
