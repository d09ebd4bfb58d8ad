"""ctypes front end of the C oracle (test infrastructure, not product code).

Compiles ``lordba_oracle.c`` with gcc on first use and marshals numpy arrays.
All arithmetic lives in the C file; this module only converts array types.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lordba_oracle.c")
_SO = os.path.join(_HERE, "liblordba_oracle.so")
_lock = threading.Lock()
_lib = None

_i64 = ctypes.c_int64
_dp = ctypes.POINTER(ctypes.c_double)
_i8p = ctypes.POINTER(ctypes.c_int8)
_u32p = ctypes.POINTER(ctypes.c_uint32)


def build(force: bool = False) -> str:
    """Compile the oracle shared object if it is missing or older than its source."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_adapter_forward.restype = ctypes.c_int
        lib.oracle_adapter_forward.argtypes = [_dp, _i8p, _i8p, _dp, _dp, _dp, _dp,
                                               _i64, _i64, _i64, _i64, _i64, _i64]
        lib.oracle_adapter_forward_ell.restype = ctypes.c_int
        lib.oracle_adapter_forward_ell.argtypes = [_dp, _i8p, _i8p, _dp, _dp, _dp, _dp,
                                                   _i64, _i64, _i64, _i64, _i64, _i64, _i64]
        lib.oracle_packed_words.restype = _i64
        lib.oracle_packed_words.argtypes = [_i64, _i64, ctypes.c_int]
        lib.oracle_pack_signs.restype = ctypes.c_int
        lib.oracle_pack_signs.argtypes = [_i8p, _i64, _i64, ctypes.c_int, _u32p]
        lib.oracle_unpack_signs.restype = ctypes.c_int
        lib.oracle_unpack_signs.argtypes = [_u32p, _i64, _i64, ctypes.c_int, _i8p]
        lib.oracle_adapter_bits.restype = _i64
        lib.oracle_adapter_bits.argtypes = [_i64, _i64, _i64, _i64]
        lib.oracle_lora_fp16_bits.restype = _i64
        lib.oracle_lora_fp16_bits.argtypes = [_i64, _i64, _i64]
        lib.oracle_bpw_tot.restype = ctypes.c_double
        lib.oracle_bpw_tot.argtypes = [_i64, _i64, _i64, _i64, _i64]
        lib.oracle_bandwidth_ratio.restype = ctypes.c_double
        lib.oracle_bandwidth_ratio.argtypes = [_i64, _i64, _i64]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def widen_bf16(bits_u16: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the exact float64 values they denote."""
    b = np.ascontiguousarray(bits_u16, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _f64(a, shape=None):
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None and a.shape != tuple(shape):
        raise ValueError("expected shape %r, got %r" % (tuple(shape), a.shape))
    return a


def _i8(a, shape):
    a = np.ascontiguousarray(a, dtype=np.int8)
    if a.shape != tuple(shape):
        raise ValueError("expected shape %r, got %r" % (tuple(shape), a.shape))
    return a


def adapter_forward(x, A_sign, B_sign, s_in, s_r, s_out, y) -> np.ndarray:
    """Return y + adapter(x) in float64 (inputs are widened, never rounded)."""
    x = _f64(x)
    T, d_in = x.shape
    r = np.asarray(A_sign).shape[0]
    d_out = np.asarray(B_sign).shape[0]
    A = _i8(A_sign, (r, d_in))
    B = _i8(B_sign, (d_out, r))
    out = _f64(y, (T, d_out)).copy()
    rc = _load().oracle_adapter_forward(
        x.ctypes.data_as(_dp), A.ctypes.data_as(_i8p), B.ctypes.data_as(_i8p),
        _f64(s_in, (d_in,)).ctypes.data_as(_dp), _f64(s_r, (r,)).ctypes.data_as(_dp),
        _f64(s_out, (d_out,)).ctypes.data_as(_dp), out.ctypes.data_as(_dp),
        T, d_in, d_out, r, d_in, d_out)
    if rc != 0:
        raise RuntimeError("oracle_adapter_forward failed (%d)" % rc)
    return out


def adapter_forward_ell(x, A_sign, B_sign, s_in, s_r, s_out, y) -> np.ndarray:
    """Multi-envelope form: s_in (ell,d_in), s_r (ell,r), s_out (ell,d_out)."""
    x = _f64(x)
    T, d_in = x.shape
    r = np.asarray(A_sign).shape[0]
    d_out = np.asarray(B_sign).shape[0]
    s_in = _f64(s_in)
    ell = s_in.shape[0]
    A = _i8(A_sign, (r, d_in))
    B = _i8(B_sign, (d_out, r))
    out = _f64(y, (T, d_out)).copy()
    rc = _load().oracle_adapter_forward_ell(
        x.ctypes.data_as(_dp), A.ctypes.data_as(_i8p), B.ctypes.data_as(_i8p),
        _f64(s_in, (ell, d_in)).ctypes.data_as(_dp), _f64(s_r, (ell, r)).ctypes.data_as(_dp),
        _f64(s_out, (ell, d_out)).ctypes.data_as(_dp), out.ctypes.data_as(_dp),
        T, d_in, d_out, r, ell, d_in, d_out)
    if rc != 0:
        raise RuntimeError("oracle_adapter_forward_ell failed (%d)" % rc)
    return out


def packed_words(rows: int, cols: int, role: int) -> int:
    return int(_load().oracle_packed_words(rows, cols, role))


def pack_signs(signs, role: int) -> np.ndarray:
    s = np.ascontiguousarray(signs, dtype=np.int8)
    rows, cols = s.shape
    out = np.empty(max(packed_words(rows, cols, role), 0), dtype=np.uint32)
    rc = _load().oracle_pack_signs(s.ctypes.data_as(_i8p), rows, cols, role,
                                   out.ctypes.data_as(_u32p))
    if rc != 0:
        raise RuntimeError("oracle_pack_signs failed (%d)" % rc)
    return out


def unpack_signs(packed, rows: int, cols: int, role: int) -> np.ndarray:
    p = np.ascontiguousarray(packed, dtype=np.uint32)
    if p.size != packed_words(rows, cols, role):
        raise ValueError("wrong number of packed words")
    out = np.empty((rows, cols), dtype=np.int8)
    rc = _load().oracle_unpack_signs(p.ctypes.data_as(_u32p), rows, cols, role,
                                     out.ctypes.data_as(_i8p))
    if rc != 0:
        raise RuntimeError("oracle_unpack_signs failed (%d)" % rc)
    return out


def adapter_bits(d_in: int, d_out: int, r: int, ell: int = 1) -> int:
    return int(_load().oracle_adapter_bits(d_in, d_out, r, ell))


def lora_fp16_bits(d_in: int, d_out: int, r0: int) -> int:
    return int(_load().oracle_lora_fp16_bits(d_in, d_out, r0))


def bpw_tot(d_in: int, d_out: int, r: int, ell: int, r0: int) -> float:
    return float(_load().oracle_bpw_tot(d_in, d_out, r, ell, r0))


def bandwidth_ratio(d_in: int, d_out: int, r0: int) -> float:
    return float(_load().oracle_bandwidth_ratio(d_in, d_out, r0))
