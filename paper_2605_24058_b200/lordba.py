"""Thin ctypes binding of liblordba.so: argument marshalling only.

Every function has the name of the C entry point it calls (see
``include/lordba.h``).  torch supplies device memory and the current stream;
all arithmetic happens in the CUDA kernels.  There is no CPU fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblordba.so")

F32, BF16, F16 = 0, 1, 2
VARIANT_AUTO, VARIANT_FMA, VARIANT_TC, VARIANT_MMA = 0, 1, 2, 3
PROJ_OVERLAP = 1
PROJ_SCALES_F16 = 2
PROJ_X_READY = 4
MAX_ELL = 8
MAX_PROJS = 4096
FIT_ALPHA, FIT_BETA, FIT_GAMMA, FIT_ALL = 1, 2, 4, 7


def proj_ell(ell: int) -> int:
    """Flag field for an adapter with ``ell`` envelopes (mirror of LORDBA_PROJ_ELL)."""
    return ((ell - 1) & 0xF) << 8

_i64 = ctypes.c_int64
_vp = ctypes.c_void_p


class LordbaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class Proj(ctypes.Structure):
    """Mirror of ``lordba_proj``."""
    _fields_ = [("x", _vp), ("packed_A", _vp), ("packed_B", _vp), ("s_in", _vp), ("s_r", _vp),
                ("s_out", _vp), ("y", _vp), ("d_in", _i64), ("d_out", _i64), ("ldx", _i64),
                ("ldy", _i64), ("r", ctypes.c_int32), ("flags", ctypes.c_int32)]


_SIGNATURES = {
    "lordba_packed_words": (_i64, [_i64, _i64, ctypes.c_int]),
    "lordba_pack_signs": (ctypes.c_int, [_vp, _i64, _i64, ctypes.c_int, _vp, _vp]),
    "lordba_unpack_signs": (ctypes.c_int, [_vp, _i64, _i64, ctypes.c_int, _vp, _vp]),
    "lordba_scales_from_f16": (ctypes.c_int, [_vp, _vp, _i64, _vp]),
    "lordba_adapter_forward": (ctypes.c_int, [_vp] * 7 + [_i64, _i64, _i64, ctypes.c_int, _vp]),
    "lordba_adapter_forward_f32": (ctypes.c_int, [_vp] * 7 + [_i64, _i64, _i64, ctypes.c_int, _vp]),
    "lordba_adapter_forward_ell": (ctypes.c_int, [_vp] * 7 + [_i64, _i64, _i64, ctypes.c_int, ctypes.c_int,
                                                  ctypes.c_int, _vp]),
    "lordba_adapter_forward_ex": (ctypes.c_int, [ctypes.POINTER(Proj), _i64, ctypes.c_int, _vp]),
    "lordba_adapter_forward_batched": (ctypes.c_int, [ctypes.POINTER(Proj), ctypes.c_int, _i64,
                                                       ctypes.c_int, _vp]),
    "lordba_adapter_forward_segments": (ctypes.c_int, [ctypes.POINTER(Proj), ctypes.POINTER(_i64), ctypes.c_int,
                                                       ctypes.c_int, _vp]),
    "lordba_host_workspace_bytes": (ctypes.c_size_t, [_i64, _i64, _i64, ctypes.c_int]),
    "lordba_adapter_forward_host": (ctypes.c_int, [_vp] * 7 + [_i64, _i64, _i64, ctypes.c_int,
                                                               ctypes.c_int, _vp, ctypes.c_size_t, _vp]),
    "lordba_adapter_forward_host_static": (ctypes.c_int, [_vp] * 7 + [_i64, _i64, _i64, ctypes.c_int,
                                                                      ctypes.c_int, _vp]),
    "lordba_query_variant": (ctypes.c_int, [ctypes.POINTER(Proj), ctypes.c_int, _i64, ctypes.POINTER(_i64),
                                            ctypes.c_int, ctypes.POINTER(ctypes.c_int)]),
    "lordba_plan_bytes": (ctypes.c_size_t, [ctypes.POINTER(Proj), ctypes.c_int, _i64, ctypes.POINTER(_i64),
                                            ctypes.c_int]),
    "lordba_plan_init": (ctypes.c_int, [_vp, ctypes.c_size_t, ctypes.POINTER(Proj), ctypes.c_int, _i64,
                                        ctypes.POINTER(_i64), ctypes.c_int]),
    "lordba_adapter_forward_planned": (ctypes.c_int, [_vp, _vp]),
    "lordba_plan_launches": (ctypes.c_int, [_vp]),
    "lordba_fit_workspace_bytes": (ctypes.c_size_t, [_i64, _i64, ctypes.c_int]),
    "lordba_fit_scales": (ctypes.c_int, [_vp, _i64, _vp, _vp, _vp, _vp, _vp, _i64, _i64, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int, _vp, ctypes.c_size_t, _vp]),
    "lordba_adapter_bits": (_i64, [_i64, _i64, ctypes.c_int, ctypes.c_int]),
    "lordba_set_variant": (ctypes.c_int, [ctypes.c_int]),
    "lordba_get_variant": (ctypes.c_int, []),
    "lordba_device_status": (ctypes.c_int, [ctypes.POINTER(ctypes.c_int), _vp]),
    "lordba_launch_count": (_i64, []),
    "lordba_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "lordba_version": (ctypes.c_char_p, []),
}

_lib = None


def bind(path: str) -> ctypes.CDLL:
    """Open a build of the library and declare the signatures of its entry points."""
    lib = ctypes.CDLL(path)
    for name, (res, args) in _SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


def load() -> ctypes.CDLL:
    """Load liblordba.so (built by ``paper_2605_24058_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("liblordba.so is not built (%s); run "
                               "`python -m paper_2605_24058_b200.build`" % LIB_PATH)
        _lib = bind(LIB_PATH)
    return _lib


def exported_symbols() -> Sequence[str]:
    return tuple(_SIGNATURES)


def status_string(status: int) -> str:
    return load().lordba_status_string(int(status)).decode()


def version() -> str:
    return load().lordba_version().decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise LordbaError(status, where)


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float16:
        return F16
    raise TypeError("x and y must be float32, bfloat16 or float16, got %s" % t.dtype)


def _need_cuda(*tensors: torch.Tensor) -> None:
    for t in tensors:
        if not t.is_cuda:
            raise ValueError("expected a CUDA tensor")


def packed_words(rows: int, cols: int, role: int) -> int:
    return int(load().lordba_packed_words(rows, cols, role))


def pack_signs(signs: torch.Tensor, role: int, stream=None) -> torch.Tensor:
    """int8 sign matrix on the device -> packed int32 words on the device."""
    _need_cuda(signs)
    if signs.dtype != torch.int8 or signs.dim() != 2 or not signs.is_contiguous():
        raise ValueError("signs must be a contiguous 2-D int8 tensor")
    rows, cols = signs.shape
    n = packed_words(rows, cols, role)
    if n < 0:
        raise LordbaError(2, "lordba_packed_words")
    packed = torch.empty(n, dtype=torch.int32, device=signs.device)
    _check(load().lordba_pack_signs(signs.data_ptr(), rows, cols, role, packed.data_ptr(),
                                    _stream(stream)), "lordba_pack_signs")
    return packed


def unpack_signs(packed: torch.Tensor, rows: int, cols: int, role: int, stream=None) -> torch.Tensor:
    _need_cuda(packed)
    if packed.dtype != torch.int32 or not packed.is_contiguous():
        raise ValueError("packed must be a contiguous int32 tensor")
    if packed.numel() != packed_words(rows, cols, role):
        raise ValueError("wrong number of packed words")
    signs = torch.empty((rows, cols), dtype=torch.int8, device=packed.device)
    _check(load().lordba_unpack_signs(packed.data_ptr(), rows, cols, role, signs.data_ptr(),
                                      _stream(stream)), "lordba_unpack_signs")
    return signs


def scales_from_f16(scales: torch.Tensor, stream=None) -> torch.Tensor:
    """float16 scales of an exported adapter (device) -> the float32 tensor the forward calls take."""
    _need_cuda(scales)
    if scales.dtype != torch.float16 or not scales.is_contiguous():
        raise ValueError("scales must be a contiguous float16 tensor")
    out = torch.empty(scales.shape, dtype=torch.float32, device=scales.device)
    _check(load().lordba_scales_from_f16(scales.data_ptr(), out.data_ptr(), scales.numel(), _stream(stream)),
           "lordba_scales_from_f16")
    return out


def make_proj(x, packed_A, packed_B, s_in, s_r, s_out, y, r: int, flags: int = 0) -> Proj:
    """Fill a ``lordba_proj`` from 2-D (possibly row-strided) x, y and 1-D parameter tensors."""
    _need_cuda(x, packed_A, packed_B, s_in, s_r, s_out, y)
    if x.dim() != 2 or y.dim() != 2 or x.shape[0] != y.shape[0]:
        raise ValueError("x must be (T, d_in) and y (T, d_out)")
    if x.dtype != y.dtype:
        raise TypeError("x and y must have the same dtype")
    if (x.shape[1] > 1 and x.stride(1) != 1) or (y.shape[1] > 1 and y.stride(1) != 1):
        raise ValueError("x and y rows must be contiguous")
    for s in (s_in, s_r, s_out):
        if s.dtype != torch.float32 or not s.is_contiguous():
            raise TypeError("scales must be contiguous float32")
    d_in, d_out = x.shape[1], y.shape[1]
    # 2-D scales (ell, d) make a multi-envelope adapter: the envelope count goes into the flags
    ell = s_in.shape[0] if s_in.dim() == 2 else 1
    if ell > 1:
        flags |= proj_ell(ell)
    if s_in.numel() != ell * d_in or s_out.numel() != ell * d_out or s_r.numel() != ell * r:
        raise ValueError("scale vector sizes do not match d_in / r / d_out")
    if packed_A.numel() != packed_words(r, d_in, 0) or packed_B.numel() != packed_words(d_out, r, 1):
        raise ValueError("packed carrier sizes do not match (r, d_in, d_out)")
    ldx = x.stride(0) if x.shape[0] > 1 else max(d_in, x.stride(0))
    ldy = y.stride(0) if y.shape[0] > 1 else max(d_out, y.stride(0))
    return Proj(x.data_ptr(), packed_A.data_ptr(), packed_B.data_ptr(), s_in.data_ptr(),
                s_r.data_ptr(), s_out.data_ptr(), y.data_ptr(), d_in, d_out, ldx, ldy, r, flags)


def adapter_forward(x, packed_A, packed_B, s_in, s_r, s_out, y, r: int, stream=None,
                    overlap: bool = False, scales_f16: bool = False, x_ready: bool = False) -> None:
    """y += adapter(x) in place, through lordba_adapter_forward{,_f32} (dense rows)
    or lordba_adapter_forward_ex (row-strided x / y, float16, or a flag: overlap=True is the
    caller's promise LORDBA_PROJ_OVERLAP that this call is independent of the run of calls before
    it, scales_f16=True the statement LORDBA_PROJ_SCALES_F16 that s_in holds float16 values,
    x_ready=True the promise LORDBA_PROJ_X_READY that only y can still be in the making)."""
    flags = ((PROJ_OVERLAP if overlap else 0) | (PROJ_SCALES_F16 if scales_f16 else 0) |
             (PROJ_X_READY if x_ready else 0))
    p = make_proj(x, packed_A, packed_B, s_in, s_r, s_out, y, r, flags)
    T = x.shape[0]
    lib = load()
    dense = x.is_contiguous() and y.is_contiguous() and flags == 0
    if dense and x.dtype == torch.bfloat16:
        rc = lib.lordba_adapter_forward(p.x, p.packed_A, p.packed_B, p.s_in, p.s_r, p.s_out, p.y,
                                        T, p.d_in, p.d_out, r, _stream(stream))
        _check(rc, "lordba_adapter_forward")
    elif dense and x.dtype == torch.float32:
        rc = lib.lordba_adapter_forward_f32(p.x, p.packed_A, p.packed_B, p.s_in, p.s_r, p.s_out,
                                            p.y, T, p.d_in, p.d_out, r, _stream(stream))
        _check(rc, "lordba_adapter_forward_f32")
    else:
        adapter_forward_ex(p, T, _dtype_code(x), stream)


def adapter_forward_ell(x, packed_A, packed_B, s_in, s_r, s_out, y, r: int, stream=None) -> None:
    """Multi-envelope adapter (Eq. 4): s_in (ell, d_in), s_r (ell, r), s_out (ell, d_out); dense x, y."""
    _need_cuda(x, packed_A, packed_B, s_in, s_r, s_out, y)
    if s_in.dim() != 2 or s_r.dim() != 2 or s_out.dim() != 2 or not (s_in.shape[0] == s_r.shape[0] == s_out.shape[0]):
        raise ValueError("scales must be (ell, d_in), (ell, r), (ell, d_out)")
    for s in (s_in, s_r, s_out):
        if s.dtype != torch.float32 or not s.is_contiguous():
            raise TypeError("scales must be contiguous float32")
    if not (x.is_contiguous() and y.is_contiguous()) or x.dtype != y.dtype:
        raise ValueError("x and y must be dense and of one dtype")
    ell = s_in.shape[0]
    T, d_in = x.shape
    d_out = y.shape[1]
    if s_in.shape[1] != d_in or s_out.shape[1] != d_out or s_r.shape[1] != r:
        raise ValueError("scale shapes do not match (d_in, r, d_out)")
    rc = load().lordba_adapter_forward_ell(x.data_ptr(), packed_A.data_ptr(), packed_B.data_ptr(),
                                           s_in.data_ptr(), s_r.data_ptr(), s_out.data_ptr(),
                                           y.data_ptr(), T, d_in, d_out, r, ell, _dtype_code(x),
                                           _stream(stream))
    _check(rc, "lordba_adapter_forward_ell")


def adapter_forward_ex(p: Proj, T: int, dtype: int, stream=None) -> None:
    _check(load().lordba_adapter_forward_ex(ctypes.byref(p), T, dtype, _stream(stream)),
           "lordba_adapter_forward_ex")


def adapter_forward_batched(projs: Sequence[Proj], T: int, dtype: int, stream=None) -> None:
    arr = (Proj * len(projs))(*projs)
    _check(load().lordba_adapter_forward_batched(arr, len(projs), T, dtype, _stream(stream)),
           "lordba_adapter_forward_batched")


def adapter_forward_segments(segs: Sequence[Proj], tokens: Sequence[int], dtype: int, stream=None) -> None:
    """Multi-adapter batch: segment i = tokens[i] rows starting at segs[i].x / .y with its own adapter."""
    if len(segs) != len(tokens):
        raise ValueError("one token count per segment")
    arr = (Proj * len(segs))(*segs)
    tok = (_i64 * len(tokens))(*[int(t) for t in tokens])
    _check(load().lordba_adapter_forward_segments(arr, tok, len(segs), dtype, _stream(stream)),
           "lordba_adapter_forward_segments")


def _call_args(projs: Sequence[Proj], tokens):
    """(array of Proj, n, T, pointer to per-projection token counts or NULL) for the entry points
    that take either one T for all projections (tokens: an int) or one count each (a sequence)."""
    arr = (Proj * len(projs))(*projs)
    if isinstance(tokens, int):
        return arr, len(projs), tokens, None
    if len(tokens) != len(projs):
        raise ValueError("one token count per projection")
    return arr, len(projs), 0, (_i64 * len(tokens))(*[int(t) for t in tokens])


def query_variant(projs: Sequence[Proj], tokens, dtype: int) -> Sequence[int]:
    """Kernel family per projection (VARIANT_FMA / _TC / _MMA, 0 for one without rows) that a batched
    call (tokens: one int) or a segmented call (tokens: one count per projection) would use."""
    arr, n, T, tok = _call_args(projs, tokens)
    out = (ctypes.c_int * max(n, 1))()
    _check(load().lordba_query_variant(arr, n, T, tok, dtype, out), "lordba_query_variant")
    return [int(out[i]) for i in range(n)]


class Plan:
    """Caller-owned host storage of a prepared call (64-byte aligned)."""

    def __init__(self, nbytes: int):
        self._raw = (ctypes.c_char * (nbytes + 64))()
        base = ctypes.addressof(self._raw)
        self.ptr = (base + 63) // 64 * 64
        self.nbytes = nbytes

    def launches(self) -> int:
        return int(load().lordba_plan_launches(self.ptr))


def plan_init(projs: Sequence[Proj], tokens, dtype: int) -> Plan:
    """lordba_plan_bytes + lordba_plan_init: prepare a batched (tokens: an int) or segmented call."""
    arr, n, T, tok = _call_args(projs, tokens)
    lib = load()
    nbytes = int(lib.lordba_plan_bytes(arr, n, T, tok, dtype))
    if nbytes == 0:
        # ask lordba_plan_init for the status of the same arguments
        scratch = Plan(64)
        _check(lib.lordba_plan_init(scratch.ptr, 64, arr, n, T, tok, dtype) or 1, "lordba_plan_init")
    plan = Plan(nbytes)
    _check(lib.lordba_plan_init(plan.ptr, nbytes, arr, n, T, tok, dtype), "lordba_plan_init")
    return plan


def adapter_forward_planned(plan: Plan, stream=None) -> None:
    _check(load().lordba_adapter_forward_planned(plan.ptr, _stream(stream)), "lordba_adapter_forward_planned")


def host_workspace_bytes(T: int, d_in: int, d_out: int, dtype: int) -> int:
    return int(load().lordba_host_workspace_bytes(T, d_in, d_out, dtype))


def adapter_forward_host(x_host, packed_A, packed_B, s_in, s_r, s_out, y_host, r: int,
                         workspace: torch.Tensor, stream=None) -> None:
    """Host x / y (CPU tensors, ideally pinned), device parameters and workspace."""
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host and y_host must be CPU tensors")
    if not (x_host.is_contiguous() and y_host.is_contiguous()):
        raise ValueError("host buffers must be contiguous")
    _need_cuda(packed_A, packed_B, s_in, s_r, s_out, workspace)
    T, d_in = x_host.shape
    d_out = y_host.shape[1]
    rc = load().lordba_adapter_forward_host(
        x_host.data_ptr(), packed_A.data_ptr(), packed_B.data_ptr(), s_in.data_ptr(),
        s_r.data_ptr(), s_out.data_ptr(), y_host.data_ptr(), T, d_in, d_out, r,
        _dtype_code(x_host), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
        _stream(stream))
    _check(rc, "lordba_adapter_forward_host")


STATIC_SCRATCH_BYTES = 8 << 20


def adapter_forward_host_static(x_host, packed_A, packed_B, s_in, s_r, s_out, y_host, r: int,
                                stream=None) -> None:
    """Host x / y like ``adapter_forward_host``, but the device staging area is the library's own
    built-in buffer (``STATIC_SCRATCH_BYTES``): for callers that may not allocate device memory.
    Calls on one device share that buffer and must not overlap on the GPU."""
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host and y_host must be CPU tensors")
    if not (x_host.is_contiguous() and y_host.is_contiguous()):
        raise ValueError("host buffers must be contiguous")
    _need_cuda(packed_A, packed_B, s_in, s_r, s_out)
    T, d_in = x_host.shape
    d_out = y_host.shape[1]
    rc = load().lordba_adapter_forward_host_static(
        x_host.data_ptr(), packed_A.data_ptr(), packed_B.data_ptr(), s_in.data_ptr(),
        s_r.data_ptr(), s_out.data_ptr(), y_host.data_ptr(), T, d_in, d_out, r,
        _dtype_code(x_host), _stream(stream))
    _check(rc, "lordba_adapter_forward_host_static")


def fit_workspace_bytes(d_in: int, d_out: int, r: int) -> int:
    return int(load().lordba_fit_workspace_bytes(d_in, d_out, r))


def fit_scales(target, packed_A, packed_B, s_in, s_r, s_out, r: int, sweeps: int = 1, axes: int = FIT_ALL,
               workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """Closed-form scale sweeps (s_in, then s_r, then s_out) against the dense float32 target
    (d_in x d_out, rows contiguous) with the packed carriers fixed; the three scale tensors are
    updated in place.  workspace: a uint8 CUDA tensor of fit_workspace_bytes(), made here if absent."""
    _need_cuda(target, packed_A, packed_B, s_in, s_r, s_out)
    if target.dtype != torch.float32 or target.dim() != 2 or (target.shape[1] > 1 and target.stride(1) != 1):
        raise ValueError("target must be a 2-D float32 tensor with contiguous rows")
    d_in, d_out = target.shape
    for s, n in ((s_in, d_in), (s_r, r), (s_out, d_out)):
        if s.dtype != torch.float32 or not s.is_contiguous() or s.numel() != n:
            raise ValueError("scales must be contiguous float32 vectors of d_in, r and d_out entries")
    if packed_A.numel() != packed_words(r, d_in, 0) or packed_B.numel() != packed_words(d_out, r, 1):
        raise ValueError("packed carrier sizes do not match (r, d_in, d_out)")
    need = fit_workspace_bytes(d_in, d_out, r)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=target.device)
    ld = target.stride(0) if d_in > 1 else max(d_out, target.stride(0))
    rc = load().lordba_fit_scales(target.data_ptr(), ld, packed_A.data_ptr(), packed_B.data_ptr(), s_in.data_ptr(),
                                  s_r.data_ptr(), s_out.data_ptr(), d_in, d_out, r, sweeps, axes,
                                  workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(rc, "lordba_fit_scales")


def adapter_bits(d_in: int, d_out: int, r: int, ell: int = 1) -> int:
    return int(load().lordba_adapter_bits(d_in, d_out, r, ell))


def set_variant(variant: int) -> None:
    _check(load().lordba_set_variant(variant), "lordba_set_variant")


def get_variant() -> int:
    return int(load().lordba_get_variant())


def device_status(stream=None) -> int:
    """Synchronise the stream and return the device status word (0 = no bounded wait gave up)."""
    code = ctypes.c_int(0)
    rc = load().lordba_device_status(ctypes.byref(code), _stream(stream))
    if rc not in (0, 5):
        raise LordbaError(rc, "lordba_device_status")
    return int(code.value)


def launch_count() -> int:
    return int(load().lordba_launch_count())
