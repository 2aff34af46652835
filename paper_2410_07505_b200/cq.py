"""Thin binding of the C-ABI library ``libcq.so`` (argument marshalling only).

Every function has the name of the C entry point without the ``cq_`` prefix and does no
arithmetic of its own: torch supplies device memory and the current stream, ctypes passes raw
pointers.  A missing or unloadable library is an error -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcq.so")

CQ_F16, CQ_BF16, CQ_F32 = 0, 1, 2
_DT = {torch.float16: CQ_F16, torch.bfloat16: CQ_BF16, torch.float32: CQ_F32}

EXPORTS = (
    "cq_version", "cq_status_string", "cq_absmax_rows", "cq_absmax_cols", "cq_absmax_rows_cols",
    "cq_workspace_bytes", "cq_quantize_act", "cq_host_scratch_bytes", "cq_quantize_act_host",
    "cq_dequantize", "cq_kernel_count", "cq_kernel_count_x", "cq_quantize_weight_per_channel",
    "cq_set_tuning", "cq_set_timing_events", "cq_quantize_act_noalloc",
    "cq_quantize_weight_groupwise", "cq_case_indicators", "cq_remove_kernel", "cq_stage_fault",
    "cq_vector_max", "cq_quantize_act_given",
)


class CQError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


_lib = None


def lib() -> C.CDLL:
    """Load libcq.so (built by ``paper_2410_07505_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2410_07505_b200.build`")
        L = C.CDLL(LIB_PATH)
        i64, vp, dbl, ci = C.c_int64, C.c_void_p, C.c_double, C.c_int
        L.cq_version.restype = ci
        L.cq_status_string.restype = C.c_char_p
        L.cq_status_string.argtypes = [ci]
        L.cq_absmax_rows.argtypes = [vp, ci, i64, i64, i64, vp, vp]
        L.cq_absmax_cols.argtypes = [vp, ci, i64, i64, i64, vp, vp]
        L.cq_absmax_rows_cols.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp]
        L.cq_workspace_bytes.restype = C.c_size_t
        L.cq_workspace_bytes.argtypes = [i64, i64]
        L.cq_quantize_act.argtypes = [vp, ci, i64, i64, i64, dbl, ci, vp, vp, vp, vp, vp, vp, ci, vp, vp,
                                      C.c_size_t, vp]
        L.cq_vector_max.argtypes = [vp, vp, i64, vp]
        L.cq_quantize_act_given.argtypes = [vp, ci, i64, i64, i64, dbl, ci, vp, vp, vp, vp, vp, vp, ci, vp, vp,
                                            C.c_size_t, vp]
        L.cq_quantize_act_noalloc.argtypes = [vp, ci, i64, i64, i64, dbl, ci, vp, vp, vp, vp, vp, vp, ci, vp, vp]
        L.cq_host_scratch_bytes.restype = C.c_size_t
        L.cq_host_scratch_bytes.argtypes = [i64, i64, ci, ci, ci, ci]
        L.cq_quantize_act_host.argtypes = [vp, ci, i64, i64, i64, dbl, ci, vp, vp, vp, vp, vp, vp, ci, vp, vp,
                                           C.c_size_t, vp]
        L.cq_dequantize.argtypes = [vp, ci, i64, i64, vp, vp, vp, ci, vp]
        L.cq_kernel_count.argtypes = [vp, ci, i64, i64, vp, vp]
        L.cq_kernel_count_x.argtypes = [vp, ci, i64, i64, i64, dbl, ci, vp, vp, vp, vp, C.c_size_t, vp]
        L.cq_quantize_weight_per_channel.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, vp, ci, vp, vp]
        L.cq_quantize_weight_groupwise.argtypes = [vp, ci, i64, i64, i64, i64, ci, vp, vp, vp, ci, vp, vp]
        L.cq_case_indicators.argtypes = [vp, vp, vp, vp, i64, i64, ci, vp, vp]
        L.cq_remove_kernel.argtypes = [vp, ci, i64, i64, i64, dbl, ci, C.c_float, vp, vp, vp, C.c_size_t, vp]
        L.cq_stage_fault.argtypes = [vp]
        L.cq_set_tuning.argtypes = [C.c_char_p, ci]
        L.cq_set_timing_events.argtypes = [vp, vp]
        for name in EXPORTS:
            if name not in ("cq_status_string", "cq_workspace_bytes", "cq_host_scratch_bytes"):
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def version() -> int:
    return int(lib().cq_version())


def status_string(status: int) -> str:
    return lib().cq_status_string(int(status)).decode()


def set_tuning(key: str, value: int) -> None:
    _check(lib().cq_set_tuning(key.encode(), int(value)), "cq_set_tuning")


def set_timing_events(before: "torch.cuda.Event | None", after: "torch.cuda.Event | None") -> None:
    """Have quantize_act record two (already created) CUDA events around its quantize pass."""
    if before is None or after is None:
        lib().cq_set_timing_events(None, None)
    else:
        lib().cq_set_timing_events(C.c_void_p(before.cuda_event), C.c_void_p(after.cuda_event))


def _check(status: int, where: str) -> None:
    if status != 0:
        raise CQError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream():
    """The current CUDA stream of the current device as a void* (the raw handle where torch exposes it
    directly: several times cheaper than building a Stream object on every call)."""
    if _raw_stream is not None:
        return C.c_void_p(_raw_stream(torch.cuda.current_device()))
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _matrix_args(X: torch.Tensor):
    if X.dim() != 2 or X.dtype not in (torch.float16, torch.bfloat16):
        raise TypeError("expected a 2-D float16 / bfloat16 tensor")
    if not X.is_cuda:
        raise TypeError("expected a CUDA tensor")
    T, I = X.shape
    if I > 0 and T > 0 and X.stride(1) != 1:
        raise ValueError("columns must be contiguous")
    ld = X.stride(0) if T > 1 else max(I, 1)
    return T, I, ld


def workspace_bytes(T: int, I: int) -> int:
    return int(lib().cq_workspace_bytes(T, I))


def _workspace(T, I, device):
    return torch.empty(workspace_bytes(T, I), dtype=torch.uint8, device=device)


# ----------------------------------------------------------------------------- absmax
def _f32_vector(out, n: int, device, what: str) -> torch.Tensor:
    if out is None:
        return torch.empty(n, dtype=torch.float32, device=device)
    if out.dtype != torch.float32 or out.numel() != n or not out.is_contiguous() or out.device != device:
        raise ValueError(f"{what} must be a contiguous float32 vector of {n} elements on {device}")
    return out


def _counts(out, n: int, device, what: str) -> torch.Tensor:
    """An int64 device tensor of n elements (a scalar for n == 1) that receives 64-bit counts."""
    if out is None:
        return torch.zeros((), dtype=torch.int64, device=device) if n == 1 else torch.zeros(n, dtype=torch.int64, device=device)
    if out.dtype != torch.int64 or out.numel() != n or not out.is_contiguous() or out.device != device:
        raise ValueError(f"{what} must be a contiguous int64 tensor of {n} element(s) on {device}")
    return out


def absmax_rows(X: torch.Tensor, *, out: torch.Tensor | None = None) -> torch.Tensor:
    T, I, ld = _matrix_args(X)
    t = _f32_vector(out, T, X.device, "out")
    _check(lib().cq_absmax_rows(_ptr(X), _DT[X.dtype], T, I, ld, _ptr(t), _stream()), "cq_absmax_rows")
    return t


def absmax_cols(X: torch.Tensor, *, out: torch.Tensor | None = None) -> torch.Tensor:
    T, I, ld = _matrix_args(X)
    c = _f32_vector(out, I, X.device, "out")
    _check(lib().cq_absmax_cols(_ptr(X), _DT[X.dtype], T, I, ld, _ptr(c), _stream()), "cq_absmax_cols")
    return c


def absmax_rows_cols(X: torch.Tensor, *, workspace: torch.Tensor | None = None, out=None):
    """(t, c) from one read of X.  With a `workspace` (>= workspace_bytes(T, I)) the first pass of
    cq_quantize_act is used (partial maxima in the workspace, no atomics: faster on large matrices);
    without one, cq_absmax_rows_cols.  `out` = (t, c) tensors to fill."""
    T, I, ld = _matrix_args(X)
    t = _f32_vector(out[0] if out is not None else None, T, X.device, "out[0]")
    c = _f32_vector(out[1] if out is not None else None, I, X.device, "out[1]")
    if workspace is None:
        _check(lib().cq_absmax_rows_cols(_ptr(X), _DT[X.dtype], T, I, ld, _ptr(t), _ptr(c), _stream()),
               "cq_absmax_rows_cols")
    else:
        # alpha = 1 keeps the scale-vector step free of pow; no output but t and c is requested
        _check(lib().cq_quantize_act(_ptr(X), _DT[X.dtype], T, I, ld, 1.0, 8, _ptr(t), _ptr(c), None, None, None, None,
                                     _DT[X.dtype], None, _ptr(workspace), workspace.numel(), _stream()),
               "cq_quantize_act")
    return t, c


# ----------------------------------------------------------------------------- quantize
@dataclass
class ActQuant:
    t: torch.Tensor | None
    c: torch.Tensor | None
    row_scale: torch.Tensor | None
    col_scale: torch.Tensor | None
    codes: torch.Tensor | None        # int8 [T, I] or uint8 [T, I/2]
    deq: torch.Tensor | None
    zero_count: torch.Tensor | None   # uint64 scalar stored as int64 on the device
    bits: int

    def kernel_proportion(self) -> float:
        n = self.t.numel() * self.c.numel()
        return int(self.zero_count.item()) / n if n else 0.0


class ActBuffers:
    """Pre-allocated outputs and workspace for repeated calls on one shape."""

    def __init__(self, T, I, dtype, bits, *, codes=True, deq=True, deq_dtype=None, count=True, device="cuda"):
        dev = torch.device(device)
        self.T, self.I, self.bits = T, I, bits
        self.t = torch.empty(T, dtype=torch.float32, device=dev)
        self.c = torch.empty(I, dtype=torch.float32, device=dev)
        self.row_scale = torch.empty(T, dtype=torch.float32, device=dev)
        self.col_scale = torch.empty(I, dtype=torch.float32, device=dev)
        self.codes = None
        if codes:
            self.codes = (torch.empty((T, I), dtype=torch.int8, device=dev) if bits == 8
                          else torch.empty((T, I // 2), dtype=torch.uint8, device=dev))
        self.deq = torch.empty((T, I), dtype=deq_dtype or dtype, device=dev) if deq else None
        self.zero_count = torch.zeros((), dtype=torch.int64, device=dev) if count else None
        self.workspace = _workspace(T, I, dev)


def _check_act_buffers(b: "ActBuffers", T: int, I: int, dtype: torch.dtype, bits: int, where: str) -> None:
    """The kernels trust the sizes they are told: refuse buffers made for another shape, dtype or bit width."""
    def bad(what):
        raise ValueError(f"{where}: buffers.{what} does not match a {T} x {I} {dtype} matrix quantized to {bits} bits")
    for name, n in (("t", T), ("c", I), ("row_scale", T), ("col_scale", I)):
        v = getattr(b, name)
        if v is not None and (v.dtype != torch.float32 or v.numel() != n or not v.is_contiguous()):
            bad(name)
    if b.codes is not None:
        want = T * I if bits == 8 else T * (I // 2)
        if b.codes.element_size() != 1 or b.codes.numel() != want or not b.codes.is_contiguous():
            bad("codes")
    if b.deq is not None and (b.deq.dtype not in (dtype, torch.float32) or b.deq.numel() != T * I or not b.deq.is_contiguous()):
        bad("deq")
    if b.zero_count is not None and (b.zero_count.dtype != torch.int64 or b.zero_count.numel() != 1):
        bad("zero_count")


def quantize_act(X: torch.Tensor, alpha: float = 0.15, bits: int = 8, *, codes: bool = True,
                 deq: bool = True, deq_dtype: torch.dtype | None = None, count: bool = True,
                 buffers: ActBuffers | None = None) -> ActQuant:
    """CrossQuant of X (tokens x channels): t, c, scale vectors, codes, dequantized X, |K(CQ)|."""
    T, I, ld = _matrix_args(X)
    if bits == 4 and I % 2:
        raise CQError(6, "cq_quantize_act")
    b = buffers or ActBuffers(T, I, X.dtype, bits, codes=codes, deq=deq, deq_dtype=deq_dtype, count=count,
                              device=X.device)
    _check_act_buffers(b, T, I, X.dtype, bits, "quantize_act")
    deq_dt = _DT[b.deq.dtype] if b.deq is not None else _DT[X.dtype]
    st = lib().cq_quantize_act(_ptr(X), _DT[X.dtype], T, I, ld, float(alpha), int(bits), _ptr(b.t), _ptr(b.c),
                               _ptr(b.row_scale), _ptr(b.col_scale), _ptr(b.codes), _ptr(b.deq), deq_dt,
                               _ptr(b.zero_count), _ptr(b.workspace), b.workspace.numel(), _stream())
    _check(st, "cq_quantize_act")
    return ActQuant(b.t, b.c, b.row_scale, b.col_scale, b.codes, b.deq, b.zero_count, bits)


NOALLOC_SCRATCH_BYTES = 8 << 20


def vector_max_(acc: torch.Tensor, v: torch.Tensor) -> torch.Tensor:
    """acc = max(acc, v) elementwise, in place (float32 device vectors of equal length)."""
    if acc.dtype != torch.float32 or v.dtype != torch.float32 or acc.numel() != v.numel():
        raise ValueError("vector_max_ wants two float32 vectors of equal length")
    _check(lib().cq_vector_max(_ptr(acc), _ptr(v), acc.numel(), _stream()), "cq_vector_max")
    return acc


def quantize_act_given(X: torch.Tensor, t: torch.Tensor, c: torch.Tensor, alpha: float = 0.15, bits: int = 8, *,
                       codes: bool = True, deq: bool = True, deq_dtype: torch.dtype | None = None, count: bool = True,
                       buffers: ActBuffers | None = None) -> ActQuant:
    """CrossQuant of a row block of a larger matrix: t are this block's row maxima, c the column maxima
    of the whole matrix (combined over all blocks).  The result's t and c are the given vectors."""
    T, I, ld = _matrix_args(X)
    if bits == 4 and I % 2:
        raise CQError(6, "cq_quantize_act_given")
    if t.dtype != torch.float32 or c.dtype != torch.float32 or t.numel() != T or c.numel() != I:
        raise ValueError("t must be float32[T] and c float32[I]")
    b = buffers or ActBuffers(T, I, X.dtype, bits, codes=codes, deq=deq, deq_dtype=deq_dtype, count=count,
                              device=X.device)
    _check_act_buffers(b, T, I, X.dtype, bits, "quantize_act_given")
    deq_dt = _DT[b.deq.dtype] if b.deq is not None else _DT[X.dtype]
    st = lib().cq_quantize_act_given(_ptr(X), _DT[X.dtype], T, I, ld, float(alpha), int(bits), _ptr(t), _ptr(c),
                                     _ptr(b.row_scale), _ptr(b.col_scale), _ptr(b.codes), _ptr(b.deq), deq_dt,
                                     _ptr(b.zero_count), _ptr(b.workspace), b.workspace.numel(), _stream())
    _check(st, "cq_quantize_act_given")
    return ActQuant(t=t, c=c, row_scale=b.row_scale, col_scale=b.col_scale, codes=b.codes, deq=b.deq,
                    zero_count=b.zero_count, bits=bits)


def quantize_act_noalloc(X: torch.Tensor, alpha: float = 0.15, bits: int = 8, *, buffers: ActBuffers) -> ActQuant:
    """quantize_act for callers that cannot allocate device memory: the scratch space is a fixed 8 MiB
    array inside the library instead of ``buffers.workspace`` (which is not used).  The caller supplies
    every output through ``buffers``; shapes whose scratch exceeds 8 MiB raise CQError (status 9).  Calls
    on one device must not overlap on the GPU -- they share the array.  The first call on a device looks
    the array up and should come before any stream capture."""
    T, I, ld = _matrix_args(X)
    b = buffers
    _check_act_buffers(b, T, I, X.dtype, bits, "quantize_act_noalloc")
    deq_dt = _DT[b.deq.dtype] if b.deq is not None else _DT[X.dtype]
    st = lib().cq_quantize_act_noalloc(_ptr(X), _DT[X.dtype], T, I, ld, float(alpha), int(bits), _ptr(b.t), _ptr(b.c),
                                       _ptr(b.row_scale), _ptr(b.col_scale), _ptr(b.codes), _ptr(b.deq), deq_dt,
                                       _ptr(b.zero_count), _stream())
    _check(st, "cq_quantize_act_noalloc")
    return ActQuant(b.t, b.c, b.row_scale, b.col_scale, b.codes, b.deq, b.zero_count, bits)


class HostBuffers:
    """Page-locked host outputs plus the device scratch of the host-buffer entry point."""

    def __init__(self, T, I, dtype, bits, *, codes=True, deq=True, deq_dtype=None, device="cuda"):
        self.T, self.I, self.bits = T, I, bits
        pin = dict(pin_memory=True)
        self.t = torch.empty(T, dtype=torch.float32, **pin)
        self.c = torch.empty(I, dtype=torch.float32, **pin)
        self.row_scale = torch.empty(T, dtype=torch.float32, **pin)
        self.col_scale = torch.empty(I, dtype=torch.float32, **pin)
        self.codes = None
        if codes:
            self.codes = (torch.empty((T, I), dtype=torch.int8, **pin) if bits == 8
                          else torch.empty((T, I // 2), dtype=torch.uint8, **pin))
        self.deq = torch.empty((T, I), dtype=deq_dtype or dtype, **pin) if deq else None
        self.zero_count = torch.zeros((), dtype=torch.int64, **pin)
        deq_dt = _DT[self.deq.dtype] if self.deq is not None else _DT[dtype]
        n = int(lib().cq_host_scratch_bytes(T, I, bits, int(codes), int(deq), deq_dt))
        self.scratch = torch.empty(n, dtype=torch.uint8, device=device)

    def d2h_bytes(self) -> int:
        n = 4 * (2 * self.T + 2 * self.I) + 8
        for x in (self.codes, self.deq):
            if x is not None:
                n += x.numel() * x.element_size()
        return n


def quantize_act_host(X_host: torch.Tensor, alpha: float = 0.15, bits: int = 8, *,
                      buffers: HostBuffers) -> ActQuant:
    """Same as quantize_act on a HOST matrix; results land in ``buffers`` (host) once the current
    stream has been synchronised."""
    if X_host.is_cuda or X_host.dim() != 2 or X_host.dtype not in (torch.float16, torch.bfloat16):
        raise TypeError("expected a 2-D float16 / bfloat16 host tensor")
    T, I = X_host.shape
    ld = X_host.stride(0) if T > 1 else max(I, 1)
    b = buffers
    deq_dt = _DT[b.deq.dtype] if b.deq is not None else _DT[X_host.dtype]
    st = lib().cq_quantize_act_host(_ptr(X_host), _DT[X_host.dtype], T, I, ld, float(alpha), int(bits),
                                    _ptr(b.t), _ptr(b.c), _ptr(b.row_scale), _ptr(b.col_scale), _ptr(b.codes),
                                    _ptr(b.deq), deq_dt, _ptr(b.zero_count), _ptr(b.scratch), b.scratch.numel(),
                                    _stream())
    _check(st, "cq_quantize_act_host")
    return ActQuant(b.t, b.c, b.row_scale, b.col_scale, b.codes, b.deq, b.zero_count, bits)


def dequantize(codes: torch.Tensor, bits: int, T: int, I: int, row_scale: torch.Tensor, col_scale: torch.Tensor,
               out_dtype: torch.dtype = torch.float32, *, out: torch.Tensor | None = None) -> torch.Tensor:
    if out is None:
        out = torch.empty((T, I), dtype=out_dtype, device=codes.device)
    elif out.dtype != out_dtype or out.numel() != T * I or not out.is_contiguous():
        raise ValueError("out must be a contiguous [T, I] tensor of out_dtype")
    if row_scale.numel() != T or col_scale.numel() != I or codes.numel() * codes.element_size() != (T * I if bits == 8 else T * (I // 2)):
        raise ValueError("codes / scale vectors do not match T, I and bits")
    _check(lib().cq_dequantize(_ptr(codes), int(bits), T, I, _ptr(row_scale), _ptr(col_scale), _ptr(out),
                               _DT[out_dtype], _stream()), "cq_dequantize")
    return out


def kernel_count(codes: torch.Tensor, bits: int, T: int, I: int, *, count: torch.Tensor | None = None) -> torch.Tensor:
    count = _counts(count, 1, codes.device, "count")
    if codes.numel() * codes.element_size() != (T * I if bits == 8 else T * (I // 2)):
        raise ValueError("codes do not match T, I and bits")
    _check(lib().cq_kernel_count(_ptr(codes), int(bits), T, I, _ptr(count), _stream()), "cq_kernel_count")
    return count


def kernel_count_x(X: torch.Tensor, alpha: float, bits: int, t: torch.Tensor, c: torch.Tensor,
                   workspace: torch.Tensor | None = None, *, count: torch.Tensor | None = None) -> torch.Tensor:
    T, I, ld = _matrix_args(X)
    if t.dtype != torch.float32 or c.dtype != torch.float32 or t.numel() != T or c.numel() != I:
        raise ValueError("t must be float32[T] and c float32[I]")
    ws = workspace if workspace is not None else _workspace(T, I, X.device)
    count = _counts(count, 1, X.device, "count")
    _check(lib().cq_kernel_count_x(_ptr(X), _DT[X.dtype], T, I, ld, float(alpha), int(bits), _ptr(t), _ptr(c),
                                   _ptr(count), _ptr(ws), ws.numel(), _stream()), "cq_kernel_count_x")
    return count


@dataclass
class WeightQuant:
    scale: torch.Tensor
    codes: torch.Tensor | None
    deq: torch.Tensor | None
    zero_count: torch.Tensor | None
    bits: int


def _check_weight_out(out: "WeightQuant", R: int, Cc: int, n_scales: int, dtype: torch.dtype, bits: int, where: str) -> None:
    def bad(what):
        raise ValueError(f"{where}: out.{what} does not match a {R} x {Cc} {dtype} matrix quantized to {bits} bits")
    if out.scale is not None and (out.scale.dtype != torch.float32 or out.scale.numel() != n_scales or not out.scale.is_contiguous()):
        bad("scale")
    if out.codes is not None:
        want = R * Cc if bits == 8 else R * (Cc // 2)
        if out.codes.element_size() != 1 or out.codes.numel() != want or not out.codes.is_contiguous():
            bad("codes")
    if out.deq is not None and (out.deq.dtype not in (dtype, torch.float32) or out.deq.numel() != R * Cc or not out.deq.is_contiguous()):
        bad("deq")
    if out.zero_count is not None and (out.zero_count.dtype != torch.int64 or out.zero_count.numel() != 1):
        bad("zero_count")


def quantize_weight_per_channel(W: torch.Tensor, bits: int = 8, *, codes: bool = True, deq: bool = True,
                                deq_dtype: torch.dtype | None = None, count: bool = True,
                                out: WeightQuant | None = None) -> WeightQuant:
    """Eq. 2: one scale per stored row of W (store weights as [out_channels, in_channels])."""
    R, Cc, ld = _matrix_args(W)
    if bits == 4 and Cc % 2:
        raise CQError(6, "cq_quantize_weight_per_channel")
    if out is None:
        dev = W.device
        codes_t = None
        if codes:
            codes_t = (torch.empty((R, Cc), dtype=torch.int8, device=dev) if bits == 8
                       else torch.empty((R, Cc // 2), dtype=torch.uint8, device=dev))
        out = WeightQuant(torch.empty(R, dtype=torch.float32, device=dev), codes_t,
                          torch.empty((R, Cc), dtype=deq_dtype or W.dtype, device=dev) if deq else None,
                          torch.zeros((), dtype=torch.int64, device=dev) if count else None, bits)
    _check_weight_out(out, R, Cc, R, W.dtype, bits, "quantize_weight_per_channel")
    deq_dt = _DT[out.deq.dtype] if out.deq is not None else _DT[W.dtype]
    st = lib().cq_quantize_weight_per_channel(_ptr(W), _DT[W.dtype], R, Cc, ld, int(bits), _ptr(out.codes),
                                              _ptr(out.scale), _ptr(out.deq), deq_dt, _ptr(out.zero_count),
                                              _stream())
    _check(st, "cq_quantize_weight_per_channel")
    return out


def quantize_weight_groupwise(W: torch.Tensor, group: int = 128, bits: int = 4, *, codes: bool = True, deq: bool = True,
                              deq_dtype: torch.dtype | None = None, count: bool = True,
                              out: WeightQuant | None = None) -> WeightQuant:
    """Group-wise weight quantization: every run of ``group`` consecutive elements of a stored row gets
    its own scale (``out.scale`` has R * C / group entries, row by row)."""
    R, Cc, ld = _matrix_args(W)
    if out is None:
        dev = W.device
        codes_t = None
        if codes:
            codes_t = (torch.empty((R, Cc), dtype=torch.int8, device=dev) if bits == 8
                       else torch.empty((R, Cc // 2), dtype=torch.uint8, device=dev))
        n_groups = R * (Cc // group) if group > 0 else 0
        out = WeightQuant(torch.empty(n_groups, dtype=torch.float32, device=dev), codes_t,
                          torch.empty((R, Cc), dtype=deq_dtype or W.dtype, device=dev) if deq else None,
                          torch.zeros((), dtype=torch.int64, device=dev) if count else None, bits)
    if group > 0 and Cc % group == 0:
        _check_weight_out(out, R, Cc, R * (Cc // group), W.dtype, bits, "quantize_weight_groupwise")
    deq_dt = _DT[out.deq.dtype] if out.deq is not None else _DT[W.dtype]
    st = lib().cq_quantize_weight_groupwise(_ptr(W), _DT[W.dtype], R, Cc, ld, int(group), int(bits), _ptr(out.codes),
                                            _ptr(out.scale), _ptr(out.deq), deq_dt, _ptr(out.zero_count), _stream())
    _check(st, "cq_quantize_weight_groupwise")
    return out


def case_indicators(r: ActQuant, *, counts: torch.Tensor | None = None) -> torch.Tensor:
    """Table 1 indicators of a quantize_act result: int64[2] on the device,
    (#pairs with c_j >= t_i, #pairs whose CrossQuant zero bound is below the per-token bound)."""
    counts = _counts(counts, 2, r.t.device, "counts")
    _check(lib().cq_case_indicators(_ptr(r.t), _ptr(r.c), _ptr(r.row_scale), _ptr(r.col_scale), r.t.numel(),
                                    r.c.numel(), int(r.bits), _ptr(counts), _stream()), "cq_case_indicators")
    return counts


def remove_kernel(X: torch.Tensor, alpha: float = 0.15, bits: int = 8, bound_scale: float = 1.0,
                  workspace: torch.Tensor | None = None, *, out: torch.Tensor | None = None,
                  counts: torch.Tensor | None = None):
    """Remove-Kernel operator: returns (X with the kernel elements set to +0 and the rest untouched,
    int64[3] device counts: removed, per-token kernel size, CrossQuant kernel size)."""
    T, I, ld = _matrix_args(X)
    ws = workspace if workspace is not None else _workspace(T, I, X.device)
    if out is None:
        out = torch.empty((T, I), dtype=X.dtype, device=X.device)
    elif out.dtype != X.dtype or tuple(out.shape) != (T, I) or not out.is_contiguous():
        raise ValueError("out must be a contiguous [T, I] tensor of X's dtype")
    counts = _counts(counts, 3, X.device, "counts")
    _check(lib().cq_remove_kernel(_ptr(X), _DT[X.dtype], T, I, ld, float(alpha), int(bits), float(bound_scale), _ptr(out),
                                  _ptr(counts), _ptr(ws), ws.numel(), _stream()), "cq_remove_kernel")
    return out, counts


def stage_fault() -> int:
    """1 if a bounded wait on a staged row copy ever gave up on the current device, else 0."""
    flag = C.c_uint(0)
    _check(lib().cq_stage_fault(C.byref(flag)), "cq_stage_fault")
    return int(flag.value)
