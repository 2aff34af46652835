"""Guard bands around every output buffer of the GPU tests.

The parity tests compare the inside of every output with the oracle; a kernel that stored one vector past the end
of a buffer (or before its start) would pass them all.  Here every output and workspace a test hands to the library is
carved out of one arena filled with a canary byte, with at least PAD canary bytes before and directly after it (the
canary starts at the first byte past the payload, so an overrun of a single byte shows).  After each call the canaries
are checked.  Everything is host-side bookkeeping plus a comparison on the device: nothing here can fault.

`Guarded(cq)` wraps the binding module: same function names, outputs allocated in guarded arenas, canaries checked
after the call.  Tests use it in place of the module (see the `cq` fixture in conftest.py).
"""
from __future__ import annotations

import torch

CANARY = 0xA5
PAD = 4096


def _round_up(v: int, m: int) -> int:
    return (v + m - 1) // m * m


class Arena:
    """A set of named device tensors separated by canary bytes."""

    def __init__(self, device="cuda"):
        self.device = torch.device(device)
        self._specs = []          # (name, shape, dtype, align, skew)
        self.views = {}
        self._spans = []          # (name, start, end) byte offsets of the payloads
        self.buf = None

    def add(self, name: str, shape, dtype: torch.dtype, *, align: int = 256, skew: int = 0) -> None:
        """Reserve a tensor; its first byte sits `skew` bytes past an `align`-byte boundary."""
        self._specs.append((name, tuple(shape) if not isinstance(shape, int) else (shape,), dtype, align, skew))

    def build(self) -> "Arena":
        off = PAD
        plan = []
        for name, shape, dtype, align, skew in self._specs:
            item = torch.empty((), dtype=dtype).element_size()
            n = 1
            for d in shape:
                n *= d
            start = _round_up(off, align) + skew
            plan.append((name, shape, dtype, start, n * item))
            off = start + n * item + PAD
        self.buf = torch.full((off,), CANARY, dtype=torch.uint8, device=self.device)
        assert self.device.type != "cuda" or self.buf.data_ptr() % 256 == 0
        for name, shape, dtype, start, nbytes in plan:
            self.views[name] = self.buf[start:start + nbytes].view(dtype).view(shape)
            self._spans.append((name, start, start + nbytes))
        return self

    def __getitem__(self, name: str) -> torch.Tensor:
        return self.views[name]

    def check(self, where: str = "") -> None:
        """Assert that every byte outside the payloads still holds the canary."""
        if self.device.type == "cuda":
            torch.cuda.synchronize(self.device)
        gaps, cur = [], 0
        for name, start, end in self._spans:
            gaps.append((cur, start, f"before {name}"))
            cur = end
        gaps.append((cur, self.buf.numel(), f"after {self._spans[-1][0]}" if self._spans else "arena"))
        joined = torch.cat([self.buf[s:e] for s, e, _ in gaps if e > s])
        if bool((joined != CANARY).any().item()):
            for s, e, label in gaps:
                bad = torch.nonzero(self.buf[s:e] != CANARY).flatten()
                if bad.numel():
                    first, last = int(bad[0].item()), int(bad[-1].item())
                    prev = [n for n, _, en in self._spans if en == s]
                    raise AssertionError(
                        f"{where}: {bad.numel()} guard byte(s) overwritten {label}"
                        f"{' / after ' + prev[0] if prev else ''}: gap bytes [{first}, {last}] of {e - s}")
            raise AssertionError(f"{where}: guard bytes overwritten")


def act_buffers(cq, T: int, I: int, dtype: torch.dtype, bits: int, *, codes=True, deq=True, deq_dtype=None, count=True,
                device="cuda", workspace=True):
    """cq.ActBuffers with every member (and the workspace) inside one guarded arena; `.arena` holds it."""
    ar = Arena(device)
    ar.add("t", T, torch.float32)
    ar.add("c", I, torch.float32)
    ar.add("row_scale", T, torch.float32)
    ar.add("col_scale", I, torch.float32)
    if codes:
        if bits == 8:
            ar.add("codes", (T, I), torch.int8)
        else:
            ar.add("codes", (T, I // 2), torch.uint8)
    if deq:
        ar.add("deq", (T, I), deq_dtype or dtype)
    if count:
        ar.add("zero_count", (), torch.int64)
    if workspace:
        ar.add("workspace", cq.workspace_bytes(T, I), torch.uint8)
    ar.build()
    b = object.__new__(cq.ActBuffers)
    b.T, b.I, b.bits = T, I, bits
    b.t, b.c, b.row_scale, b.col_scale = ar["t"], ar["c"], ar["row_scale"], ar["col_scale"]
    b.codes = ar["codes"] if codes else None
    b.deq = ar["deq"] if deq else None
    b.zero_count = ar["zero_count"] if count else None
    if count:
        b.zero_count.zero_()
    b.workspace = ar["workspace"] if workspace else None
    b.arena = ar
    return b


def weight_out(cq, R: int, Cc: int, n_scales: int, dtype: torch.dtype, bits: int, *, codes=True, deq=True, deq_dtype=None,
               count=True, device="cuda"):
    ar = Arena(device)
    ar.add("scale", n_scales, torch.float32)
    if codes:
        if bits == 8:
            ar.add("codes", (R, Cc), torch.int8)
        else:
            ar.add("codes", (R, Cc // 2), torch.uint8)
    if deq:
        ar.add("deq", (R, Cc), deq_dtype or dtype)
    if count:
        ar.add("zero_count", (), torch.int64)
    ar.build()
    out = cq.WeightQuant(ar["scale"], ar["codes"] if codes else None, ar["deq"] if deq else None,
                         ar["zero_count"] if count else None, bits)
    if count:
        out.zero_count.zero_()
    out.arena = ar
    return out


class Guarded:
    """The binding module with guarded outputs: same names and arguments as `paper_2410_07505_b200.cq`.

    Outputs the caller does not supply are allocated in a guarded arena; buffers made by `self.ActBuffers` are guarded
    too; after every call the canaries around what that call may have written are checked.  Anything not overridden
    here (errors, constants, tuning knobs) is the module's own.
    """

    def __init__(self, cq):
        self._cq = cq
        self.calls_checked = 0

    def __getattr__(self, name):
        return getattr(self._cq, name)

    # ---- helpers
    def _done(self, where: str, *arenas) -> None:
        if torch.cuda.is_current_stream_capturing():     # nothing has run yet; the test checks after the replay
            return
        for ar in arenas:
            if ar is not None:
                ar.check(where)
                self.calls_checked += 1

    def _vector(self, n: int, device, name: str = "out"):
        ar = Arena(device)
        ar.add(name, n, torch.float32)
        return ar.build()

    def _count(self, n: int, device):
        ar = Arena(device)
        ar.add("counts", () if n == 1 else (n,), torch.int64)
        ar.build()
        ar["counts"].zero_()
        return ar

    def _ws(self, T: int, I: int, device):
        ar = Arena(device)
        ar.add("workspace", self._cq.workspace_bytes(T, I), torch.uint8)
        return ar.build()

    def ActBuffers(self, T, I, dtype, bits, *, codes=True, deq=True, deq_dtype=None, count=True, device="cuda"):
        return act_buffers(self._cq, T, I, dtype, bits, codes=codes, deq=deq, deq_dtype=deq_dtype, count=count, device=device)

    # ---- absmax
    def absmax_rows(self, X):
        ar = self._vector(X.shape[0], X.device)
        t = self._cq.absmax_rows(X, out=ar["out"])
        self._done("absmax_rows", ar)
        return t

    def absmax_cols(self, X):
        ar = self._vector(X.shape[1], X.device)
        c = self._cq.absmax_cols(X, out=ar["out"])
        self._done("absmax_cols", ar)
        return c

    def absmax_rows_cols(self, X, *, workspace=None, out=None):
        ar = None
        if out is None:
            ar = Arena(X.device)
            ar.add("t", X.shape[0], torch.float32)
            ar.add("c", X.shape[1], torch.float32)
            ar.build()
            out = (ar["t"], ar["c"])
        r = self._cq.absmax_rows_cols(X, workspace=workspace, out=out)
        self._done("absmax_rows_cols", ar)
        return r

    # ---- activations
    def _act(self, fn, where, X, args, kw):
        buffers = kw.pop("buffers", None)
        if buffers is None:
            bits = args[1] if len(args) > 1 else kw.get("bits", 8)
            buffers = self.ActBuffers(X.shape[0], X.shape[1], X.dtype, bits, codes=kw.pop("codes", True),
                                      deq=kw.pop("deq", True), deq_dtype=kw.pop("deq_dtype", None),
                                      count=kw.pop("count", True), device=X.device)
        return buffers

    def quantize_act(self, X, alpha=0.15, bits=8, **kw):
        b = self._act(None, "quantize_act", X, (alpha, bits), kw)
        r = self._cq.quantize_act(X, alpha, bits, buffers=b)
        self._done("quantize_act", getattr(b, "arena", None))
        return r

    def quantize_act_given(self, X, t, c, alpha=0.15, bits=8, **kw):
        b = self._act(None, "quantize_act_given", X, (alpha, bits), kw)
        r = self._cq.quantize_act_given(X, t, c, alpha, bits, buffers=b)
        self._done("quantize_act_given", getattr(b, "arena", None))
        return r

    def quantize_act_noalloc(self, X, alpha=0.15, bits=8, *, buffers):
        r = self._cq.quantize_act_noalloc(X, alpha, bits, buffers=buffers)
        self._done("quantize_act_noalloc", getattr(buffers, "arena", None))
        return r

    # ---- stored codes
    def dequantize(self, codes, bits, T, I, row_scale, col_scale, out_dtype=torch.float32):
        ar = Arena(codes.device)
        ar.add("out", (T, I), out_dtype)
        ar.build()
        r = self._cq.dequantize(codes, bits, T, I, row_scale, col_scale, out_dtype, out=ar["out"])
        self._done("dequantize", ar)
        return r

    def kernel_count(self, codes, bits, T, I):
        ar = self._count(1, codes.device)
        r = self._cq.kernel_count(codes, bits, T, I, count=ar["counts"])
        self._done("kernel_count", ar)
        return r

    def kernel_count_x(self, X, alpha, bits, t, c, workspace=None):
        ar = self._count(1, X.device)
        ws = None
        if workspace is None:
            ws = self._ws(X.shape[0], X.shape[1], X.device)
            workspace = ws["workspace"]
        r = self._cq.kernel_count_x(X, alpha, bits, t, c, workspace, count=ar["counts"])
        self._done("kernel_count_x", ar, ws)
        return r

    def case_indicators(self, r):
        ar = self._count(2, r.t.device)
        out = self._cq.case_indicators(r, counts=ar["counts"])
        self._done("case_indicators", ar)
        return out

    def remove_kernel(self, X, alpha=0.15, bits=8, bound_scale=1.0, workspace=None):
        T, I = X.shape
        ar = Arena(X.device)
        ar.add("out", (T, I), X.dtype)
        ar.add("counts", (3,), torch.int64)
        if workspace is None:
            ar.add("workspace", self._cq.workspace_bytes(T, I), torch.uint8)
        ar.build()
        ar["counts"].zero_()
        r = self._cq.remove_kernel(X, alpha, bits, bound_scale, workspace if workspace is not None else ar["workspace"],
                                   out=ar["out"], counts=ar["counts"])
        self._done("remove_kernel", ar)
        return r

    # ---- weights
    def quantize_weight_per_channel(self, W, bits=8, *, codes=True, deq=True, deq_dtype=None, count=True, out=None):
        if out is None:
            out = weight_out(self._cq, W.shape[0], W.shape[1], W.shape[0], W.dtype, bits, codes=codes, deq=deq,
                             deq_dtype=deq_dtype, count=count, device=W.device)
        r = self._cq.quantize_weight_per_channel(W, bits, out=out)
        self._done("quantize_weight_per_channel", getattr(out, "arena", None))
        return r

    def quantize_weight_groupwise(self, W, group=128, bits=4, *, codes=True, deq=True, deq_dtype=None, count=True, out=None):
        R, Cc = W.shape
        if out is None and group > 0 and Cc % group == 0:
            out = weight_out(self._cq, R, Cc, R * (Cc // group), W.dtype, bits, codes=codes, deq=deq, deq_dtype=deq_dtype,
                             count=count, device=W.device)
        r = self._cq.quantize_weight_groupwise(W, group, bits, codes=codes, deq=deq, deq_dtype=deq_dtype, count=count, out=out)
        self._done("quantize_weight_groupwise", getattr(out, "arena", None))
        return r

    def vector_max_(self, acc, v):
        return self._cq.vector_max_(acc, v)
