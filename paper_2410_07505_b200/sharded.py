"""One activation matrix held in several row blocks: tokens split over ranks, or X streamed in chunks.

The CrossQuant scale needs c_j, the column absmax over ALL tokens (Section 4.2), so between the absmax
pass and the quantize pass the blocks' column maxima are combined: by one all-reduce (MAX) of I floats
when the blocks live on different ranks, by a running maximum when they pass through one device.  The
row maxima t_i stay with the block that holds row i, and the sizes of the quantization kernel
(Definition 1) add up.  Every step on the data runs in the library's kernels; ``torch.distributed``
only moves the I-float vector and the one count.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist

from . import cq


def shard_rows(T: int, world: int, rank: int) -> tuple[int, int]:
    """Rows [r0, r1) of a T-row matrix that rank `rank` of `world` holds: contiguous, sizes differ by <= 1."""
    if world < 1 or not 0 <= rank < world or T < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(T, world)
    r0 = rank * base + min(rank, extra)
    return r0, r0 + base + (1 if rank < extra else 0)


def _world(group) -> int:
    return dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1


def combine_column_maxima(c_local: torch.Tensor, group=None) -> torch.Tensor:
    """In place: c_local becomes the elementwise maximum over all ranks of `group` (no-op without a group)."""
    if _world(group) > 1:
        dist.all_reduce(c_local, op=dist.ReduceOp.MAX, group=group)
    return c_local


def combine_counts(count_local: torch.Tensor, group=None) -> torch.Tensor:
    """Sum of the ranks' kernel sizes (a new int64 tensor; the local count is left as it is)."""
    total = count_local.clone()
    if _world(group) > 1:
        dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    return total


def quantize_act_row_sharded(X_local: torch.Tensor, alpha: float = 0.15, bits: int = 8, *, group=None,
                             buffers: "cq.ActBuffers | None" = None):
    """CrossQuant of this rank's row block of a matrix whose tokens are split over the ranks of `group`.

    Returns (ActQuant of the block, with t local and c global; int64 tensor: |K(CQ)| of the whole matrix).
    Identical, block by block, to quantizing the whole matrix on one device.
    """
    T, I = X_local.shape
    b = buffers or cq.ActBuffers(T, I, X_local.dtype, bits, device=X_local.device)
    t, c = cq.absmax_rows_cols(X_local, workspace=b.workspace, out=(b.t, b.c))
    combine_column_maxima(c, group)
    out = cq.quantize_act_given(X_local, t, c, alpha, bits, buffers=b)
    return out, combine_counts(out.zero_count, group)


def quantize_act_col_sharded(X_local: torch.Tensor, alpha: float = 0.15, bits: int = 8, *, group=None,
                             buffers: "cq.ActBuffers | None" = None):
    """The same for channels split over the ranks (how tensor-parallel FC2 inputs arrive): the column maxima
    are local, the row maxima t_i are combined (all-reduce MAX of T floats).  X_local may be a column slice
    of a wider matrix (rows `stride(0)` apart).  Returns (ActQuant with t global and c local, total count)."""
    T, I = X_local.shape
    b = buffers or cq.ActBuffers(T, I, X_local.dtype, bits, device=X_local.device)
    t, c = cq.absmax_rows_cols(X_local, workspace=b.workspace, out=(b.t, b.c))
    combine_column_maxima(t, group)            # the same exchange, on the other vector
    out = cq.quantize_act_given(X_local, t, c, alpha, bits, buffers=b)
    return out, combine_counts(out.zero_count, group)


def quantize_act_column_blocks(blocks: Sequence[torch.Tensor], alpha: float = 0.15, bits: int = 8):
    """One device, the matrix given as column blocks (each [T, I_k], same T): running maximum of t over the
    blocks, then each block quantized with the final t and its own c.  Returns (list of ActQuant, total)."""
    if not blocks:
        return [], 0
    bufs = [cq.ActBuffers(X.shape[0], X.shape[1], X.dtype, bits, device=X.device) for X in blocks]
    t = None
    for X, b in zip(blocks, bufs):
        t_k, _ = cq.absmax_rows_cols(X, workspace=b.workspace, out=(b.t, b.c))
        t = t_k if t is None else cq.vector_max_(t, t_k)
    outs = [cq.quantize_act_given(X, t, b.c, alpha, bits, buffers=b) for X, b in zip(blocks, bufs)]
    return outs, sum(int(o.zero_count.item()) for o in outs)


def quantize_act_chunked(chunks: Sequence[torch.Tensor], alpha: float = 0.15, bits: int = 8):
    """CrossQuant of a matrix that passes through the device as row chunks (each [T_k, I], same I).

    First sweep: each chunk's absmax vectors, c kept as a running maximum.  Second sweep: each chunk is
    quantized with its own t and the final c.  Returns (list of ActQuant, total kernel size as int).
    """
    if not chunks:
        return [], 0
    bufs = [cq.ActBuffers(X.shape[0], X.shape[1], X.dtype, bits, device=X.device) for X in chunks]
    c = None
    for X, b in zip(chunks, bufs):
        _, c_k = cq.absmax_rows_cols(X, workspace=b.workspace, out=(b.t, b.c))
        c = c_k if c is None else cq.vector_max_(c, c_k)
    outs = [cq.quantize_act_given(X, b.t, c, alpha, bits, buffers=b) for X, b in zip(chunks, bufs)]
    total = sum(int(o.zero_count.item()) for o in outs)
    return outs, total
