"""Sharding the path over gradient coordinates (one process per GPU).

Every step of the path is independent per coordinate except the locator's
projection e = f R, a sum over coordinates.  So rank p keeps columns
[c0, c1) of all n rows, and the only exchange is one all-reduce of the projection
record (3 n doubles: the n complex projections and the n squared vector norms that
set the locator's rank cutoff; both add up over coordinates) between the projection
kernel and the small locator solve, which every rank then repeats identically.  The repetition code needs no
exchange for the sum; its per-node flags are OR-ed (a MAX all-reduce of n bytes).
"""
from __future__ import annotations


def shard_range(d_total: int, world: int, rank: int, align: int = 2048) -> tuple[int, int]:
    """Columns [c0, c1) owned by ``rank``: contiguous, starts aligned to ``align``
    coordinates (the projection tile, which also keeps every row slice 16-byte aligned)."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("bad world / rank")
    blocks = -(-d_total // align)
    per, extra = divmod(blocks, world)
    b0 = rank * per + min(rank, extra)
    b1 = b0 + per + (1 if rank < extra else 0)
    return min(b0 * align, d_total), min(b1 * align, d_total)


def locate_sharded(plan, R, f, flags, e_buf, group=None, stream=None):
    """Cyclic locator over a d-sharded R: local projection, all-reduce(sum) of e, local solve.

    ``plan`` is the rank's plan for its own slice; ``e_buf`` a float64 tensor of 3 n
    values on the same device as R.  Every rank ends with the same flags.

    ``stream`` (a ``torch.cuda.Stream``, or None for torch's current stream) carries all three
    steps: the collective is enqueued by torch on its *current* stream, so a given stream is
    made current for the duration of the call; the all-reduce then sees the projection's result
    and the solve sees the all-reduce's.
    """
    import contextlib

    import torch.distributed as dist
    if stream is None:
        ctx = contextlib.nullcontext()
    else:
        import torch
        ctx = torch.cuda.stream(stream)
    with ctx:
        plan.cyc_project(R, f, e_buf, stream=stream)
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(e_buf, op=dist.ReduceOp.SUM, group=group)
        plan.cyc_locate_from_projection(e_buf, flags, stream=stream)
    return flags


def merge_flags(flags, group=None, stream=None):
    """Repetition code: a node is flagged if any shard saw it disagree (element-wise MAX).
    ``stream``: as in ``locate_sharded`` (the stream the decode that wrote ``flags`` ran on)."""
    import contextlib

    import torch.distributed as dist
    if stream is None:
        ctx = contextlib.nullcontext()
    else:
        import torch
        ctx = torch.cuda.stream(stream)
    with ctx:
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(flags, op=dist.ReduceOp.MAX, group=group)
    return flags
