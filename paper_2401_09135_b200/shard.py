"""Range sharding of the flat vector over ranks, and the only cross-rank reductions the path needs.

Every step of the server path is elementwise over the flat index, so rank r of G owns one contiguous
range of theta, m, Delta and of every worker's buffers and runs the same host-issued arrival list on
it.  No data-path exchange exists.  What crosses ranks is host-side only: the maximum of device
times (benchmark), and the sum / OR of the optional pseudo-gradient diagnostics.
"""
from __future__ import annotations


def shard_bounds(P: int, world: int, align: int = 128):
    """[lo, hi) of every rank: contiguous, covering [0, P), split points rounded to `align`."""
    assert world >= 1 and align >= 1
    units = (P + align - 1) // align
    cuts = [min(P, ((units * r) // world) * align) for r in range(world)] + [P]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def shard_tensors(tensors, offsets, lo: int, hi: int):
    """The (numel, decay) table of the sub-vector [lo, hi) of a laid-out tensor list, for a context
    created with align_elems = 1: tensor pieces keep their decay flag, padding becomes undecayed
    pieces, so the shard's weight-decay pattern is exactly the slice of the full one."""
    out = []
    cur = lo

    def push(n, decay):
        if n <= 0:
            return
        if out and out[-1][1] == decay:
            out[-1] = (out[-1][0] + n, decay)
        else:
            out.append((n, decay))

    for t, off in zip(tensors, offsets):
        a, b = max(int(off), lo), min(int(off) + t.numel, hi)
        if a >= b:
            continue
        push(a - cur, False)          # padding (or nothing) before this piece
        push(b - a, bool(t.decay))
        cur = b
    push(hi - cur, False)
    return out


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def reduce_diagnostics(gnorm2, nonfinite, device=None):
    """Sum of per-shard squared norms and OR of per-shard non-finite flags, one entry per arrival."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(x) for x in gnorm2], [int(bool(x)) for x in nonfinite]
    dev = device if device is not None else "cpu"
    s = torch.tensor(gnorm2, dtype=torch.float64, device=dev)
    f = torch.tensor([int(bool(x)) for x in nonfinite], dtype=torch.int64, device=dev)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    dist.all_reduce(f, op=dist.ReduceOp.MAX)
    return [float(x) for x in s.cpu()], [int(x) for x in f.cpu()]
