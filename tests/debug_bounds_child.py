"""Child process of test_gpu_debug_bounds.py: everything here runs against libalsgd_dbg.so, the build whose
kernels range-check every access to an arena-owned vector (a process loads one build of the library only).
No access ever leaves the arena: the refusals are provoked by narrowing the range the checks accept."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2401_09135_b200 import binding as B  # noqa: E402

B.use_debug_library()

from harness import Pair  # noqa: E402
from paper_2401_09135_b200 import synth  # noqa: E402

SEED = synth.SEED + 90


def dev(x):
    return torch.from_numpy(x).cuda()


def word_view(ctx):
    off = ctx.alsgd_debug_word_ptr() - ctx.arena.data_ptr()
    return ctx.arena[off:off + 4].view(torch.int32)


def clean_runs_record_nothing():
    # ragged layout, batches with boundaries anywhere, k = 11 split over launches, odd sizes with scalar tails
    for tensors, W, batches, align in (
            (synth.ragged_tensors(), 5, [[0], [1, 2], [3, 4, 0], [1, 2, 3, 4], [0, 1, 2, 3, 4]], 8),
            (synth.ragged_tensors(), 12, [[5, 0, 11, 3, 7, 1, 9, 2, 10, 4, 8], [6]], 1),
            (synth.flat_tensors(1023), 2, [[0, 1], [1], [0]], 1),
            (synth.flat_tensors(7), 2, [[1, 0]], 1)):
        for pg_current in (False, True):
            pair = Pair(tensors, W, 3, 0.9, 0.7, c=0.2, pg_current=pg_current, align=align)
            pair.set_global(synth.theta0(tensors, pair.offsets, pair.P, SEED))
            for w in range(W):
                pair.pull(w)
            step = [0] * W
            for ids in batches:
                for w in ids:
                    step[w] += 1
                    g = synth.zero_padding(synth.normal_vec(pair.P, 1e-2, SEED, synth.STREAM_GRAD, sub=w * 8 + step[w]),
                                           tensors, pair.offsets)
                    pair.inner_adamw(w, dev(g), g, step[w], 1e-3)
                pair.arrive(ids, reseed=True, norm=True)
                pair.check_all("debug build")
            pair.ctx.alsgd_sync()                                  # raises on ALSGD_E_BOUNDS
            assert int(word_view(pair.ctx).item()) == 0
            pair.close()


def status_follows_the_word():
    ctx = B.Context(synth.flat_tensors(4096), 1, 2, 0.9, 0.7)
    assert ctx.raw("alsgd_sync") == B.OK
    word_view(ctx).fill_(4)                                        # as if a momentum access had been refused
    torch.cuda.synchronize()
    assert ctx.raw("alsgd_sync") == B.E_BOUNDS
    assert ctx.raw("alsgd_sync") == B.E_BOUNDS                     # sticky until the caller clears it
    word_view(ctx).zero_()
    torch.cuda.synchronize()
    assert ctx.raw("alsgd_sync") == B.OK
    assert B.lib().alsgd_strerror(B.E_BOUNDS) not in (b"ok", b"unknown status")
    ctx.close()


def narrowed_range_refuses_and_records():
    P = 8192 + 3
    ctx = B.Context(synth.flat_tensors(P), 2, 2, 0.9, 0.7, align_elems=1)
    theta0 = synth.theta0(synth.flat_tensors(P), ctx.offsets, ctx.P, SEED)
    ctx.alsgd_set_global(theta0)
    for w in range(2):
        ctx.alsgd_pull(w)
    ctx.alsgd_sync()
    # The last slice of the arena is worker 1's bf16 replica: exclude it from the accepted range.
    rep = ctx.alsgd_worker_state_ptrs(1)["replica"]
    before = rep.clone()
    limit = rep.data_ptr() - (ctx.arena.data_ptr() + (-ctx.arena.data_ptr()) % 256)
    assert ctx.raw("alsgd_debug_guard_limit", limit) == B.OK
    g = dev(synth.normal_vec(P, 1e-2, SEED, synth.STREAM_GRAD))
    ctx.alsgd_inner_adamw(1, g, 1, 1e-3)
    assert ctx.raw("alsgd_sync") == B.E_BOUNDS
    assert int(word_view(ctx).item()) == 512                       # replica stores, nothing else
    assert torch.equal(rep, before)                                # refused, not performed
    p = ctx.alsgd_worker_state_ptrs(1)["p"]
    assert not torch.equal(p.cpu(), torch.from_numpy(theta0))      # the in-range part of the step was done
    # an arrival that re-seeds worker 1 would write that replica too
    word_view(ctx).zero_()
    ctx.alsgd_arrive([1], B.ARRIVE_RESEED, want_info=False)
    assert ctx.raw("alsgd_sync") == B.E_BOUNDS
    assert int(word_view(ctx).item()) == 512
    assert torch.equal(rep, before)
    # whole arena again: nothing is refused any more
    assert ctx.raw("alsgd_debug_guard_limit", 0) == B.OK
    word_view(ctx).zero_()
    ctx.alsgd_inner_adamw(1, g, 2, 1e-3)
    ctx.alsgd_arrive([0], B.ARRIVE_RESEED, want_info=False)
    assert ctx.raw("alsgd_sync") == B.OK
    assert ctx.raw("alsgd_debug_guard_limit", ctx.arena_bytes + 1) == B.E_ARG
    ctx.close()


if __name__ == "__main__":
    clean_runs_record_nothing()
    status_follows_the_word()
    narrowed_range_refuses_and_records()
    print("DEBUG-BOUNDS-OK")
