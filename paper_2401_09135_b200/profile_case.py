"""A small fixed case for profiler captures: a few launches of each kernel on vectors larger than L2
but only ~2.4 GB on the device in total.

    python -m paper_2401_09135_b200.profile_case [--elems N]

Launch order: 2 pulls, 3 AdamW steps on worker 0, 3 on worker 1, then four times (one AdamW step,
one single arrival with fused re-seed) through one Delayed-Nesterov cycle of N = 4 (first / middle /
middle / boundary), then one AdamW step per worker and one batch of two: 19 launches.
"""
import argparse

import torch

from . import binding as B
from . import synth


def batches_case():
    n = 32 * 1024 * 1024
    tensors = synth.flat_tensors(n)
    W = 8
    ctx = B.Context(tensors, W, 8, 0.9, 0.7)
    ctx.alsgd_set_global(synth.theta0(tensors, ctx.offsets, ctx.P))
    g = torch.from_numpy(synth.normal_vec(ctx.P, 1e-2, synth.SEED, synth.STREAM_GRAD)).cuda()
    for w in range(W):
        ctx.alsgd_pull(w)
    for w in range(W):
        ctx.alsgd_inner_adamw(w, g, 1, 1e-3)
    ctx.alsgd_arrive([0, 1, 2, 3], B.ARRIVE_RESEED, want_info=False)     # first of the cycle, four distinct snapshots
    ctx.alsgd_arrive([4, 5, 6, 7], B.ARRIVE_RESEED, want_info=False)     # ends the cycle of N = 8 (boundary inside)
    for w in range(W):
        ctx.alsgd_inner_adamw(w, g, 2, 1e-3)
    ctx.alsgd_arrive(list(range(W)), B.ARRIVE_RESEED, want_info=False)   # whole cycle in one pass, two shared snapshots
    ctx.alsgd_sync()
    print(f"batches case done: P={ctx.P}, t={ctx.alsgd_counters()[0]}")
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--elems", type=int, default=48 * 1024 * 1024)
    ap.add_argument("--batches", action="store_true",
                    help="8 workers on 32Mi elements (4.3 GB): one AdamW step each, two batches of 4, one AdamW step each, one batch of 8")
    args = ap.parse_args()
    if args.batches:
        return batches_case()
    n = args.elems
    tensors = [synth.Tensor("w0", n // 2, True, "matrix"), synth.Tensor("g0", 4096, False, "gain"),
               synth.Tensor("w1", n - n // 2 - 4096, True, "matrix")]
    ctx = B.Context(tensors, 2, 4, 0.9, 0.7)
    theta0 = torch.from_numpy(synth.theta0(tensors, ctx.offsets, ctx.P))
    ctx.alsgd_set_global(theta0.numpy())
    g = torch.from_numpy(synth.normal_vec(ctx.P, 1e-2, synth.SEED, synth.STREAM_GRAD)).cuda()
    for w in range(2):
        ctx.alsgd_pull(w)
    for w in range(2):
        for s in range(1, 4):
            ctx.alsgd_inner_adamw(w, g, s, 1e-3)
    step = [3, 3]
    for w in (0, 1, 0, 1):
        step[w] += 1
        ctx.alsgd_inner_adamw(w, g, step[w], 1e-3)
        ctx.alsgd_arrive([w], B.ARRIVE_RESEED, want_info=False)
    for w in range(2):
        step[w] += 1
        ctx.alsgd_inner_adamw(w, g, step[w], 1e-3)
    ctx.alsgd_arrive([0, 1], B.ARRIVE_RESEED, want_info=False)
    ctx.alsgd_sync()
    print(f"profile case done: P={ctx.P}, t={ctx.alsgd_counters()[0]}")
    ctx.close()


if __name__ == "__main__":
    main()
