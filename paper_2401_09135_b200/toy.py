"""A small end-to-end run of the method on self-made data (in the spirit of Section 6's toy example:
classification of a mixture of mixtures of Gaussians), with real gradients.

The model (a tiny MLP) and its forward/backward pass are plain PyTorch: they are the part of training
this library does not provide.  Everything the paper's server and workers do with the parameters goes
through the library: dispatch, inner AdamW steps, arrival with Delayed Nesterov (or plain Nesterov with
N = 1), DyLU step counts (Eq. 6), the learning-rate schedule (Eq. 3), shard sampling (Eq. 2) and the
grace-period scheduler (Algorithm 2).

    python -m paper_2401_09135_b200.toy            # prints a small comparison table
"""
from __future__ import annotations

import argparse
import math

import numpy as np
import torch

from . import binding as B
from . import synth

HIDDEN = 64
CLASSES = 4


def mlp_tensors():
    T = synth.Tensor
    return [T("w1", 2 * HIDDEN, True, "matrix"), T("b1", HIDDEN, False, "bias"),
            T("w2", HIDDEN * HIDDEN, True, "matrix"), T("b2", HIDDEN, False, "bias"),
            T("w3", HIDDEN * CLASSES, True, "matrix"), T("b3", CLASSES, False, "bias")]


def make_data(n_shards, points_per_shard, seed, device):
    """Every class is a mixture of three Gaussians in the plane; every shard sees all classes but in
    different proportions, so shards differ without being disjoint."""
    g = torch.Generator().manual_seed(seed)
    centers = 3.0 * torch.randn(CLASSES, 3, 2, generator=g)
    shards = []
    for s in range(n_shards):
        prop = torch.softmax(1.5 * torch.randn(CLASSES, generator=g), 0)
        y = torch.multinomial(prop, points_per_shard, replacement=True, generator=g)
        comp = torch.randint(0, 3, (points_per_shard,), generator=g)
        x = centers[y, comp] + 0.6 * torch.randn(points_per_shard, 2, generator=g)
        shards.append((x.to(device), y.to(device)))
    yv = torch.arange(CLASSES).repeat_interleave(500)
    xv = centers[yv, torch.randint(0, 3, (yv.numel(),), generator=g)] + 0.6 * torch.randn(yv.numel(), 2, generator=g)
    return shards, (xv.to(device), yv.to(device))


def unpack(flat, offsets):
    o = offsets
    w1 = flat[o[0]:o[0] + 2 * HIDDEN].view(2, HIDDEN)
    b1 = flat[o[1]:o[1] + HIDDEN]
    w2 = flat[o[2]:o[2] + HIDDEN * HIDDEN].view(HIDDEN, HIDDEN)
    b2 = flat[o[3]:o[3] + HIDDEN]
    w3 = flat[o[4]:o[4] + HIDDEN * CLASSES].view(HIDDEN, CLASSES)
    b3 = flat[o[5]:o[5] + CLASSES]
    return w1, b1, w2, b2, w3, b3


def loss_of(flat, offsets, x, y):
    w1, b1, w2, b2, w3, b3 = unpack(flat, offsets)
    h = torch.tanh(x @ w1 + b1)
    h = torch.tanh(h @ w2 + b2)
    return torch.nn.functional.cross_entropy(h @ w3 + b3, y)


def gradient(flat, offsets, x, y):
    p = flat.detach().clone().requires_grad_(True)
    loss_of(p, offsets, x, y).backward()
    return p.grad


def batch_of(shard, worker, step, batch, seed):
    x, y = shard
    g = torch.Generator().manual_seed(seed * 1_000_003 + worker * 10_007 + step)
    idx = torch.randint(0, x.shape[0], (batch,), generator=g).to(x.device)
    return x[idx], y[idx]


def init_theta(P, offsets, seed):
    g = torch.Generator().manual_seed(seed)
    th = torch.zeros(P)
    for t, off, fan_in in zip(mlp_tensors(), offsets, (2, 0, HIDDEN, 0, HIDDEN, 0)):
        if t.kind == "matrix":
            th[off:off + t.numel] = torch.randn(t.numel, generator=g) / math.sqrt(fan_in)
    return th


def run(speeds, N, outer_lr=0.7, beta=0.9, H=20, dylu=True, tau_grace=0.0, total_local_steps=4000, batch=64,
        lr_max=3e-3, lr_min=1e-5, warmup=50, seed=7, buffered=False, sgdm=False, device=0, log_every=0,
        sample_shards=True):
    """Asynchronous Local-SGD on the toy task through the library.  Returns (validation loss, accuracy,
    number of server updates, final theta as a CPU tensor)."""
    torch.cuda.set_device(device)
    dev = torch.device("cuda", device)
    W = len(speeds)
    tensors = mlp_tensors()
    ctx = B.Context(tensors, W, N, beta, outer_lr, adam=(0.9, 0.95, 1e-8, 0.1), align_elems=4, device=device, buffered=buffered,
                    sgdm=sgdm)
    P, offsets = ctx.P, ctx.offsets
    shards, val = make_data(W, 4000, seed, dev)
    ctx.alsgd_set_global(init_theta(P, offsets, seed).numpy())
    steps = B.alsgd_dylu_steps(speeds, H) if dylu else [H] * W
    sched = B.Scheduler(W, tau_grace, t_max=total_local_steps)
    T_shard = total_local_steps // W
    sizes = [float(s[0].shape[0]) for s in shards]
    learned = [0.0] * W
    shard_step = [0] * W                       # Eq. 3 runs per data shard
    life = [0] * W                             # AdamW step count per worker, never reset
    rng = np.random.default_rng(seed)

    def train(w):
        """train() of Algorithm 2 for one worker: pick a shard (Eq. 2), run its local steps, book its job."""
        if sample_shards:
            probs = B.alsgd_shard_probs(sizes, learned)
            s = int(rng.choice(W, p=np.asarray(probs) / sum(probs)))
        else:
            s = w                              # one fixed shard per worker (k workers, k shards)
        pw = ctx.alsgd_worker_state_ptrs(w)["p"]
        for _ in range(steps[w]):
            lr = B.alsgd_lr_at(lr_max, lr_min, warmup, T_shard, shard_step[s])
            x, y = batch_of(shards[s], w, life[w], batch, seed)
            g = gradient(pw, offsets, x, y)
            life[w] += 1
            shard_step[s] += 1
            ctx.alsgd_inner_adamw(w, g, life[w], lr)
        learned[s] += steps[w] * batch
        sched.dispatch(w, steps[w] / speeds[w], steps[w])

    for w in range(W):
        ctx.alsgd_pull(w)
    for w in range(W):
        train(w)
    updates = 0
    while True:
        ids, _, _ = sched.next_batch()
        if not ids:
            break
        ctx.alsgd_arrive(ids, B.ARRIVE_RESEED, want_info=False)
        updates += len(ids)
        if log_every and updates % log_every < len(ids):
            th = ctx.alsgd_state_ptrs()[0]
            print(f"  update {updates}: val loss {float(loss_of(th, offsets, *val)):.4f}")
        for w in ids:
            train(w)
    theta = ctx.alsgd_state_ptrs()[0].clone()
    ctx.alsgd_sync()
    with torch.no_grad():
        w1, b1, w2, b2, w3, b3 = unpack(theta, offsets)
        logits = torch.tanh(torch.tanh(val[0] @ w1 + b1) @ w2 + b2) @ w3 + b3
        vloss = float(torch.nn.functional.cross_entropy(logits, val[1]))
        acc = float((logits.argmax(1) == val[1]).float().mean())
    ctx.close()
    return vloss, acc, updates, theta.cpu()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=4000)
    args = ap.parse_args()
    hetero = [1.0, 1.5, 2.0, 3.0]
    rows = [
        ("synchronous (equal speeds, one window, N = 4)", dict(speeds=[1.0] * 4, N=4, dylu=False)),
        ("async Nesterov (N = 1), heterogeneous", dict(speeds=hetero, N=1, dylu=False)),
        ("async SGD Momentum at every arrival (N = 1), heterogeneous", dict(speeds=hetero, N=1, dylu=False, sgdm=True)),
        ("async plain outer SGD (SGD Momentum with beta = 0), heterogeneous", dict(speeds=hetero, N=1, dylu=False, sgdm=True, beta=0.0)),
        ("async buffered (N = 4), heterogeneous", dict(speeds=hetero, N=4, dylu=False, buffered=True)),
        ("async Delayed Nesterov (N = 4), heterogeneous", dict(speeds=hetero, N=4, dylu=False)),
        ("async Delayed Nesterov + DyLU, grace 0.5", dict(speeds=hetero, N=4, dylu=True, tau_grace=0.5)),
    ]
    print(f"{'setting':70s} {'val loss':>9s} {'accuracy':>9s} {'server updates':>15s}")
    for name, kw in rows:
        vloss, acc, updates, _ = run(total_local_steps=args.steps, **kw)
        print(f"{name:70s} {vloss:9.4f} {acc:9.4f} {updates:15d}")


if __name__ == "__main__":
    main()
