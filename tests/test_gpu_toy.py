"""End-to-end behaviour on the toy task (real gradients from a tiny MLP; see paper_2401_09135_b200/toy.py).

1. Pipeline validation, the way the paper validates its own: homogeneous workers driven through the
   asynchronous framework (grace window, Delayed Nesterov with N = k) must reproduce synchronous DiLoCo
   (Algorithm 1) with the Nesterov outer step of Eq. 4, written here in plain PyTorch.
2. The qualitative finding of Sections 4-5 on this task: applying Nesterov at every asynchronous arrival
   is much worse than Delayed Nesterov, and synchronous training is the reference to approach.
"""
import pytest
import torch

from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import toy

pytestmark = pytest.mark.gpu


def diloco_reference(W, H, rounds, outer_lr, beta, batch, lr_max, lr_min, warmup, T_shard, seed):
    dev = torch.device("cuda", 0)
    tensors = toy.mlp_tensors()
    P, offsets = B.alsgd_layout_size(tensors, 4)
    decay = torch.zeros(P, device=dev)
    for t, off in zip(tensors, offsets):
        if t.decay:
            decay[off:off + t.numel] = 1.0
    shards, val = toy.make_data(W, 4000, seed, dev)
    theta = toy.init_theta(P, offsets, seed).to(dev)
    m = torch.zeros_like(theta)
    am = [torch.zeros_like(theta) for _ in range(W)]
    av = [torch.zeros_like(theta) for _ in range(W)]
    life = [0] * W
    b1, b2, eps, wd = (torch.tensor(x, dtype=torch.float32).item() for x in (0.9, 0.95, 1e-8, 0.1))
    for _ in range(rounds):
        deltas = []
        for w in range(W):                                         # worker w on its shard w
            p = theta.clone()
            for _ in range(H):
                lr = B.alsgd_lr_at(lr_max, lr_min, warmup, T_shard, life[w])
                g = toy.gradient(p, offsets, *toy.batch_of(shards[w], w, life[w], batch, seed))
                life[w] += 1
                am[w] = b1 * am[w] + (1 - b1) * g
                av[w] = b2 * av[w] + (1 - b2) * g * g
                r = (am[w] / (1 - b1 ** life[w])) / ((av[w] / (1 - b2 ** life[w])).sqrt() + eps)
                p = p - lr * (r + wd * decay * p)
            deltas.append(theta - p)
        D = sum(deltas) / W                                        # outer gradient of Algorithm 1
        theta = theta - outer_lr * (beta * beta * m + (1 + beta) * D)   # Eq. 4
        m = beta * m + D
    return theta.cpu(), float(toy.loss_of(theta, offsets, *val))


def test_homogeneous_async_pipeline_equals_synchronous_diloco():
    W, H, rounds = 4, 20, 10
    kw = dict(outer_lr=0.7, beta=0.9, batch=64, lr_max=3e-3, lr_min=1e-5, warmup=50, seed=11)
    vloss, acc, updates, theta = toy.run(speeds=[1.0] * W, N=W, H=H, dylu=False, tau_grace=0.0,
                                         total_local_steps=W * H * rounds, sample_shards=False, **kw)
    ref_theta, ref_loss = diloco_reference(W, H, rounds, T_shard=H * rounds, **kw)
    assert updates == W * rounds
    scale = float(ref_theta.abs().max())
    assert float((theta - ref_theta).abs().max()) <= 2e-3 * scale
    assert abs(vloss - ref_loss) <= 2e-3 * max(1.0, ref_loss)


def test_delayed_nesterov_beats_per_arrival_nesterov_on_heterogeneous_workers():
    hetero = [1.0, 1.5, 2.0, 3.0]
    sync = toy.run(speeds=[1.0] * 4, N=4, dylu=False, total_local_steps=4000)[0]
    nesterov = toy.run(speeds=hetero, N=1, dylu=False, total_local_steps=4000)[0]
    dn = toy.run(speeds=hetero, N=4, dylu=False, total_local_steps=4000)[0]
    dn_dylu = toy.run(speeds=hetero, N=4, dylu=True, tau_grace=0.5, total_local_steps=4000)[0]
    assert dn < 0.5 * nesterov and dn_dylu < 0.5 * nesterov
    assert sync < dn
