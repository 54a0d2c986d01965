"""Seeded random walks over the whole ABI against the oracle: dispatches, AdamW steps (fp32 and bf16
gradients), arrivals of random batches with random options, parameter overwrites and read-backs,
checkpoint round trips into a fresh context.  Every few operations the complete state is compared."""
import numpy as np
import pytest
import torch

from harness import Pair, assert_fp32
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed,pg_current,buffered,c,N", [(1, False, False, 0.0, 3), (2, True, False, 0.0, 4),
                                                          (3, False, True, 0.0, 2), (4, False, False, 0.125, 4),
                                                          (5, False, False, 0.0, 1), (6, True, True, 0.0, 5)])
def test_random_walk(seed, pg_current, buffered, c, N):
    walk(seed, pg_current, buffered, c, N)


@pytest.mark.parametrize("seed,pg_current,N,kw", [(7, False, 3, dict(sgdm=True)), (8, True, 1, dict(sgdm=True)),
                                                  (9, False, 4, dict(stable_ptrs=True)), (10, True, 2, dict(stable_ptrs=True, buffered=True)),
                                                  (11, False, 8, dict(W=11)), (12, True, 3, dict(W=9, stable_ptrs=True))])
def test_random_walk_outer_modes_stable_pointers_and_large_batches(seed, pg_current, N, kw):
    """The same walk with the SGD Momentum outer step, with permanent pointers, and with enough workers for
    batches of eight and batches split over launches."""
    walk(seed, pg_current, kw.pop("buffered", False), 0.0, N, **kw)


def walk(seed, pg_current, buffered, c, N, sgdm=False, stable_ptrs=False, W=6, steps=160):
    r = np.random.default_rng(seed)
    tensors = synth.ragged_tensors()
    align = int(r.choice([1, 4, 8]))
    pair = Pair(tensors, W, N, 0.9, 0.7, c=c, pg_current=pg_current, align=align, buffered=buffered, sgdm=sgdm,
                stable_ptrs=stable_ptrs)
    P = pair.P
    pair.set_global(synth.theta0(tensors, pair.offsets, P, synth.SEED + seed))
    dispatched = set()
    arrived = set()
    life = [0] * W
    scratch = torch.empty(P, dtype=torch.float32, device="cuda")

    def vec(std, stream):
        return synth.zero_padding(synth.normal_vec(P, std, synth.SEED + seed, stream, sub=int(r.integers(0, 1 << 30))),
                                  tensors, pair.offsets)

    for step in range(steps):
        op = r.choice(["pull", "adam", "adam16", "arrive", "arrive", "set", "get", "ckpt"],
                      p=[0.12, 0.25, 0.08, 0.15, 0.15, 0.08, 0.09, 0.08])
        if op == "pull" or not dispatched:
            w = int(r.integers(0, W))
            pair.pull(w)
            dispatched.add(w); arrived.discard(w)
        elif op in ("adam", "adam16"):
            w = int(r.choice(sorted(dispatched | arrived)))
            life[w] += 1
            g = vec(1e-2, synth.STREAM_GRAD)
            if op == "adam16":
                g16 = torch.from_numpy(g).to(torch.bfloat16)
                pair.ctx.alsgd_inner_adamw_bf16(w, g16.cuda(), life[w], 1e-3)
                pair.orc.inner_adamw(w, pair.take(g16.to(torch.float32).numpy()), life[w], 1e-3)
            else:
                pair.inner_adamw(w, torch.from_numpy(g).cuda(), g, life[w], 1e-3)
        elif op == "arrive":
            k = int(r.integers(1, len(dispatched) + 1))
            ids = [int(x) for x in r.permutation(sorted(dispatched))[:k]]
            reseed = bool(r.integers(0, 4))
            kind = r.choice(["plain", "weights", "poly", "thres", "dc"])
            kw = {}
            if kind == "weights":
                kw["weights"] = [float(x) for x in r.uniform(0.2, 1.2, k)]
            elif kind == "poly":
                kw["poly"] = True
            elif kind == "thres":
                kw.update(poly=True, stale_threshold=int(r.integers(0, 6)))
            elif kind == "dc" and not pg_current:
                kw["dc_lambda"] = 0.5
            pair.arrive(ids, reseed=reseed, norm=bool(r.integers(0, 2)), **kw)
            if not reseed:
                dispatched -= set(ids); arrived |= set(ids)
        elif op == "set":
            w = int(r.choice(sorted(dispatched | arrived)))
            z = vec(0.05, synth.STREAM_DELTA)
            pair.ctx.alsgd_set_worker_params(w, z)
            pair.orc.p[w][:] = pair.take(z)
        elif op == "get":
            w = int(r.integers(0, W))
            pair.ctx.alsgd_get_worker_params(w, scratch)
            pair.ctx.alsgd_sync()
            assert_fp32(f"get_worker_params[{w}] at step {step}", pair.fetch(scratch), pair.orc.p[w])
        elif op == "ckpt":
            image = pair.ctx.alsgd_export_state()
            fresh = B.Context(tensors, W, N, 0.9, 0.7, c=c, pg_base=B.PG_CURRENT if pg_current else B.PG_DISPATCH,
                              align_elems=align, buffered=buffered, sgdm=sgdm, stable_ptrs=stable_ptrs)
            fresh.alsgd_import_state(image)
            pair.ctx.close()
            pair.ctx = fresh
        if step % 7 == 0:
            pair.check_all(f"seed {seed} step {step} after {op}")
    pair.check_all(f"seed {seed} end")
    pair.close()
