"""GPU parity for the Section 4 variants of the server step (alsgd_arrive_ex and the buffered outer
step): staleness weights, Poly / PolyThres, delay compensation, "Async. Buffer"."""
import ctypes as C

import numpy as np
import pytest
import torch

from harness import Pair
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu
SEED = synth.SEED + 40


def dev(x):
    return torch.from_numpy(x).cuda()


def start(pair):
    pair.set_global(synth.theta0(pair.tensors, pair.offsets, pair.P, SEED))
    for w in range(pair.W):
        pair.pull(w)


def perturb_all(pair, ids, rnd, std=1e-2):
    for w in ids:
        z = synth.normal_vec(pair.P, std, SEED, synth.STREAM_DELTA, sub=rnd * 64 + w)
        pair.perturb(w, dev(z), z)


BATCHES = [[0], [1, 2], [3, 4, 0], [2], [1, 3, 4, 0, 2], [4, 1], [0, 2, 3]]


@pytest.mark.parametrize("pg_current,N,c", [(False, 3, 0.0), (True, 2, 0.0), (False, 4, 0.25)])
def test_explicit_weights(pg_current, N, c):
    pair = Pair(synth.ragged_tensors(), 5, N, 0.9, 0.7, c=c, pg_current=pg_current, align=4)
    start(pair)
    r = np.random.default_rng(3)
    for b, ids in enumerate(BATCHES):
        perturb_all(pair, ids, b)
        weights = [1.0 if (b + j) % 3 == 0 else float(r.uniform(0.1, 1.5)) for j in range(len(ids))]
        pair.arrive(ids, reseed=True, norm=True, weights=weights)
        pair.check_all(f"batch {b}")
    pair.close()


@pytest.mark.parametrize("threshold", [None, 2])
def test_poly_and_poly_thres(threshold):
    pair = Pair(synth.ragged_tensors(), 6, 4, 0.9, 0.7, align=8)
    start(pair)
    dropped = 0
    seen_stale = set()
    order = [[0], [1], [2, 3], [0], [4], [1, 0], [5, 2], [3], [4, 5, 1], [0, 2]]
    for b, ids in enumerate(order):
        perturb_all(pair, ids, b)
        info = pair.arrive(ids, reseed=True, norm=True, poly=True, stale_threshold=threshold)
        dropped += sum(i["dropped"] for i in info)
        seen_stale |= {i["staleness"] for i in info}
        pair.check_all(f"batch {b}")
    assert max(seen_stale) >= 4
    assert (dropped > 0) == (threshold is not None)
    pair.close()


def test_all_updates_discarded_still_redispatches():
    pair = Pair(synth.flat_tensors(5000), 3, 4, 0.9, 0.7, align=1)
    start(pair)
    perturb_all(pair, [0, 1, 2], 0)
    pair.arrive([0], reseed=True)
    perturb_all(pair, [0], 1)
    pair.arrive([0], reseed=True)
    info = pair.arrive([1, 2], reseed=True, poly=True, stale_threshold=1)
    assert all(i["dropped"] for i in info) and pair.ctx.alsgd_counters()[0] == 2
    pair.check_all("after discarded batch")
    pair.close()


@pytest.mark.parametrize("pg_current", [False, True])
def test_delay_compensation(pg_current):
    pair = Pair(synth.ragged_tensors(), 4, 3, 0.9, 0.7, pg_current=pg_current, align=1)
    start(pair)
    for b, ids in enumerate([[0], [1], [2, 3], [0, 1], [3], [2, 0, 1]]):
        perturb_all(pair, ids, b, std=0.3)
        pair.arrive(ids, reseed=True, norm=True, dc_lambda=0.5)
        pair.check_all(f"batch {b}")
    pair.close()


@pytest.mark.parametrize("N", [1, 3, 4])
def test_buffered_outer_step(N):
    pair = Pair(synth.ragged_tensors(), 5, N, 0.9, 0.7, align=8, buffered=True)
    start(pair)
    for b, ids in enumerate(BATCHES):
        perturb_all(pair, ids, b)
        theta_before = pair.ctx.alsgd_state_ptrs()[0].clone()
        info = pair.arrive(ids, reseed=True, norm=True)
        pair.check_all(f"batch {b}")
        if not any(i["boundary"] for i in info):           # theta frozen between boundaries
            assert torch.equal(theta_before, pair.ctx.alsgd_state_ptrs()[0])
    pair.close()


def test_buffered_with_weights_and_poly_at_23m_sampled():
    tensors = synth.layout_23m()
    pair = Pair(tensors, 8, 4, 0.9, 0.7, n_sample=50_000, buffered=True)
    start(pair)
    zpool = [synth.normal_vec(pair.P, 1e-3, SEED, synth.STREAM_DELTA, sub=i) for i in range(2)]
    zdev = [dev(z) for z in zpool]
    for b, ids in enumerate([[0, 1, 2], [3], [4, 5, 6, 7, 0], [1, 2], [3, 4, 5, 6, 7, 0, 1, 2]]):
        for w in ids:
            pair.perturb(w, zdev[(w + b) % 2], zpool[(w + b) % 2])
        pair.arrive(ids, reseed=True, poly=True, dc_lambda=0.25)
        pair.check_server(f"batch {b}")
        for w in ids:
            pair.check_worker(w, f"batch {b}")
    pair.close()


def test_arrive_ex_argument_errors():
    ctx = B.Context(synth.flat_tensors(1024), 2, 2, 0.9, 0.7)
    ctx.alsgd_set_global(np.zeros(ctx.P, np.float32))
    ctx.alsgd_pull(0)
    ids = (C.c_uint32 * 1)(0)
    o = B.ArriveOpts()
    o.dc_lambda = -1.0
    assert ctx.raw("alsgd_arrive_ex", ids, 1, 0, C.byref(o), None) == B.E_ARG
    o.dc_lambda = 0.0
    o.staleness_rule = 9
    assert ctx.raw("alsgd_arrive_ex", ids, 1, 0, C.byref(o), None) == B.E_ARG
    o.staleness_rule = 0
    w = (C.c_float * 1)(float("nan"))
    o.weights = w
    assert ctx.raw("alsgd_arrive_ex", ids, 1, 0, C.byref(o), None) == B.E_ARG
    assert ctx.alsgd_counters()[0] == 0
    assert ctx.raw("alsgd_arrive_ex", ids, 1, 0, None, None) == B.OK       # NULL opts == alsgd_arrive
    assert ctx.alsgd_counters()[0] == 1
    ctx.close()


@pytest.mark.parametrize("N", [1, 3, 4])
def test_sgd_momentum_outer_step(N):
    """ALSGD_CFG_OUTER_SGDM: the heavy-ball step on the buffer mean at every N-th arrival (N = 1: at every arrival)."""
    pair = Pair(synth.ragged_tensors(), 5, N, 0.9, 0.7, align=8, sgdm=True)
    start(pair)
    for b, ids in enumerate(BATCHES):
        perturb_all(pair, ids, b)
        theta_before = pair.ctx.alsgd_state_ptrs()[0].clone()
        info = pair.arrive(ids, reseed=True, norm=True, weights=[0.5] * len(ids) if b == 3 else None)
        pair.check_all(f"batch {b}")
        if not any(i["boundary"] for i in info):
            assert torch.equal(theta_before, pair.ctx.alsgd_state_ptrs()[0])
    pair.close()


def test_outer_modes_exclude_each_other():
    cfg_flags = B.CFG_OUTER_BUFFERED | B.CFG_OUTER_SGDM
    tab = B.tensor_table(synth.flat_tensors(64))
    cfg = B.Config()
    cfg.n_workers, cfg.N, cfg.flags, cfg.beta, cfg.outer_lr = 1, 1, cfg_flags, 0.9, 0.7
    cfg.adam_b1, cfg.adam_b2, cfg.adam_eps, cfg.adam_wd = 0.9, 0.95, 1e-8, 0.1
    n = C.c_uint64()
    assert B.lib().alsgd_arena_bytes(tab, 1, 1, C.byref(cfg), C.byref(n)) == B.E_ARG
