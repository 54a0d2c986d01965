"""What the borrowed pointers of alsgd_state_ptrs / alsgd_worker_state_ptrs show over time: in the default mode
(deferred stores, shared snapshots) exactly what the header documents, and with ALSGD_CFG_STABLE_PTRS the current
state at all times without asking again."""
import numpy as np
import pytest
import torch

from harness import Pair, assert_fp32
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu
SEED = synth.SEED + 70


def dev(x):
    return torch.from_numpy(x).cuda()


def test_default_mode_kept_pointer_shows_the_previous_round_until_asked_again():
    pair = Pair(synth.ragged_tensors(), 2, 2, 0.9, 0.7, align=4)
    pair.set_global(synth.theta0(pair.tensors, pair.offsets, pair.P, SEED))
    for w in range(2):
        pair.pull(w)
    z = synth.normal_vec(pair.P, 1e-2, SEED, synth.STREAM_DELTA)
    pair.perturb(0, dev(z), z)
    kept = pair.ctx.alsgd_worker_state_ptrs(0)["p"]            # kept across the dispatch below
    trained = pair.orc.p[0].copy()
    pair.arrive([0], reseed=True)
    pair.ctx.alsgd_sync()
    # documented: the re-seeded parameters are not copied into p; the kept view still shows the round that arrived
    assert_fp32("kept p", kept.cpu().numpy(), trained)
    again = pair.ctx.alsgd_worker_state_ptrs(0)["p"]            # asking again makes the copy
    pair.ctx.alsgd_sync()
    assert again.data_ptr() == kept.data_ptr()
    assert_fp32("p after asking again", again.cpu().numpy(), pair.orc.theta)
    pair.check_all("after")
    pair.close()


@pytest.mark.parametrize("pg_current,N", [(False, 2), (True, 3), (False, 1)])
def test_stable_pointers_stay_current_without_asking_again(pg_current, N):
    tensors = synth.ragged_tensors()
    W = 4
    pair = Pair(tensors, W, N, 0.9, 0.7, align=8, pg_current=pg_current, stable_ptrs=True)
    pair.set_global(synth.theta0(tensors, pair.offsets, pair.P, SEED + 1))
    for w in range(W):
        pair.pull(w)
    theta, m, delta = pair.ctx.alsgd_state_ptrs()               # asked once, held for the whole test
    views = [pair.ctx.alsgd_worker_state_ptrs(w) for w in range(W)]
    ptrs = [(v["p"].data_ptr(), None if v["base"] is None else v["base"].data_ptr()) for v in views]
    if not pg_current:
        assert len({b for _, b in ptrs}) == W                   # every worker keeps a snapshot of its own
    step = [0] * W
    for b, ids in enumerate([[0], [1, 2], [3, 0, 1], [2], [0, 1, 2, 3], [3]]):
        for w in ids:
            step[w] += 1
            g = synth.zero_padding(synth.normal_vec(pair.P, 1e-2, SEED + 1, synth.STREAM_GRAD, sub=w * 16 + step[w]),
                                   tensors, pair.offsets)
            pair.inner_adamw(w, dev(g), g, step[w], 1e-3)
        pair.arrive(ids, reseed=True, norm=True)
        pair.ctx.alsgd_sync()
        where = f"batch {b}"
        assert_fp32(f"theta {where}", theta.cpu().numpy(), pair.orc.theta)
        assert_fp32(f"m {where}", m.cpu().numpy(), pair.orc.m)
        assert_fp32(f"Delta {where}", delta.cpu().numpy(), pair.orc.Delta)
        for w in range(W):
            assert_fp32(f"p[{w}] {where}", views[w]["p"].cpu().numpy(), pair.orc.p[w])
            if views[w]["base"] is not None:
                assert_fp32(f"base[{w}] {where}", views[w]["base"].cpu().numpy(), pair.orc.base[w])
            assert np.array_equal(views[w]["replica"].cpu().numpy().view(np.uint16), pair.orc.replica[w])
        now = [pair.ctx.alsgd_worker_state_ptrs(w) for w in range(W)]
        assert ptrs == [(v["p"].data_ptr(), None if v["base"] is None else v["base"].data_ptr()) for v in now]
    pair.close()
