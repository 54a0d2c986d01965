"""Range sharding with the real kernels: three contexts, each owning one contiguous range of the flat
vector (as three ranks would, here side by side on one GPU; nothing in this path waits on another
context), driven by the same arrival list, must reproduce the unsharded context bit for bit."""
import numpy as np
import pytest
import torch

from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import shard, synth

pytestmark = pytest.mark.gpu


def test_three_range_shards_equal_the_unsharded_run():
    tensors = synth.ragged_tensors()
    align, W, N, G = 8, 4, 3, 3
    full = B.Context(tensors, W, N, 0.9, 0.7, align_elems=align)
    P, offs = full.P, full.offsets
    bounds = shard.shard_bounds(P, G, align)
    parts = [B.Context(shard.shard_tensors(tensors, offs, lo, hi), W, N, 0.9, 0.7, align_elems=1) for lo, hi in bounds]
    assert [c.P for c in parts] == [hi - lo for lo, hi in bounds]
    theta0 = synth.theta0(tensors, offs, P)
    full.alsgd_set_global(theta0)
    for c, (lo, hi) in zip(parts, bounds):
        c.alsgd_set_global(np.ascontiguousarray(theta0[lo:hi]))
    for ctx in [full] + parts:
        for w in range(W):
            ctx.alsgd_pull(w)
    life = [0] * W
    norms_full, norms_parts = [], []
    for b, ids in enumerate([[0, 1], [2], [3, 0, 1], [2, 3, 0, 1], [1]]):
        for w in ids:
            life[w] += 1
            g = synth.zero_padding(synth.normal_vec(P, 1e-2, synth.SEED, synth.STREAM_GRAD, sub=w * 16 + life[w]), tensors, offs)
            gd = torch.from_numpy(g).cuda()
            full.alsgd_inner_adamw(w, gd, life[w], 1e-3)
            for c, (lo, hi) in zip(parts, bounds):
                c.alsgd_inner_adamw(w, gd[lo:hi].clone(), life[w], 1e-3)
        flags = B.ARRIVE_RESEED | B.ARRIVE_NORM | B.ARRIVE_NANCHECK
        norms_full += [i["gnorm2"] for i in full.alsgd_arrive(ids, flags)]
        per = [[i["gnorm2"] for i in c.alsgd_arrive(ids, flags)] for c in parts]
        norms_parts += [sum(x) for x in zip(*per)]               # what the all-reduce of the diagnostics would give
    fs = full.alsgd_state_ptrs()
    for k, name in enumerate(("theta", "m", "Delta")):
        got = torch.cat([c.alsgd_state_ptrs()[k] for c in parts])
        assert torch.equal(got.view(torch.int32), fs[k].view(torch.int32)), name
    for w in range(W):
        fw = full.alsgd_worker_state_ptrs(w)
        pw = [c.alsgd_worker_state_ptrs(w) for c in parts]
        for key in ("p", "base", "adam_m", "adam_v", "replica"):
            got = torch.cat([x[key] for x in pw])
            assert torch.equal(got.view(torch.int16), fw[key].view(torch.int16)), (w, key)
    np.testing.assert_allclose(norms_parts, norms_full, rtol=1e-6)
    assert full.alsgd_counters() == parts[0].alsgd_counters()
    for c in [full] + parts:
        c.close()
