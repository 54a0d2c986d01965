"""The N > 1 path on CPU: two gloo ranks, each owning a contiguous range of the flat vector.

The path is elementwise, so a rank that runs the same arrival list on its own range must reproduce
the corresponding slice of the unsharded result bit for bit, with the weight-decay pattern of its
range (tensor pieces and padding) and with only host-side reductions crossing ranks.  The ranks run
the CPU oracle here (there is no GPU in this test); what is under test is the sharding logic and the
reductions that bench.py uses at N > 1.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import shard, synth


def test_shard_bounds_tile_the_vector():
    for P, world, align in [(12576, 2, 8), (109_549_056, 8, 128), (1000, 3, 128), (5, 4, 1), (4096, 1, 128)]:
        b = shard.shard_bounds(P, world, align)
        assert b[0][0] == 0 and b[-1][1] == P and len(b) == world
        for (lo, hi), (lo2, _) in zip(b, b[1:]):
            assert hi == lo2 and lo <= hi
        assert all(lo % align == 0 for lo, _ in b)


def test_shard_tensor_table_reproduces_the_decay_slice():
    tensors = synth.ragged_tensors()
    for align in (1, 8, 128):
        P, offs = B.alsgd_layout_size(tensors, align)
        full = oracle.decay_mask([t.numel for t in tensors], [t.decay for t in tensors], offs, P)
        for world in (1, 2, 3, 5):
            for lo, hi in shard.shard_bounds(P, world, align):
                if lo == hi:
                    continue
                tab = shard.shard_tensors(tensors, offs, lo, hi)
                assert sum(n for n, _ in tab) == hi - lo
                Ps, offs_s = B.alsgd_layout_size(tab, 1)          # the library accepts the shard's table
                assert Ps == hi - lo
                mask = oracle.decay_mask([n for n, _ in tab], [d for _, d in tab], offs_s, Ps)
                assert np.array_equal(mask, full[lo:hi])


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, result_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        tensors = synth.ragged_tensors()
        align, W, N = 8, 3, 2
        offs, P = oracle.layout_offsets([t.numel for t in tensors], align)
        lo, hi = shard.shard_bounds(P, world, align)[rank]
        tab = shard.shard_tensors(tensors, offs, lo, hi)
        offs_s, Ps = oracle.layout_offsets([n for n, _ in tab], 1)
        mask = oracle.decay_mask([n for n, _ in tab], [d for _, d in tab], offs_s, Ps)
        srv = oracle.OracleServer(hi - lo, W, N, 0.9, 0.7, decay=mask)
        theta0 = synth.theta0(tensors, offs, P)
        srv.set_global(theta0[lo:hi].copy())
        for w in range(W):
            srv.pull(w)
        norms, flags = [], []
        step = 0
        for batch in ([0, 2], [1], [2, 0, 1]):
            for w in batch:
                step += 1
                g = synth.zero_padding(synth.normal_vec(P, 1e-2, synth.SEED, synth.STREAM_GRAD, sub=step), tensors, offs)
                srv.inner_adamw(w, g[lo:hi].copy(), step, 1e-3)
            info = srv.arrive(batch, norm=True)
            s, f = shard.reduce_diagnostics([i["gnorm2"] for i in info], [i["nonfinite"] for i in info])
            norms += s
            flags += f
        times = shard.max_over_ranks([1.0 + rank, 5.0 - rank])
        np.savez(os.path.join(result_dir, f"rank{rank}.npz"), lo=lo, hi=hi, theta=srv.theta, m=srv.m, Delta=srv.Delta,
                 p0=srv.p[0], rep1=srv.replica[1], norms=np.array(norms), flags=np.array(flags), times=np.array(times))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_run(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    # the unsharded run
    tensors = synth.ragged_tensors()
    align, W, N = 8, 3, 2
    offs, P = oracle.layout_offsets([t.numel for t in tensors], align)
    mask = oracle.decay_mask([t.numel for t in tensors], [t.decay for t in tensors], offs, P)
    srv = oracle.OracleServer(P, W, N, 0.9, 0.7, decay=mask)
    srv.set_global(synth.theta0(tensors, offs, P))
    for w in range(W):
        srv.pull(w)
    norms = []
    step = 0
    for batch in ([0, 2], [1], [2, 0, 1]):
        for w in batch:
            step += 1
            g = synth.zero_padding(synth.normal_vec(P, 1e-2, synth.SEED, synth.STREAM_GRAD, sub=step), tensors, offs)
            srv.inner_adamw(w, g, step, 1e-3)
        norms += [i["gnorm2"] for i in srv.arrive(batch, norm=True)]
    parts = [np.load(os.path.join(str(tmp_path), f"rank{r}.npz")) for r in range(world)]
    assert int(parts[0]["lo"]) == 0 and int(parts[-1]["hi"]) == P
    for key, ref in (("theta", srv.theta), ("m", srv.m), ("Delta", srv.Delta), ("p0", srv.p[0]), ("rep1", srv.replica[1])):
        got = np.concatenate([p[key] for p in parts])
        assert got.dtype == ref.dtype and np.array_equal(got.view(np.uint8), ref.view(np.uint8)), key
    for p in parts:
        np.testing.assert_allclose(p["norms"], norms, rtol=1e-12)
        assert not p["flags"].any()
        assert list(p["times"]) == [2.0, 5.0]              # max over ranks of (1+r, 5-r)
