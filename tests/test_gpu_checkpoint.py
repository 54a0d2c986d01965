"""Checkpoint / resume: exporting the state after part of a run and importing it into a fresh context
must continue bit for bit like the uninterrupted run (server state, worker state, bookkeeping)."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu
SEED = synth.SEED + 60
BATCHES = [[0], [1, 2], [3, 0], [2], [1, 3, 0, 2], [1], [0, 3], [2, 1], [3], [0, 1, 2, 3]]


def run(ctx, batches, life, first_batch):
    infos = []
    for b, ids in enumerate(batches, start=first_batch):
        for w in ids:
            for _ in range(1 + (w + b) % 2):
                life[w] += 1
                g = synth.normal_vec(ctx.P, 1e-2, SEED, synth.STREAM_GRAD, sub=w * 100 + life[w])
                ctx.alsgd_inner_adamw(w, torch.from_numpy(g).cuda(), life[w], 1e-3)
        infos += ctx.alsgd_arrive(ids, B.ARRIVE_RESEED)
    return infos


def fresh(pg=B.PG_DISPATCH, replica=True):
    tensors = synth.ragged_tensors()
    ctx = B.Context(tensors, 4, 3, 0.9, 0.7, pg_base=pg, replica=replica, align_elems=8)
    return tensors, ctx


def same(a, b):
    for x, y in zip(a.alsgd_state_ptrs(), b.alsgd_state_ptrs()):
        assert torch.equal(x.view(torch.int32), y.view(torch.int32))
    for w in range(4):
        va, vb = a.alsgd_worker_state_ptrs(w), b.alsgd_worker_state_ptrs(w)
        for k in va:
            if va[k] is None:
                assert vb[k] is None
            else:
                assert torch.equal(va[k].view(torch.int16), vb[k].view(torch.int16)), (w, k)
    assert a.alsgd_counters() == b.alsgd_counters()


@pytest.mark.parametrize("pg,replica,cut", [(B.PG_DISPATCH, True, 5), (B.PG_DISPATCH, True, 3), (B.PG_CURRENT, False, 4)])
def test_export_import_continues_bit_for_bit(pg, replica, cut):
    tensors, straight = fresh(pg, replica)
    _, first = fresh(pg, replica)
    theta0 = synth.theta0(tensors, straight.offsets, straight.P, SEED)
    for c in (straight, first):
        c.alsgd_set_global(theta0)
        for w in range(4):
            c.alsgd_pull(w)
    life_a, life_b = [0] * 4, [0] * 4
    info_a = run(straight, BATCHES, life_a, 0)
    info_b = run(first, BATCHES[:cut], life_b, 0)
    image = first.alsgd_export_state()
    assert image.size == first.alsgd_state_bytes()
    first.close()
    _, resumed = fresh(pg, replica)
    resumed.alsgd_import_state(image)
    info_b += run(resumed, BATCHES[cut:], life_b, cut)
    straight.alsgd_sync(); resumed.alsgd_sync()
    same(straight, resumed)
    assert info_a == info_b                                  # ticks, boundaries, staleness after the resume too
    straight.close(); resumed.close()


def test_import_rejects_foreign_images():
    tensors, ctx = fresh()
    image = ctx.alsgd_export_state()
    bad = image.copy(); bad[0] ^= 0xFF
    assert ctx.raw("alsgd_import_state", bad.ctypes.data, bad.size) == B.E_ARG            # not an image
    assert ctx.raw("alsgd_import_state", image.ctypes.data, image.size - 1) == B.E_ARG     # truncated
    small = np.zeros(16, np.uint8)
    assert ctx.raw("alsgd_export_state", small.ctypes.data, small.size) == B.E_NOMEM
    other = B.Context(tensors, 4, 4, 0.9, 0.7, align_elems=8)                                # N differs
    assert other.raw("alsgd_import_state", image.ctypes.data, image.size) == B.E_ARG
    other.close()
    other = B.Context(tensors, 3, 3, 0.9, 0.7, align_elems=8)                                # W differs
    assert other.raw("alsgd_import_state", image.ctypes.data, image.size) == B.E_ARG
    other.close(); ctx.close()
