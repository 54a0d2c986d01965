"""Sizes beyond 32-bit offsets: a vector whose buffers are larger than 4 GiB each (byte offsets need 64 bits)
and, when the device has the room, one with more than 2^32 elements (element indices need 64 bits).
Inputs are generated on the device from a seeded generator; the oracle runs on a sample of positions
(random picks, tensor edges, and the neighbourhoods of the 2^30 / 2^31 / 2^32 element marks)."""
import numpy as np
import pytest
import torch

import oracle
from harness import assert_fp32
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu


def fill_normal(view, std, seed):
    gen = torch.Generator(device="cuda").manual_seed(seed)
    step = 1 << 28
    for lo in range(0, view.numel(), step):
        hi = min(lo + step, view.numel())
        view[lo:hi] = torch.randn(hi - lo, generator=gen, device="cuda", dtype=torch.float32) * std


@pytest.mark.parametrize("P,need_gib", [((1 << 30) + 4099, 40), ((1 << 32) + 1029, 150)])
def test_vectors_beyond_32_bit_offsets(P, need_gib):
    free, _ = torch.cuda.mem_get_info()
    if free < need_gib * (1 << 30):
        pytest.skip(f"needs {need_gib} GiB of free device memory")
    a = P // 2 + 1
    tensors = [synth.Tensor("a", a, True, "matrix"), synth.Tensor("b", 7, False, "gain"),
               synth.Tensor("c", P - a - 7, True, "matrix")]
    ctx = B.Context(tensors, 1, 2, 0.9, 0.7, pg_base=B.PG_CURRENT, replica=False, align_elems=1)
    assert ctx.P == P
    r = np.random.default_rng(5)
    marks = [m for m in (1 << 30, 1 << 31, 1 << 32) if m < P]
    parts = [r.integers(0, P, size=150_000, dtype=np.int64), np.arange(0, 16), np.arange(P - 16, P),
             np.arange(a - 8, a + 16)] + [np.arange(m - 8, m + 8) for m in marks]
    idx = np.unique(np.concatenate(parts))
    idx_dev = torch.from_numpy(idx).cuda()
    mask = np.zeros(idx.shape[0], np.uint8)
    mask[(idx < a) | (idx >= a + 7)] = 1
    orc = oracle.OracleServer(idx.shape[0], 1, 2, 0.9, 0.7, pg_current=True, decay=mask, replica=False)

    theta, m, delta = ctx.alsgd_state_ptrs()
    fill_normal(theta, 0.02, 1)
    orc.set_global(theta[idx_dev].cpu().numpy())
    grads = torch.empty(P, dtype=torch.float32, device="cuda")
    fill_normal(grads, 1e-2, 2)
    g_s = grads[idx_dev].cpu().numpy()

    ctx.alsgd_pull(0); orc.pull(0)
    for step in (1, 2):
        ctx.alsgd_inner_adamw(0, grads, step, 1e-3); orc.inner_adamw(0, g_s, step, 1e-3)
        got = ctx.alsgd_arrive([0], B.ARRIVE_RESEED | B.ARRIVE_NANCHECK)
        ref = orc.arrive([0])
        assert got[0]["boundary"] == ref[0]["boundary"] == (step == 2) and got[0]["nonfinite"] == 0
    ctx.alsgd_sync()
    theta, m, delta = ctx.alsgd_state_ptrs()
    w = ctx.alsgd_worker_state_ptrs(0)
    ctx.alsgd_sync()
    for name, dev_t, ref in (("theta", theta, orc.theta), ("m", m, orc.m), ("Delta", delta, orc.Delta),
                             ("p", w["p"], orc.p[0]), ("adam_m", w["adam_m"], orc.am[0]), ("adam_v", w["adam_v"], orc.av[0])):
        assert_fp32(f"{name} at P={P}", dev_t[idx_dev].cpu().numpy(), ref)
    assert float(m.abs().max()) > 0                      # the boundary really updated the momentum everywhere sampled
    ctx.close()
    del grads, ctx
    torch.cuda.empty_cache()


def test_110m_norms_of_batches_of_eight_against_the_oracle_on_the_full_vectors():
    """The diagnostics in the launch configuration the benchmark times (110M elements, eight arrivals in one pass:
    213 963 blocks, one partial per block per arrival, one reduction launch): every arrival's squared norm against
    the oracle's double-precision sum over the complete vectors, first with eight distinct dispatch snapshots, then
    with one shared snapshot, and a non-finite entry in the very last element."""
    import oracle
    tensors = synth.layout_110m()
    W = 8
    ctx = B.Context(tensors, W, 8, 0.9, 0.7)
    plain = B.Context(tensors, W, 8, 0.9, 0.7)               # the same run without diagnostics: same bits expected
    P = ctx.P
    for c in (ctx, plain):
        c.alsgd_set_global(synth.theta0(tensors, ctx.offsets, P, synth.SEED + 31))
        for w in range(W):
            c.alsgd_pull(w)
    z = [torch.from_numpy(synth.normal_vec(P, 1e-3 * (i + 1), synth.SEED + 31, synth.STREAM_DELTA, sub=i)).cuda() for i in range(2)]
    for rnd in range(2):
        ids = [3, 0, 7, 1, 6, 2, 5, 4] if rnd == 0 else [6, 4, 0, 2, 7, 5, 3, 1]
        want = []
        for j, w in enumerate(ids):
            v = ctx.alsgd_worker_state_ptrs(w)
            v["p"].sub_(z[(w + rnd) % 2])
            if rnd == 1 and j == 5:
                v["p"][P - 1] = float("inf")
            base, p = v["base"].cpu().numpy(), v["p"].cpu().numpy()
            want.append(oracle.pg_norm2(base, base, p))
            plain.alsgd_worker_state_ptrs(w)["p"].copy_(v["p"])
        bases = {ctx.alsgd_worker_state_ptrs(w)["base"].data_ptr() for w in ids}
        assert len(bases) == (8 if rnd == 0 else 1)
        info = ctx.alsgd_arrive(ids, B.ARRIVE_RESEED | B.ARRIVE_NORM | B.ARRIVE_NANCHECK)
        for j, (got, (norm, bad)) in enumerate(zip(info, want)):
            assert got["nonfinite"] == bad == (1 if (rnd == 1 and j == 5) else 0)
            if not bad:
                assert abs(got["gnorm2"] - norm) <= 1e-6 * norm, (rnd, j, got["gnorm2"], norm)
        plain.alsgd_arrive(ids, B.ARRIVE_RESEED)
        for a, b in zip(ctx.alsgd_state_ptrs(), plain.alsgd_state_ptrs()):
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    ctx.alsgd_sync()
    plain.alsgd_sync()
    ctx.close()
    plain.close()
