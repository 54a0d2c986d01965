"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the same seeded
inputs.  fp32 state within 2e-6*max(1,|ref|) (and, because both sides do the same IEEE operations in
the same order, bit for bit); bf16 replicas and all bookkeeping bit-exact."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from harness import Pair, assert_fp32
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu

SEED = synth.SEED


def dev(x):
    return torch.from_numpy(x).cuda()


def start(pair, seed=SEED):
    theta0 = synth.theta0(pair.tensors, pair.offsets, pair.P, seed)
    pair.set_global(theta0)
    for w in range(pair.W):
        pair.pull(w)
    return theta0


# --------------------------------------------------------------------------------------------------
# Flat 2^20 vector, 4 workers, N=4, 16 round-robin single arrivals (the small configuration)
# --------------------------------------------------------------------------------------------------
def test_flat_vector_single_arrivals():
    P = 1 << 20
    pair = Pair(synth.flat_tensors(P), 4, 4, 0.9, 0.7, replica=False)
    start(pair, SEED + 1)
    pair.check_all("after pull")
    order = synth.round_robin_order(4, 16, SEED + 1)
    visits = [0] * 4
    for a, w in enumerate(order):
        z = synth.normal_vec(P, 1e-3, SEED + 1, synth.STREAM_DELTA, sub=w * 64 + visits[w])
        visits[w] += 1
        pair.perturb(w, dev(z), z)
        info = pair.arrive([w], reseed=False, norm=True)
        assert info[0]["boundary"] == ((a + 1) % 4 == 0)
        pair.check_server(f"arrival {a}")
        pair.pull(w)
        pair.check_worker(w, f"arrival {a}")
    pair.close()


# --------------------------------------------------------------------------------------------------
# Ragged layouts: tails, padding, segment edges inside a vector, c != 0, N = 3, both pseudo-gradient
# bases, batches with a boundary anywhere (also k > N), AdamW on decayed / undecayed tensors
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("align,pg_current,c,N", [(8, False, 0.0, 3), (1, False, 0.0, 4), (1, True, 0.0, 2),
                                                  (4, False, 0.2, 3), (1, True, 0.5, 2), (128, False, 0.0, 1)])
def test_ragged_layout_batches_and_adamw(align, pg_current, c, N):
    tensors = synth.ragged_tensors()
    W = 5
    pair = Pair(tensors, W, N, 0.9, 0.7, c=c, pg_current=pg_current, align=align)
    P = pair.P
    start(pair, SEED + 2)
    steps = [0] * W
    batches = [[0], [1, 2], [3, 4, 0], [1, 2, 3, 4], [0, 1, 2, 3, 4], [4], [3, 2], [1, 0, 4, 2, 3]]
    for b, ids in enumerate(batches):
        for w in ids:
            for _ in range(1 + (w + b) % 3):
                steps[w] += 1
                g = synth.zero_padding(synth.normal_vec(P, 1e-2, SEED + 2, synth.STREAM_GRAD, sub=w * 100 + steps[w]),
                                       tensors, pair.offsets)
                pair.inner_adamw(w, dev(g), g, steps[w], 1e-3)
            pair.check_worker(w, f"batch {b} after AdamW")
        pair.arrive(ids, reseed=True, norm=True)
        pair.check_all(f"batch {b}")
    pair.close()


@pytest.mark.parametrize("P", [1, 2, 3, 5, 7, 1023, (1 << 20) + 3])
def test_odd_sizes(P):
    pair = Pair(synth.flat_tensors(P), 2, 2, 0.9, 0.7, align=1)
    start(pair, SEED + 3)
    for rnd in range(3):
        for w in range(2):
            g = synth.normal_vec(P, 1e-2, SEED + 3, synth.STREAM_GRAD, sub=rnd * 2 + w)
            pair.inner_adamw(w, dev(g), g, rnd + 1, 1e-3)
        pair.arrive([1, 0] if rnd % 2 else [0, 1], reseed=True, norm=True)
        pair.check_all(f"round {rnd}")
    pair.close()


def test_more_arrivals_than_one_launch_holds():
    """k = 11 > 8: the batch is split over launches; every worker is still re-seeded with the final theta."""
    tensors = synth.ragged_tensors()
    W = 12
    pair = Pair(tensors, W, 4, 0.9, 0.7, align=8)
    start(pair, SEED + 4)
    for rnd in range(2):
        for w in range(W):
            z = synth.normal_vec(pair.P, 1e-3, SEED + 4, synth.STREAM_DELTA, sub=rnd * W + w)
            pair.perturb(w, dev(z), z)
        pair.arrive([5, 0, 11, 3, 7, 1, 9, 2, 10, 4, 8], reseed=True, norm=True)
        pair.check_all(f"round {rnd}")
        pair.arrive([6], reseed=True)
        pair.check_all(f"round {rnd} single")
    pair.close()


# --------------------------------------------------------------------------------------------------
# ~23M transformer layout, 4 heterogeneous workers, DyLU inner steps, host scheduler, 64 arrivals
# --------------------------------------------------------------------------------------------------
def scheduled_arrivals(W, speeds, H, n_arrivals, tau_grace, seed):
    steps = B.alsgd_dylu_steps(speeds, H)
    assert steps == oracle.dylu(speeds, H)
    dur = synth.job_durations(speeds, steps, n_arrivals + 2, seed)
    s = B.Scheduler(W, tau_grace)
    rounds = [0] * W
    for w in range(W):
        s.dispatch(w, dur[w, 0], steps[w])
    batches = []
    n = 0
    while n < n_arrivals:
        ids, _, _ = s.next_batch()
        ids = ids[:n_arrivals - n]
        batches.append(ids)
        n += len(ids)
        for w in ids:
            rounds[w] += 1
            s.dispatch(w, dur[w, rounds[w]], steps[w])
    ow, _, ob = oracle.schedule(dur, steps, tau_grace, 10**18, n_arrivals)
    assert [w for b in batches for w in b] == ow                      # arrival order: bit-exact
    assert [i for i, b in enumerate(batches) for _ in b] == ob
    return steps, batches


def test_transformer_23m_heterogeneous_dylu():
    tensors = synth.layout_23m()
    W, speeds = 4, [1.0, 1.5, 2.0, 3.0]
    pair = Pair(tensors, W, 4, 0.9, 0.7, n_sample=150_000)
    P = pair.P
    assert P == 22_914_816
    steps, batches = scheduled_arrivals(W, speeds, 50, 64, 0.0, SEED + 5)
    assert steps == [16, 25, 33, 50]
    G = 4
    pool = [synth.zero_padding(synth.normal_vec(P, 1e-2, SEED + 5, synth.STREAM_GRAD, sub=i), tensors, pair.offsets)
            for i in range(G)]
    pool_dev = [dev(g) for g in pool]
    start(pair, SEED + 5)
    life = [0] * W
    for b, ids in enumerate(batches):
        for w in ids:
            for _ in range(steps[w]):
                life[w] += 1
                i = synth.grad_pool_index(w, life[w], G)
                pair.inner_adamw(w, pool_dev[i], pool[i], life[w], 1e-3)
            pair.check_worker(w, f"batch {b} before arrival")
        pair.arrive(ids, reseed=True)
        pair.check_server(f"batch {b}")
        for w in ids:
            pair.check_worker(w, f"batch {b} after re-seed")
    assert pair.orc.t == 64
    pair.close()


# --------------------------------------------------------------------------------------------------
# ~23M layout, 16 workers, N=16, batches of k=4 through the multi-arrival kernel, random staleness;
# the same arrival list through single arrivals must give bitwise the same state
# --------------------------------------------------------------------------------------------------
def test_transformer_23m_sixteen_workers_batches_of_four():
    tensors = synth.layout_23m()
    W, k = 16, 4
    batches = synth.staleness_batches(W, k, 16, 15, SEED + 6)
    pair = Pair(tensors, W, 16, 0.9, 0.7, n_sample=100_000)
    single = B.Context(tensors, W, 16, 0.9, 0.7)
    P = pair.P
    theta0 = start(pair, SEED + 6)
    single.alsgd_set_global(theta0)
    for w in range(W):
        single.alsgd_pull(w)
    zpool = [synth.normal_vec(P, 1e-3, SEED + 6, synth.STREAM_DELTA, sub=i) for i in range(3)]
    zdev = [dev(z) for z in zpool]
    visit = 0
    stale_seen = []
    for b, ids in enumerate(batches):
        for w in ids:
            zi = (visit * 7 + w) % 3
            visit += 1
            pair.perturb(w, zdev[zi], zpool[zi])
            single.alsgd_worker_state_ptrs(w)["p"].sub_(zdev[zi])
        info = pair.arrive(ids, reseed=True)
        stale_seen += [i["staleness"] for i in info]
        for w in ids:
            single.alsgd_arrive([w], 0)
        for w in ids:
            single.alsgd_pull(w)
        pair.check_server(f"batch {b}")
        for w in ids:
            pair.check_worker(w, f"batch {b}")
        a = pair.ctx.alsgd_state_ptrs()
        s = single.alsgd_state_ptrs()
        single.alsgd_sync()
        for name, x, y in zip(("theta", "m", "Delta"), a, s):
            assert torch.equal(x.view(torch.int32), y.view(torch.int32)), f"{name}: batch != singles at batch {b}"
        for w in ids:
            va, vs = pair.ctx.alsgd_worker_state_ptrs(w), single.alsgd_worker_state_ptrs(w)
            for key in ("p", "base"):
                assert torch.equal(va[key].view(torch.int32), vs[key].view(torch.int32))
            assert torch.equal(va["replica"], vs["replica"])
    assert pair.orc.t == 64 and max(stale_seen) > 4
    single.close()
    pair.close()


# --------------------------------------------------------------------------------------------------
# ~110M layout at full size, in the launch configuration the benchmark times; sampled oracle
# --------------------------------------------------------------------------------------------------
def test_transformer_110m_lognormal_deltas():
    tensors = synth.layout_110m()
    W, speeds = 4, [1.0, 1.5, 2.0, 3.0]
    pair = Pair(tensors, W, 4, 0.9, 0.7, n_sample=200_000)
    P = pair.P
    assert P == 109_549_056
    _, batches = scheduled_arrivals(W, speeds, 50, 128, 0.0, SEED + 7)
    zpool = [synth.normal_vec(P, 1.0, SEED + 7, synth.STREAM_DELTA, sub=i) for i in range(2)]
    gpool = [synth.zero_padding(synth.normal_vec(P, 1e-2, SEED + 7, synth.STREAM_GRAD, sub=i), tensors, pair.offsets)
             for i in range(2)]
    zdev, gdev = [dev(z) for z in zpool], [dev(g) for g in gpool]
    numels = torch.tensor([t.numel for t in tensors], device="cuda")
    start(pair, SEED + 7)
    life = [0] * W
    visit = 0
    for b, ids in enumerate(batches):
        for w in ids:
            scales = synth.lognormal_tensor_scales(len(tensors), visit, seed=SEED + 7).astype(np.float32)
            s_np = synth.per_element_scale(tensors, pair.offsets, P, scales)
            s_dev = torch.repeat_interleave(torch.from_numpy(scales).cuda(), numels)
            assert s_dev.numel() == P                 # the 110M layout has no padding
            zi = visit % 2
            visit += 1
            pair.perturb(w, zdev[zi], zpool[zi], s_dev, s_np)
            life[w] += 1
            gi = synth.grad_pool_index(w, life[w], 2)
            pair.inner_adamw(w, gdev[gi], gpool[gi], life[w], 1e-3)
        pair.arrive(ids, reseed=True)
        if b % 8 == 7 or b < 4:
            pair.check_server(f"batch {b}")
            for w in ids:
                pair.check_worker(w, f"batch {b}")
    pair.check_all("end")
    assert pair.orc.t == 128
    pair.close()


@pytest.mark.parametrize("k,N", [(1, 8), (2, 8), (4, 8), (8, 8), (8, 4)])
def test_transformer_110m_eight_workers_batch_sweep(k, N):
    tensors = synth.layout_110m()
    W = 8
    pair = Pair(tensors, W, N, 0.9, 0.7, n_sample=100_000)
    P = pair.P
    gpool = [synth.zero_padding(synth.normal_vec(P, 1e-2, SEED + 8, synth.STREAM_GRAD, sub=i), tensors, pair.offsets)
             for i in range(2)]
    gdev = [dev(g) for g in gpool]
    start(pair, SEED + 8)
    order = list(synth.rng(SEED + 8, synth.STREAM_ORDER, k).permutation(W))
    life = [0] * W
    for rnd in range(2):
        for w in range(W):
            for _ in range(10 if rnd == 0 else 2):
                life[w] += 1
                gi = synth.grad_pool_index(w, life[w], 2)
                pair.inner_adamw(w, gdev[gi], gpool[gi], life[w], 1e-3)
        for i in range(0, W, k):
            pair.arrive([int(w) for w in order[i:i + k]], reseed=True)
            pair.check_server(f"round {rnd} batch {i // k}")
        pair.check_all(f"round {rnd}")
    pair.close()


def test_reseeded_parameters_are_read_from_the_snapshot_until_written():
    """After a dispatch the library does not store the worker's parameters a second time; every reader
    (AdamW, an arrival, alsgd_get_worker_params) must still see them.  No device pointer of a worker is
    requested between the re-seed and the next use, so the deferred copy is never forced."""
    tensors = synth.ragged_tensors()
    W = 4
    pair = Pair(tensors, W, 3, 0.9, 0.7, align=8)
    P = pair.P
    pair.set_global(synth.theta0(tensors, pair.offsets, P, SEED + 9))
    for w in range(W):
        pair.pull(w)
    got = torch.empty(P, dtype=torch.float32, device="cuda")
    life = [0] * W

    def adam(w):
        life[w] += 1
        g = synth.zero_padding(synth.normal_vec(P, 1e-2, SEED + 9, synth.STREAM_GRAD, sub=w * 50 + life[w]), tensors, pair.offsets)
        pair.inner_adamw(w, dev(g), g, life[w], 1e-3)

    def check_params(w, where):
        pair.ctx.alsgd_get_worker_params(w, got)
        pair.ctx.alsgd_sync()
        assert_fp32(f"params[{w}] {where}", pair.fetch(got), pair.orc.p[w])

    adam(0); adam(0); adam(1)
    pair.arrive([0, 2, 1], reseed=True)          # worker 2 arrives untouched: its pseudo-gradient is exactly zero
    pair.check_server("first window")
    for w in (0, 1, 2):
        check_params(w, "after re-seed")         # equals theta, read through the snapshot
    adam(0); adam(2)                             # first step after the re-seed reads the shared snapshot
    check_params(0, "after AdamW")
    pair.arrive([2], reseed=True)
    pair.arrive([1, 3], reseed=True)             # 1 never ran a step since its dispatch; 3 never since the start
    adam(1); adam(3); adam(0)
    pair.arrive([0, 3, 1, 2], reseed=True)
    pair.check_server("last window")
    for w in range(W):
        check_params(w, "end")
    pair.check_all("end")
    pair.close()


# --------------------------------------------------------------------------------------------------
# Host gradients, diagnostics, error paths (all made on the host; nothing here faults the device)
# --------------------------------------------------------------------------------------------------
def test_host_gradients_through_staging_equal_device_gradients():
    tensors = synth.ragged_tensors()
    a = B.Context(tensors, 1, 4, 0.9, 0.7, grad_staging=True, align_elems=8)
    b = B.Context(tensors, 1, 4, 0.9, 0.7, align_elems=8)
    theta0 = synth.theta0(tensors, a.offsets, a.P, SEED)
    for c in (a, b):
        c.alsgd_set_global(theta0)
        c.alsgd_pull(0)
    for s in range(1, 4):
        g = synth.normal_vec(a.P, 1e-2, SEED, synth.STREAM_GRAD, sub=s)
        a.alsgd_inner_adamw(0, torch.from_numpy(g).pin_memory(), s, 1e-3)
        a.alsgd_sync()
        b.alsgd_inner_adamw(0, dev(g), s, 1e-3)
    va, vb = a.alsgd_worker_state_ptrs(0), b.alsgd_worker_state_ptrs(0)
    a.alsgd_sync(); b.alsgd_sync()
    for key in ("p", "adam_m", "adam_v", "replica"):
        assert torch.equal(va[key], vb[key])
    # without the staging buffer a host pointer is refused
    g = synth.normal_vec(b.P, 1e-2, SEED, synth.STREAM_GRAD, sub=9)
    assert b.raw("alsgd_inner_adamw", 0, g.ctypes.data, 0, 4, C.c_float(1e-3)) == B.E_UNSUPPORTED
    a.close(); b.close()


@pytest.mark.parametrize("align", [1, 8])
def test_bf16_gradients_equal_their_fp32_widening(align):
    """bf16 gradients are widened exactly, so the step must equal the fp32 step on the widened values
    (and therefore the oracle's), from device memory and through the host staging buffer."""
    tensors = synth.ragged_tensors()
    pair = Pair(tensors, 2, 4, 0.9, 0.7, align=align, grad_staging=True)
    start(pair, SEED + 12)
    for s in range(1, 4):
        g = synth.zero_padding(synth.normal_vec(pair.P, 1e-2, SEED + 12, synth.STREAM_GRAD, sub=s), tensors, pair.offsets)
        g16 = torch.from_numpy(g).to(torch.bfloat16)
        wide = g16.to(torch.float32).numpy()
        pair.ctx.alsgd_inner_adamw_bf16(0, g16.cuda(), s, 1e-3)
        pair.orc.inner_adamw(0, pair.take(wide), s, 1e-3)
        host = g16.pin_memory()
        pair.ctx.alsgd_inner_adamw_bf16(1, host, s, 1e-3)
        pair.ctx.alsgd_sync()
        pair.orc.inner_adamw(1, pair.take(wide), s, 1e-3)
        pair.check_worker(0, f"step {s} device bf16")
        pair.check_worker(1, f"step {s} host bf16")
    pair.arrive([0, 1], reseed=True)
    pair.check_all("after arrival")
    pair.close()


def test_extreme_values_denormals_signed_zeros_overflow():
    """The bit-for-bit claim at the edges of binary32: denormals (no flush to zero on either side), signed
    zeros, values whose products overflow to infinity or underflow to zero, and huge/tiny mixes in AdamW's
    divisions and square root."""
    P = 8192
    tensors = [synth.Tensor("a", P // 2, True, "matrix"), synth.Tensor("b", P // 2, False, "gain")]
    pair = Pair(tensors, 3, 2, 0.9, 0.7, c=0.25, align=1)
    specials = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-40, -3e-39, 1.1754944e-38, -1.1754942e-38, 1e-30, -1e-20,
                         1e-10, 1.0, -1.0, 3.0, 1e10, -1e19, 1e20, -1e30, 3e38, -3.4028235e38, 65504.0, 1e-7], np.float32)
    r = np.random.default_rng(21)

    def special_vec():
        return np.ascontiguousarray(specials[r.integers(0, specials.shape[0], P)])

    with np.errstate(all="ignore"):
        pair.set_global(special_vec())
        for w in range(3):
            pair.pull(w)
        for rnd in range(4):
            for w in range(3):
                z = special_vec()
                pair.perturb(w, dev(z), z)
                g = special_vec()
                pair.inner_adamw(w, dev(g), g, rnd + 1, 1e-3)
            pair.arrive([[0, 1, 2], [2, 0], [1], [1, 2, 0]][rnd], reseed=True, norm=True)
            pair.check_all(f"round {rnd}")
    th = pair.orc.theta
    assert np.isinf(th).any() or np.isnan(th).any()          # the inputs did reach overflow
    v = pair.orc.av[0]
    assert ((v > 0) & (v < 1.1754944e-38)).any()             # ... and the denormal range (second moments of tiny gradients)
    pair.close()


def test_nothing_is_written_past_the_end_of_a_slice():
    """Every arena slice starts on a 256-byte boundary; with P = 4099 + ... odd sizes the bytes between the end
    of a slice and the next boundary belong to nobody.  They are filled with a canary before the run and must
    still hold it afterwards (vector stores, tails, re-seed and bf16 stores all end exactly at P)."""
    tensors = synth.ragged_tensors()
    W = 5
    pair = Pair(tensors, W, 2, 0.9, 0.7, align=1)
    P = pair.P
    assert P % 64 != 0
    ctx = pair.ctx
    arena, base = ctx.arena, ctx.arena.data_ptr()
    gaps = []

    def gap_after(tensor):
        if tensor is None:
            return
        end = tensor.data_ptr() + tensor.numel() * tensor.element_size() - base
        stop = (end + 255) // 256 * 256
        if stop > end and stop <= arena.numel():
            gaps.append((end, stop))

    for v in ctx.alsgd_state_ptrs():
        gap_after(v)
    for w in range(W):
        for v in ctx.alsgd_worker_state_ptrs(w).values():
            gap_after(v)
    assert len(gaps) >= 3 + 5 * W - W
    ctx.alsgd_sync()
    for lo, hi in gaps:
        arena[lo:hi] = 0xA5
    start(pair, SEED + 13)
    life = [0] * W
    for b, ids in enumerate([[0, 1], [2], [3, 4, 0], [1, 2, 3, 4, 0], [2, 4]]):
        for w in ids:
            life[w] += 1
            g = synth.zero_padding(synth.normal_vec(P, 1e-2, SEED + 13, synth.STREAM_GRAD, sub=w * 10 + life[w]), tensors, pair.offsets)
            pair.inner_adamw(w, dev(g), g, life[w], 1e-3)
        pair.arrive(ids, reseed=True, norm=True)
    pair.check_all("canary run")
    for lo, hi in gaps:
        assert bool((arena[lo:hi] == 0xA5).all()), f"bytes {lo}..{hi} of the arena were overwritten"
    pair.close()


def test_error_codes_leave_state_untouched():
    tensors = synth.flat_tensors(4096)
    ctx = B.Context(tensors, 3, 2, 0.9, 0.7)
    theta0 = synth.theta0(tensors, ctx.offsets, ctx.P, SEED)
    ctx.alsgd_set_global(theta0)
    ids = lambda *x: (C.c_uint32 * len(x))(*x)
    g = dev(np.zeros(ctx.P, np.float32))
    assert ctx.raw("alsgd_arrive", ids(0), 1, 0, None) == B.E_STATE          # never pulled
    assert ctx.raw("alsgd_inner_adamw", 0, g.data_ptr(), 1, 1, C.c_float(1e-3)) == B.E_STATE
    for w in range(3):
        ctx.alsgd_pull(w)
    assert ctx.raw("alsgd_arrive", ids(0, 0), 2, 0, None) == B.E_ARG         # duplicate
    assert ctx.raw("alsgd_arrive", ids(0, 3), 2, 0, None) == B.E_RANGE       # id out of range
    assert ctx.raw("alsgd_arrive", ids(0, 1, 2, 0), 4, 0, None) == B.E_ARG   # k > W
    assert ctx.raw("alsgd_arrive", ids(0), 1, 64, None) == B.E_ARG           # unknown flag
    assert ctx.raw("alsgd_arrive", None, 0, 0, None) == B.OK                 # k = 0: no-op
    assert ctx.raw("alsgd_pull", 3) == B.E_RANGE
    assert ctx.raw("alsgd_inner_adamw", 0, g.data_ptr(), 1, 0, C.c_float(1e-3)) == B.E_ARG   # step 0
    assert ctx.raw("alsgd_inner_adamw", 0, g.data_ptr() + 4, 1, 1, C.c_float(1e-3)) == B.E_ARG  # misaligned
    assert ctx.alsgd_counters() == (0, 0)
    theta, m, delta = ctx.alsgd_state_ptrs()
    ctx.alsgd_sync()
    assert np.array_equal(theta.cpu().numpy(), theta0) and not m.any() and not delta.any()
    ctx.alsgd_arrive([1], 0)                                                 # arrives without re-seed ...
    assert ctx.raw("alsgd_arrive", ids(1), 1, 0, None) == B.E_STATE          # ... so it cannot arrive again
    ctx.alsgd_pull(1)
    ctx.alsgd_arrive([1], B.ARRIVE_RESEED)
    assert ctx.alsgd_counters() == (2, 0)
    ctx.close()


def test_nonfinite_worker_is_flagged_not_trapped():
    tensors = synth.flat_tensors(10_000)
    pair = Pair(tensors, 2, 4, 0.9, 0.7)
    start(pair)
    z = np.zeros(pair.P, np.float32)
    z[1234] = np.inf
    z[77] = 1.0
    pair.perturb(0, dev(z), z)
    z2 = synth.normal_vec(pair.P, 1e-3, SEED, synth.STREAM_DELTA)
    pair.perturb(1, dev(z2), z2)
    info = pair.arrive([1, 0], reseed=True, norm=True)
    assert [i["nonfinite"] for i in info] == [0, 1]
    pair.check_all("after poisoned arrival")       # NaN/Inf propagate exactly as the definition says
    pair.close()


@pytest.mark.parametrize("pg_current,buffered,N", [(False, False, 4), (True, False, 3), (False, True, 16), (True, True, 2)])
def test_nonfinite_flags_per_arrival_in_every_mode(pg_current, buffered, N):
    """The per-arrival non-finite flag comes from a replay that only runs where the state left by the batch is
    not finite.  Poisoned entries in a vector body, in the scalar tail and in several arrivals of one batch; an
    overflow that is not a non-finite entry; batches that follow on an already poisoned model; batches of eight
    that share one dispatch snapshot."""
    P = 4 * 4099 + 3                                   # scalar tail of three elements
    W = 8
    pair = Pair(synth.flat_tensors(P), W, N, 0.9, 0.7, align=1, pg_current=pg_current, buffered=buffered)
    start(pair, SEED + 17)
    r = np.random.default_rng(17)

    def round_of(ids, poison):
        for w in ids:
            z = synth.normal_vec(P, 1e-3, SEED + 17, synth.STREAM_DELTA, sub=int(r.integers(0, 1 << 20)))
            for where, value in poison.get(w, []):
                z[where] = value
            pair.perturb(w, dev(z), z)
        with np.errstate(all="ignore"):
            info = pair.arrive(ids, reseed=True, norm=True)      # flags and norms are compared with the oracle inside
            pair.check_all(f"batch {ids}")
        return [i["nonfinite"] for i in info]

    assert round_of([0, 1, 2, 3, 4, 5, 6, 7], {}) == [0] * 8                        # clean, distinct snapshots
    assert round_of([3, 1, 4, 0, 5, 2, 7, 6], {}) == [0] * 8                        # clean, one shared snapshot
    # a finite entry large enough to overflow theta and the sum of squares: not a non-finite entry
    flags = round_of([2, 6], {6: [(11, np.float32(-3e38))]})
    assert flags == ([0, 0] if not pg_current else flags) and flags[0] == 0
    # Inf in a vector body of one arrival, NaN in the scalar tail of another, both in one batch of eight
    flags = round_of([7, 0, 1, 2, 3, 4, 5, 6], {1: [(4000, np.inf)], 4: [(P - 1, np.nan)]})
    if not pg_current:
        assert flags == [0, 0, 1, 0, 0, 1, 0, 0]
    else:                                             # later arrivals see the poisoned running theta
        assert flags[:2] == [0, 0] and flags[2] == 1 and flags[5] == 1
    # the model is poisoned now; against the dispatch snapshot (also poisoned at those elements) or the running theta
    # the oracle decides, element by element, what each arrival's pseudo-gradient holds
    round_of([0, 1], {})
    round_of([5], {5: [(123, -np.inf)]})
    pair.close()
