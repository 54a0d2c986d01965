"""Pins for the oracle's AdamW step, bf16 rounding, DyLU (Eq. 6), learning-rate schedule (Eq. 3),
re-seed and the faked-time scheduler (Algorithm 2 + Algorithm 5)."""
import math

import numpy as np
import pytest
import torch

import oracle
from conftest import read_golden


# ---- AdamW -----------------------------------------------------------------------------------------

def one(x):
    return np.array([x], np.float32)


def test_adamw_hand_case():
    for b1, b2, lr, wd, eps, p0, g, dec, m_e, v_e, p_e in read_golden("adamw_hand.txt"):
        p, m, v = one(p0), one(0), one(0)
        rep = np.zeros(1, np.uint16)
        oracle.adamw(p, m, v, one(g), rep, np.array([int(dec)], np.uint8), 1, lr, b1, b2, eps, wd)
        assert (m[0], v[0], p[0]) == (np.float32(m_e), np.float32(v_e), np.float32(p_e))
        assert rep[0] == oracle.bf16_rne_bits(int(p.view(np.uint32)[0]))


def test_adamw_first_step_is_sign_step_without_eps_and_decay():
    r = np.random.default_rng(0)
    g = r.standard_normal(500).astype(np.float32)
    g[g == 0] = 1
    p0 = r.standard_normal(500).astype(np.float32)
    p, m, v = p0.copy(), np.zeros(500, np.float32), np.zeros(500, np.float32)
    oracle.adamw(p, m, v, g, None, None, 1, 0.125, 0.9, 0.95, 0.0, 0.0)
    np.testing.assert_allclose(p, p0 - 0.125 * np.sign(g), rtol=0, atol=1e-6)


def test_adamw_constant_gradient_keeps_sign_stepping():
    p, m, v = one(3.0), one(0), one(0)
    for s in range(1, 21):
        oracle.adamw(p, m, v, one(-0.3), None, None, s, 0.0625, 0.9, 0.95, 0.0, 0.0)
    assert abs(p[0] - (3.0 + 20 * 0.0625)) < 1e-5


def test_adamw_zero_gradient_is_pure_decoupled_decay():
    lr, wd = 1e-3, 0.1
    p, m, v = one(2.0), one(0), one(0)
    ref = np.float32(2.0)
    for s in range(1, 51):
        oracle.adamw(p, m, v, one(0.0), None, np.ones(1, np.uint8), s, lr, 0.9, 0.95, 1e-8, wd)
        ref = ref - np.float32(lr) * (np.float32(0.0) + np.float32(wd) * ref)
        assert p[0] == ref
    assert m[0] == 0 and v[0] == 0
    assert abs(p[0] - 2.0 * (1 - lr * wd) ** 50) < 1e-6
    # an undecayed element with zero gradient never moves
    q = one(2.0)
    oracle.adamw(q, one(0), one(0), one(0.0), None, np.zeros(1, np.uint8), 1, lr, 0.9, 0.95, 1e-8, wd)
    assert q[0] == 2.0


def test_adamw_against_library_adamw_in_double():
    """torch.optim.AdamW (CPU, float64) is an independent statement of the textbook rule."""
    r = np.random.default_rng(4)
    n = 4096
    p0 = r.standard_normal(n).astype(np.float32)
    grads = (1e-2 * r.standard_normal((12, n))).astype(np.float32)
    lr, b1, b2, eps, wd = 1e-3, 0.9, 0.95, 1e-8, 0.1
    tp = torch.tensor(p0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([tp], lr=float(np.float32(lr)), betas=(float(np.float32(b1)), float(np.float32(b2))),
                            eps=float(np.float32(eps)), weight_decay=float(np.float32(wd)))
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    rep = np.zeros(n, np.uint16)
    dec = np.ones(n, np.uint8)
    for s in range(12):
        tp.grad = torch.tensor(grads[s], dtype=torch.float64)
        opt.step()
        oracle.adamw(p, m, v, grads[s], rep, dec, s + 1, lr, b1, b2, eps, wd)
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=2e-6, atol=2e-6)
    st = opt.state[tp]
    np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=1e-5, atol=1e-9)
    np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-5, atol=1e-12)
    np.testing.assert_array_equal(rep, oracle.cast_bf16(p))


def test_adamw_range_arguments_touch_only_the_range():
    n = 32
    p, m, v = np.ones(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.float32)
    oracle.adamw(p, m, v, np.ones(n, np.float32), None, None, 1, 0.5, 0.5, 0.75, 0.0, 0.0, lo=5, hi=9)
    assert np.all(p[:5] == 1) and np.all(p[9:] == 1) and np.all(p[5:9] == 0.5)


# ---- bf16 round-to-nearest-even -----------------------------------------------------------------------

def _neighbour_rne(bits):
    """Second, differently written rounding: pick the nearer of the two bf16 neighbours in exact
    arithmetic, ties to the even mantissa."""
    bits = bits.astype(np.uint64)
    lo = (bits >> np.uint64(16)) << np.uint64(16)
    hi = lo + np.uint64(0x10000)
    # within one sign, ordering of magnitudes equals ordering of bit patterns
    d_lo = bits - lo
    d_hi = hi - bits
    up = (d_hi < d_lo) | ((d_hi == d_lo) & (((lo >> np.uint64(16)) & np.uint64(1)) == 1))
    return (np.where(up, hi, lo) >> np.uint64(16)).astype(np.uint16)


def _check_bits(bits):
    f = bits.view(np.float32)
    got = oracle.cast_bf16(f)
    nan = np.isnan(f)
    np.testing.assert_array_equal(got[~nan], _neighbour_rne(bits[~nan]))
    with np.errstate(all="ignore"):
        lib = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got[~nan], lib[~nan])
    # NaN stays NaN, sign kept, quiet bit set
    assert np.all((got[nan] & 0x7FFF) == 0x7FC0)
    assert np.all((got[nan] >> 15) == (bits[nan] >> 31).astype(np.uint16))


def test_bf16_every_high_half_at_the_critical_low_halves():
    hi = np.arange(1 << 16, dtype=np.uint32) << 16
    for low in (0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF):
        _check_bits((hi | np.uint32(low)).astype(np.uint32))


def test_bf16_strided_sweep_of_all_bit_patterns():
    for start in (0, 1, 12345):
        bits = (np.arange(start, 1 << 32, 509, dtype=np.uint64) & 0xFFFFFFFF).astype(np.uint32)
        _check_bits(bits)


def test_bf16_named_values():
    f = lambda x: int(np.array([x], np.float32).view(np.uint32)[0])
    assert oracle.bf16_rne_bits(f(1.0)) == 0x3F80
    assert oracle.bf16_rne_bits(0x3F808000) == 0x3F80          # tie -> even (down)
    assert oracle.bf16_rne_bits(0x3F818000) == 0x3F82          # tie -> even (up)
    assert oracle.bf16_rne_bits(0x7F7FFFFF) == 0x7F80          # max float rounds to +inf
    assert oracle.bf16_rne_bits(0xFF7FFFFF) == 0xFF80
    assert oracle.bf16_rne_bits(0x80000000) == 0x8000          # -0
    assert oracle.bf16_rne_bits(0x00008000) == 0x0000          # subnormal tie -> even
    assert oracle.bf16_rne_bits(0x00018000) == 0x0002


def test_reseed_copies_and_casts():
    r = np.random.default_rng(9)
    theta = r.standard_normal(100).astype(np.float32)
    p, base, rep = np.zeros(100, np.float32), np.zeros(100, np.float32), np.zeros(100, np.uint16)
    oracle.reseed(theta, p, base, rep)
    assert np.array_equal(p, theta) and np.array_equal(base, theta)
    assert np.array_equal(rep, oracle.cast_bf16(theta))


# ---- Eq. 6 and Eq. 3 -------------------------------------------------------------------------------------

def test_dylu_values():
    assert oracle.dylu([1, 1.5, 2, 3], 50) == [16, 25, 33, 50]     # floor(50/3)=16, 25, floor(100/3)=33, 50
    assert oracle.dylu([2, 2, 2], 50) == [50, 50, 50]
    assert oracle.dylu([1e-9, 1.0], 50) == [1, 50]                # never fewer than one step
    assert oracle.dylu([3, 1], 7) == [7, 2]


def test_lr_schedule_endpoints_and_clamps():
    emax, emin, tw, T = 0.1, 1e-6, 1000, 88000
    assert oracle.lr_at(emax, emin, tw, T, 0) == 0.0
    assert oracle.lr_at(emax, emin, tw, T, 500) == pytest.approx(0.05, rel=1e-12)
    assert oracle.lr_at(emax, emin, tw, T, tw) == pytest.approx(emax, rel=1e-12)
    mid = tw + (T - tw) // 2
    assert oracle.lr_at(emax, emin, tw, T, mid) == pytest.approx(emin + 0.5 * (emax - emin), rel=1e-9)
    assert oracle.lr_at(emax, emin, tw, T, T) == pytest.approx(emin, abs=1e-15)
    assert oracle.lr_at(emax, emin, tw, T, 10 * T) == pytest.approx(emin, abs=1e-15)   # ratio clamped at 1
    assert oracle.lr_at(emax, emin, tw, tw, tw + 5) == pytest.approx(emin, abs=1e-15)  # zero-length decay
    assert oracle.lr_at(emax, emin, tw, 10, tw + 5) == pytest.approx(emin, abs=1e-15)  # T < warm-up
    q = tw + (T - tw) // 4
    expect = emin + 0.5 * (emax - emin) * (1 + math.cos(math.pi * (q - tw) / (T - tw)))
    assert oracle.lr_at(emax, emin, tw, T, q) == pytest.approx(expect, rel=1e-12)
    assert oracle.lr_at(emax, emin, 0, T, 0) == pytest.approx(emax, rel=1e-12)         # no warm-up


def test_shard_sampling_eq2():
    # sizes 1:1:2 -> shares .25 .25 .5 ; learned 10:30:60 -> shares .1 .3 .6 ; gaps .15, <0, <0 -> only shard 0
    assert oracle.shard_probs([1, 1, 2], [10, 30, 60]) == [1.0, 0.0, 0.0]
    # learned 40:10:50 -> .4 .1 .5 ; gaps <0, .15, 0 -> only shard 1
    assert oracle.shard_probs([1, 1, 2], [40, 10, 50]) == [0.0, 1.0, 0.0]
    # learned 0:25:75 -> 0 .25 .75 ; gaps .25, 0, <0
    assert oracle.shard_probs([1, 1, 2], [0, 25, 75]) == [1.0, 0.0, 0.0]
    # two under-sampled shards share in proportion to their gaps: sizes equal, learned 1:2:5 -> gaps 5/24, 2/24, <0
    p = oracle.shard_probs([1, 1, 1], [1, 2, 5])
    assert p[2] == 0.0 and abs(p[0] - 5 / 7) < 1e-12 and abs(p[1] - 2 / 7) < 1e-12
    # nothing learned yet: proportional to shard size; perfectly balanced: also the size shares
    assert oracle.shard_probs([1, 3], [0, 0]) == [0.25, 0.75]
    assert oracle.shard_probs([1, 3], [5, 15]) == [0.25, 0.75]
    r = np.random.default_rng(0)
    for _ in range(50):
        n = int(r.integers(1, 9))
        p = oracle.shard_probs(r.uniform(1, 10, n), r.uniform(0, 10, n))
        assert abs(sum(p) - 1) < 1e-12 and min(p) >= 0


def test_poly_weight():
    assert oracle.poly_weight(0) == 1.0
    assert oracle.poly_weight(3) == 0.5
    assert oracle.poly_weight(15) == 0.25


# ---- scheduler -----------------------------------------------------------------------------------------

def test_schedule_grace_window_timeline():
    """Three workers A, B, C as in the grace-period figure: B finishes inside A's window and is synced
    right after A, both restart from the same model when the window ends; C opens its own window."""
    dur = np.array([[10.0] * 4, [10.5] * 4, [12.0] * 4])
    w, t, b = oracle.schedule(dur, [50, 50, 50], tau_grace=1.0, t_max=10**9, max_arrivals=9)
    #  batch0: A@10, B@10.5 | restart A,B at 11 -> 21, 21.5.  batch1: C@12 | restart at 13 -> 25.
    #  batch2: A@21, B@21.5 | restart at 22 -> 32, 32.5.      batch3: C@25 | restart at 26 -> 38.
    #  batch4: A@32, B@32.5 | batch5: C@38 ...
    assert w == [0, 1, 2, 0, 1, 2, 0, 1, 2]
    assert t == [10.0, 10.5, 12.0, 21.0, 21.5, 25.0, 32.0, 32.5, 38.0]
    assert b == [0, 0, 1, 2, 2, 3, 4, 4, 5]


def test_schedule_equal_speeds_behave_synchronously():
    dur = np.full((4, 5), 7.0)
    w, t, b = oracle.schedule(dur, [50] * 4, tau_grace=0.0, t_max=10**9, max_arrivals=16)
    assert w == [0, 1, 2, 3] * 4
    assert b == [0] * 4 + [1] * 4 + [2] * 4 + [3] * 4
    assert t == [7.0] * 4 + [14.0] * 4 + [21.0] * 4 + [28.0] * 4


def test_schedule_zero_grace_distinct_times_gives_singletons_in_time_order():
    dur = np.array([[3.0] * 8, [2.0] * 8, [5.0] * 8])
    w, t, b = oracle.schedule(dur, [1, 1, 1], tau_grace=0.0, t_max=10**9, max_arrivals=8)
    # completion times: w1: 2,4,6,8,10  w0: 3,6,9  w2: 5,10 ; tie at 6 -> lower id first, and a tie
    # falls inside a zero-length window, so both land in one batch
    assert w == [1, 0, 1, 2, 0, 1, 1, 0]
    assert t == [2.0, 3.0, 4.0, 5.0, 6.0, 6.0, 8.0, 9.0]
    assert b == [0, 1, 2, 3, 4, 4, 5, 6]


def test_schedule_stops_at_t_max_local_updates():
    dur = np.array([[1.0] * 50, [2.0] * 50])
    w, t, b = oracle.schedule(dur, [10, 20], tau_grace=0.0, t_max=45, max_arrivals=100)
    # t_local after each arrival: 10 (w0@1), then a tie at 2 (w0, w1) -> 20, 40; w0@3 -> 50 >= 45 stops
    assert w == [0, 0, 1, 0]


def test_schedule_invariants_on_random_timelines():
    """What Algorithm 2 with Algorithm 5 guarantees on any input, checked on the oracle's output alone: a window
    is opened by the earliest pending completion; everything completing within tau_grace of it joins, in
    (time, id) order, and nothing that completes within the window is left out; the workers of a window restart
    together at tau_sync + tau_grace, so a worker's next completion is that restart plus its next duration."""
    r = np.random.default_rng(11)
    for case in range(60):
        W = int(r.integers(2, 8))
        R = 12
        dur = r.uniform(0.5, 3.0, size=(W, R))
        if case % 3 == 0:
            dur = np.round(dur * 2) / 2                     # many exact ties
        grace = float(r.choice([0.0, 0.25, 1.0, 4.0]))
        w, t, b = oracle.schedule(dur, [1] * W, grace, 10 ** 9, 5 * W)
        done = [dur[u, 0] for u in range(W)]                # current completion time of every worker's job
        rounds = [0] * W
        pending = set(range(W))
        i = 0
        while i < len(w):
            j = i
            while j < len(w) and b[j] == b[i]:
                j += 1
            batch = list(zip(w[i:j], t[i:j]))
            full = j < len(w)                               # the last window may be cut by max_arrivals
            first_w, tau_sync = batch[0]
            assert tau_sync == min(done[u] for u in pending)                     # earliest pending opens it
            assert all(done[u] == tu for u, tu in batch)                         # reported time = completion time
            assert batch == sorted(batch, key=lambda x: (x[1], x[0]))            # (time, id) order
            assert all(tu - tau_sync <= grace for _, tu in batch)                # inside the window
            if full:
                left = pending - {u for u, _ in batch}
                assert all(not (done[u] - tau_sync <= grace) for u in left)      # nobody inside was left out
            restart = tau_sync + grace
            for u, _ in batch:
                rounds[u] += 1
                if rounds[u] < R:
                    done[u] = restart + dur[u, rounds[u]]
            i = j
