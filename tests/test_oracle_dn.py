"""Pins for the oracle's Delayed-Nesterov arrival (Algorithm 3): hand traces, the paper's printed
closed forms (Eq. 4, Eq. 5), reductions the definition implies, and an exact-rational unrolling of
whole arrival sequences.  A dropped term, a wrong sign, a wrong boundary index or a transposed
operand fails at least one of these."""
from fractions import Fraction
import itertools

import numpy as np
import pytest

import oracle
from conftest import read_golden

SCALES = np.array([1, -1, 2, -2, 0.5, -0.5, 4, -0.25], dtype=np.float32)   # powers of two: exact


def run_trace(rows, N, beta, eps, c, theta0=1.0):
    theta = (theta0 * SCALES).astype(np.float32)
    m = np.zeros(8, np.float32)
    D = np.zeros(8, np.float32)
    for t, row in enumerate(rows):
        g, th, mm, dd, bnd = row
        base = theta.copy()                       # worker seeded with the current model ...
        p = (base - np.float32(g) * SCALES).astype(np.float32)   # ... moved by -g
        b = oracle.dn_arrive(theta, m, D, base, p, t, N, beta, eps, c)
        assert b == bool(bnd)
        np.testing.assert_array_equal(theta, np.float32(th) * SCALES)
        np.testing.assert_array_equal(m, np.float32(mm) * SCALES)
        np.testing.assert_array_equal(D, np.float32(dd) * SCALES)


def test_hand_trace_c0_eight_elements():
    run_trace(read_golden("dn_trace_c0.txt"), N=2, beta=0.5, eps=0.5, c=0.0)


def test_hand_trace_c_quarter_eight_elements():
    run_trace(read_golden("dn_trace_c025.txt"), N=2, beta=0.5, eps=0.5, c=0.25)


def test_eq5_four_identical_arrivals_with_N1():
    # N = 1 makes every arrival a boundary, i.e. the plain Nesterov step of Eq. 4.
    for beta, eps, g, m0, th0, m_exp, th_exp in read_golden("eq5_four_identical.txt"):
        theta = np.full(4, th0, np.float32)
        m = np.full(4, m0, np.float32)
        D = np.zeros(4, np.float32)
        for t in range(4):
            base = theta.copy()
            p = base - np.float32(g)
            assert oracle.dn_arrive(theta, m, D, base, p, t, 1, beta, eps, 0.0) is True
            assert np.all(D == 0)
        np.testing.assert_array_equal(m, np.float32(m_exp))
        np.testing.assert_array_equal(theta, np.float32(th_exp))


def test_eq4_single_nesterov_step_random():
    r = np.random.default_rng(1)
    theta0 = r.standard_normal(1000).astype(np.float32)
    m0 = r.standard_normal(1000).astype(np.float32)
    g = r.standard_normal(1000).astype(np.float32)
    beta, eps = 0.9, 0.7
    theta, m, D = theta0.copy(), m0.copy(), np.zeros(1000, np.float32)
    base = theta0.copy()
    p = base - g
    g_eff = (base - p).astype(np.float64)
    oracle.dn_arrive(theta, m, D, base, p, 0, 1, beta, eps, 0.0)
    b, e = float(np.float32(beta)), float(np.float32(eps))
    np.testing.assert_allclose(m, b * m0.astype(np.float64) + g_eff, rtol=3e-7, atol=1e-7)
    np.testing.assert_allclose(theta, theta0 - e * (b * b * m0.astype(np.float64) + (1 + b) * g_eff),
                               rtol=1e-6, atol=1e-6)


def test_beta_zero_is_plain_outer_sgd():
    r = np.random.default_rng(2)
    P, N, eps = 257, 4, 0.7
    theta = r.standard_normal(P).astype(np.float32)
    m = np.zeros(P, np.float32)
    D = np.zeros(P, np.float32)
    for t in range(9):
        before = theta.copy()
        base = r.standard_normal(P).astype(np.float32)
        p = r.standard_normal(P).astype(np.float32)
        g = base - p
        oracle.dn_arrive(theta, m, D, base, p, t, N, 0.0, eps, 0.0)
        expect = before - np.float32(eps) * (g * np.float32(0.25))
        # On a boundary the momentum term is 0*m_new = +-0 and drops out exactly.
        np.testing.assert_array_equal(theta, expect)


def test_buffer_holds_sum_and_resets_every_Nth():
    r = np.random.default_rng(3)
    P, N = 64, 4
    theta = r.standard_normal(P).astype(np.float32)
    m = np.zeros(P, np.float32)
    D = np.zeros(P, np.float32)
    run = np.zeros(P, np.float64)
    m_prev = m.copy()
    for t in range(12):
        base = r.standard_normal(P).astype(np.float32)
        p = r.standard_normal(P).astype(np.float32)
        run += (base - p).astype(np.float64)
        bnd = oracle.dn_arrive(theta, m, D, base, p, t, N, 0.9, 0.1, 0.0)
        assert bnd == ((t + 1) % N == 0)
        if bnd:
            assert np.all(D == 0)
            np.testing.assert_allclose(m - np.float32(0.9) * m_prev, run / N, rtol=1e-5, atol=1e-6)
            run[:] = 0
            m_prev = m.copy()
        else:
            np.testing.assert_allclose(D, run, rtol=1e-6, atol=1e-6)
            np.testing.assert_array_equal(m, m_prev)      # momentum update delayed


def test_momentum_weights_sum_to_beta_over_a_cycle():
    for N in (1, 2, 3, 4, 8, 16):
        for c in (0.0, 0.5 / N, 1.0 / N):
            beta = 0.9
            cb = oracle.lib().orc_boundary_weight(N, beta, c)
            cn = oracle.lib().orc_between_weight(beta, c)
            assert abs((N - 1) * cn + cb - np.float32(beta)) < 1e-6
    # c = 1/N spreads the momentum evenly: both weights are beta/N
    assert abs(oracle.lib().orc_boundary_weight(4, 0.9, 0.25) - 0.225) < 1e-7
    assert abs(oracle.lib().orc_between_weight(0.9, 0.25) - 0.225) < 1e-7


def unrolled_exact(theta0, gs, N, beta, eps, c):
    """Algorithm 3 unrolled into sums, in exact rationals:
    theta_T = theta_0 - eps/N * sum g_t - eps * sum over steps of (weight_t * momentum seen at t),
    momentum after the b-th boundary = sum_j beta^(b-j) * (cycle-j sum)/N."""
    beta, eps, c = Fraction(beta), Fraction(eps), Fraction(c)
    th = Fraction(theta0)
    cycle_sums, cur = [], Fraction(0)
    m_hist = [Fraction(0)]
    for t, g in enumerate(gs):
        g = Fraction(g)
        cur += g
        th -= eps * g / N
        if (t + 1) % N == 0:
            cycle_sums.append(cur)
            cur = Fraction(0)
            b = len(cycle_sums)
            m_new = sum(beta ** (b - j) * cycle_sums[j - 1] / N for j in range(1, b + 1))
            m_hist.append(m_new)
            th -= eps * (1 - c * N + c) * beta * m_new
        else:
            th -= eps * c * beta * m_hist[-1]
    return th, m_hist[-1], cur


@pytest.mark.parametrize("N,c", [(1, 0.0), (2, 0.0), (3, 0.0), (4, 0.0), (4, 0.125), (3, 0.25), (2, 0.5)])
def test_matches_exact_unrolled_sums(N, c):
    r = np.random.default_rng(10 + N)
    P, T = 16, 13
    beta, eps = 0.875, 0.75           # exactly representable, so the rational weights equal the float ones
    theta0 = r.standard_normal(P).astype(np.float32)
    gs = r.standard_normal((T, P)).astype(np.float32)
    theta, m, D = theta0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)
    for t in range(T):
        base = np.zeros(P, np.float32)
        p = -gs[t]                                  # base - p = g exactly
        oracle.dn_arrive(theta, m, D, base, p, t, N, beta, eps, c)
    for i in range(P):
        th, mm, dd = unrolled_exact(float(theta0[i]), [float(x) for x in gs[:, i]], N, beta, eps, c)
        assert abs(float(theta[i]) - float(th)) <= 4e-6 * max(1.0, abs(float(th)))
        assert abs(float(m[i]) - float(mm)) <= 4e-6 * max(1.0, abs(float(mm)))
        assert abs(float(D[i]) - float(dd)) <= 4e-6 * max(1.0, abs(float(dd)))


def test_one_cycle_equals_synchronous_diloco_with_nesterov():
    """Homogeneous workers, N = k, c = 0: after the k-th arrival the model equals Algorithm 1 with the
    Nesterov outer step of Eq. 4 on the mean pseudo-gradient (the paper's 'reduce to the same' remark)."""
    r = np.random.default_rng(5)
    P, k = 200, 4
    beta, eps = 0.9, 0.7
    theta0 = r.standard_normal(P).astype(np.float32)
    m0 = (0.1 * r.standard_normal(P)).astype(np.float32)
    theta, m, D = theta0.copy(), m0.copy(), np.zeros(P, np.float32)
    deltas = (1e-2 * r.standard_normal((k, P))).astype(np.float32)
    g64 = []
    for w in range(k):
        base = theta0.copy()                         # all seeded with the same model
        p = base - deltas[w]
        g64.append((base - p).astype(np.float64))
        oracle.dn_arrive(theta, m, D, base, p, w, k, beta, eps, 0.0)
    mean = np.mean(g64, axis=0)
    b, e = float(np.float32(beta)), float(np.float32(eps))
    np.testing.assert_allclose(m, b * m0 + mean, rtol=2e-6, atol=1e-7)
    np.testing.assert_allclose(theta, theta0 - e * (b * b * m0 + (1 + b) * mean), rtol=2e-6, atol=2e-6)


def test_current_mode_uses_running_theta():
    theta = np.array([1.0, 2.0], np.float32)
    m = np.zeros(2, np.float32)
    D = np.zeros(2, np.float32)
    p = np.array([0.5, 2.5], np.float32)
    oracle.dn_arrive(theta, m, D, None, p, 0, 4, 0.5, 0.5, 0.0, pg_current=True)
    # g = theta - p = (0.5, -0.5); theta -= 0.5 * g/4
    np.testing.assert_array_equal(D, [0.5, -0.5])
    np.testing.assert_array_equal(theta, [1.0 - 0.0625, 2.0 + 0.0625])
    # a dispatch snapshot, if one is handed in, plays no part in this mode
    theta2, m2, D2 = np.array([1.0, 2.0], np.float32), np.zeros(2, np.float32), np.zeros(2, np.float32)
    oracle.dn_arrive(theta2, m2, D2, np.array([99.0, -99.0], np.float32), p, 0, 4, 0.5, 0.5, 0.0, pg_current=True)
    np.testing.assert_array_equal(D2, [0.5, -0.5])
    np.testing.assert_array_equal(theta2, theta)


def test_brute_force_batch_orders_tiny():
    """Every way of drawing two batches of two from three workers, on P = 8 with a boundary inside
    the second batch: the server's batch call equals the same arrivals applied one at a time with the
    re-dispatch done after the last of them."""
    P, W, N = 8, 3, 3
    r = np.random.default_rng(7)
    theta0 = r.standard_normal(P).astype(np.float32)
    pert = (0.01 * r.standard_normal((W, P))).astype(np.float32)
    n_cases = 0
    for order in itertools.product(range(W), repeat=4):
        b1, b2 = list(order[:2]), list(order[2:])
        if len(set(b1)) < 2 or len(set(b2)) < 2:
            continue                                  # a batch never holds the same worker twice
        batched = oracle.OracleServer(P, W, N, 0.5, 0.5)
        single = oracle.OracleServer(P, W, N, 0.5, 0.5)
        for s in (batched, single):
            s.set_global(theta0)
            for w in range(W):
                s.pull(w)
                s.p[w] -= pert[w]
        infos = batched.arrive(b1) + [None]
        for w in b1:
            batched.p[w] -= pert[w]
        infos = infos[:-1] + batched.arrive(b2)
        for batch in (b1, b2):
            for w in batch:
                single.arrive([w], reseed_after=False)
            for w in batch:
                single.pull(w)
                if batch is b1:
                    single.p[w] -= pert[w]
        np.testing.assert_array_equal(batched.theta, single.theta)
        np.testing.assert_array_equal(batched.m, single.m)
        np.testing.assert_array_equal(batched.Delta, single.Delta)
        assert batched.t == single.t == 4
        assert [i["boundary"] for i in infos] == [False, False, True, False]
        for w in range(W):
            np.testing.assert_array_equal(batched.p[w], single.p[w])
        n_cases += 1
    assert n_cases == 36


def test_server_bookkeeping_ticks_boundaries_staleness():
    srv = oracle.OracleServer(4, 3, 2, 0.5, 0.5)
    srv.set_global(np.ones(4, np.float32))
    for w in range(3):
        srv.pull(w)
    a = srv.arrive([0, 1], reseed_after=True)
    b = srv.arrive([2], reseed_after=True)
    c = srv.arrive([0], reseed_after=False)
    assert [x["tick"] for x in a + b + c] == [0, 1, 2, 3]
    assert [x["boundary"] for x in a + b + c] == [False, True, False, True]
    assert [x["staleness"] for x in a + b + c] == [0, 1, 2, 1]
    assert srv.pull_tick == [2, 2, 3]


def test_pg_norm_and_nonfinite_flag():
    theta = np.zeros(3, np.float32)
    base = np.array([1, 2, 3], np.float32)
    p = np.array([0, 0, 1], np.float32)
    s, bad = oracle.pg_norm2(theta, base, p)
    assert s == 1 + 4 + 4 and bad == 0
    p[1] = np.inf
    s, bad = oracle.pg_norm2(theta, base, p)
    assert bad == 1


def test_pg_norm_in_current_mode_is_taken_against_the_running_theta():
    # the norm of theta - p, whatever the dispatch snapshot holds: (1 - 0.5)^2 + (2 - 2.5)^2 = 0.5
    theta = np.array([1.0, 2.0], np.float32)
    base = np.array([99.0, -99.0], np.float32)
    p = np.array([0.5, 2.5], np.float32)
    s, bad = oracle.pg_norm2(theta, base, p, pg_current=True)
    assert s == 0.5 and bad == 0
    s, bad = oracle.pg_norm2(theta, base, p, pg_current=False)
    assert s == 98.5 ** 2 + 101.5 ** 2 and bad == 0
    # inside a batch the second arrival's pseudo-gradient is against theta after the first:
    # N=4 beta=0.5 eps=0.5, theta=1, workers at 0.5 and 0.75.  First: g = 0.5, theta = 1 - 0.5*0.5/4 = 0.9375.
    # Second: g = 0.9375 - 0.75 = 0.1875 (against the dispatch model it would be 0.25).
    srv = oracle.OracleServer(3, 2, 4, 0.5, 0.5, pg_current=True)
    srv.set_global(np.ones(3, np.float32))
    srv.pull(0); srv.pull(1)
    srv.p[0][:] = 0.5
    srv.p[1][:] = 0.75
    info = srv.arrive([0, 1], norm=True)
    assert info[0]["gnorm2"] == 3 * 0.25 and info[1]["gnorm2"] == 3 * 0.1875 ** 2
    np.testing.assert_array_equal(srv.Delta, np.float32(0.6875))
    srv.p[0][1] = np.nan                                   # re-dispatched at theta; one poisoned entry
    info = srv.arrive([0], norm=True)
    assert info[0]["nonfinite"] == 1
