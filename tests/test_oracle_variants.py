"""Pins for the oracle's Section-4 variants of the server step: staleness weighting (Poly, PolyThres),
delay compensation on pseudo-gradients, and the buffered (FedBuff-style) outer step."""
import os

import numpy as np

import oracle
from conftest import ROOT


def rows(kind):
    out = []
    for line in open(os.path.join(ROOT, "tests", "golden", "variants_hand.txt")):
        f = line.split()
        if f and f[0] == kind:
            out.append([float(x) for x in f[1:]])
    return out


def test_buffered_hand_trace():
    theta, m, D = np.ones(3, np.float32), np.zeros(3, np.float32), np.zeros(3, np.float32)
    for t, (g, th, mm, dd, bnd) in enumerate(rows("buffered")):
        base = theta.copy()
        p = base - np.float32(g)
        b = oracle.dn_arrive(theta, m, D, base, p, t, 2, 0.5, 0.5, 0.0, buffered=True)
        assert b == bool(bnd)
        assert np.all(theta == np.float32(th)) and np.all(m == np.float32(mm)) and np.all(D == np.float32(dd))


def test_buffered_with_N1_is_plain_nesterov_and_matches_dn_at_cycle_ends():
    r = np.random.default_rng(0)
    P = 64
    gs = r.standard_normal((12, P)).astype(np.float32)
    th0 = r.standard_normal(P).astype(np.float32)
    # N = 1: both modes are Eq. 4 on every arrival
    a = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    b = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    for t in range(12):
        base = np.zeros(P, np.float32)
        oracle.dn_arrive(*a, base, -gs[t], t, 1, 0.9, 0.7, 0.0, buffered=True)
        oracle.dn_arrive(*b, base, -gs[t], t, 1, 0.9, 0.7, 0.0, buffered=False)
        np.testing.assert_allclose(a[0], b[0], rtol=3e-6, atol=3e-6)
        np.testing.assert_allclose(a[1], b[1], rtol=3e-6, atol=3e-6)
    # N = 4, pseudo-gradients independent of theta: same model after every full cycle, theta frozen in between
    a = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    b = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    for t in range(12):
        base = np.zeros(P, np.float32)
        before = a[0].copy()
        bnd = oracle.dn_arrive(*a, base, -gs[t], t, 4, 0.9, 0.7, 0.0, buffered=True)
        oracle.dn_arrive(*b, base, -gs[t], t, 4, 0.9, 0.7, 0.0, buffered=False)
        if bnd:
            np.testing.assert_allclose(a[0], b[0], rtol=1e-5, atol=1e-5)
            np.testing.assert_allclose(a[1], b[1], rtol=1e-5, atol=1e-5)
        else:
            assert np.array_equal(a[0], before)


def test_sgd_momentum_outer_step_hand_trace():
    theta, m, D = np.ones(3, np.float32), np.zeros(3, np.float32), np.zeros(3, np.float32)
    for t, (g, th, mm, dd, bnd) in enumerate(rows("sgdm")):
        base = theta.copy()
        p = base - np.float32(g)
        b = oracle.dn_arrive(theta, m, D, base, p, t, 2, 0.5, 0.5, 0.0, buffered=oracle.OUTER_SGDM)
        assert b == bool(bnd)
        assert np.all(theta == np.float32(th)) and np.all(m == np.float32(mm)) and np.all(D == np.float32(dd))


def test_sgd_momentum_outer_step_properties():
    from fractions import Fraction as F
    r = np.random.default_rng(5)
    P = 48
    gs = r.standard_normal((10, P)).astype(np.float32)
    th0 = r.standard_normal(P).astype(np.float32)
    beta, eps = np.float32(0.9), np.float32(0.7)
    # (i) N = 1: the parameter change of every step is eps times the new momentum (beta m + g is both),
    #     and the momentum recursion is the one of Eq. 4
    st = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    for t in range(10):
        before, m_old = st[0].copy(), st[1].copy()
        assert oracle.dn_arrive(*st, np.zeros(P, np.float32), -gs[t], t, 1, beta, eps, 0.0, buffered=oracle.OUTER_SGDM)
        assert np.array_equal(st[1], (beta * m_old) + gs[t])
        assert np.array_equal(st[0], before - (eps * st[1]))
        assert not st[2].any()
    # (ii) against Eq. 4 from the same state: theta_nesterov - theta_sgdm = -eps ((beta^2 - beta) m + beta g)
    a = [th0.copy(), gs[0].copy(), np.zeros(P, np.float32)]
    b = [th0.copy(), gs[0].copy(), np.zeros(P, np.float32)]
    oracle.dn_arrive(*a, np.zeros(P, np.float32), -gs[1], 0, 1, beta, eps, 0.0, buffered=oracle.OUTER_BUFFERED)
    oracle.dn_arrive(*b, np.zeros(P, np.float32), -gs[1], 0, 1, beta, eps, 0.0, buffered=oracle.OUTER_SGDM)
    b64, e64 = float(beta), float(eps)
    want = -e64 * ((b64 * b64 - b64) * gs[0].astype(np.float64) + b64 * gs[1].astype(np.float64))
    np.testing.assert_allclose(a[0].astype(np.float64) - b[0].astype(np.float64), want, rtol=0, atol=2e-6)
    assert np.array_equal(a[1], b[1])                                  # same momentum recursion
    # (iii) beta = 0: plain outer SGD on the buffer mean, theta' = theta - eps * Delta/N, m' = Delta/N
    st = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    ref = th0.copy()
    acc = np.zeros(P, np.float32)
    for t in range(8):
        bnd = oracle.dn_arrive(*st, np.zeros(P, np.float32), -gs[t], t, 4, 0.0, eps, 0.0, buffered=oracle.OUTER_SGDM)
        acc = acc + gs[t]
        if bnd:
            mean = acc * np.float32(0.25)
            ref = ref - (eps * mean)
            assert np.array_equal(st[1], mean)
            acc[:] = 0
        assert np.array_equal(st[0], ref)
    # (iv) constant g, N = 1, k steps, exact rationals: m_k = g (1 - beta^k)/(1 - beta), theta_k = theta_0 - eps sum_j m_j
    g, k = np.float32(0.375), 6
    st = [np.ones(2, np.float32), np.zeros(2, np.float32), np.zeros(2, np.float32)]
    for t in range(k):
        oracle.dn_arrive(*st, np.zeros(2, np.float32), np.full(2, -g, np.float32), t, 1, beta, eps, 0.0, buffered=oracle.OUTER_SGDM)
    bq, eq, gq = F(float(beta)), F(float(eps)), F(float(g))
    mq = [gq * (1 - bq ** j) / (1 - bq) for j in range(1, k + 1)]
    assert abs(float(st[1][0]) - float(mq[-1])) < 1e-6
    assert abs(float(st[0][0]) - float(1 - eq * sum(mq))) < 2e-6
    # (v) theta frozen between boundaries, as in the buffered Nesterov form
    st = [th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)]
    for t in range(3):
        assert not oracle.dn_arrive(*st, np.zeros(P, np.float32), -gs[t], t, 4, beta, eps, 0.0, buffered=oracle.OUTER_SGDM)
        assert np.array_equal(st[0], th0)


def test_delay_compensation_hand_case_and_zero_drift():
    (lam, base, p, th_now, d_exp, th_exp), = rows("dc")
    theta, m, D = np.full(2, th_now, np.float32), np.zeros(2, np.float32), np.zeros(2, np.float32)
    oracle.dn_arrive(theta, m, D, np.full(2, base, np.float32), np.full(2, p, np.float32), 0, 4, 0.9, 0.5, 0.0, dc_lambda=lam)
    assert np.all(D == np.float32(d_exp)) and np.all(theta == np.float32(th_exp))
    # no drift (theta has not moved since dispatch): compensation vanishes exactly
    r = np.random.default_rng(1)
    th = r.standard_normal(100).astype(np.float32)
    p = r.standard_normal(100).astype(np.float32)
    a = [th.copy(), np.zeros(100, np.float32), np.zeros(100, np.float32)]
    b = [th.copy(), np.zeros(100, np.float32), np.zeros(100, np.float32)]
    oracle.dn_arrive(*a, th.copy(), p, 0, 4, 0.9, 0.7, 0.0, dc_lambda=3.0)
    oracle.dn_arrive(*b, th.copy(), p, 0, 4, 0.9, 0.7, 0.0, dc_lambda=0.0)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_weighted_arrival_hand_case_and_homogeneity():
    (w, base, p, th, d_exp, th_exp), = rows("weight")
    theta, m, D = np.full(2, th, np.float32), np.zeros(2, np.float32), np.zeros(2, np.float32)
    oracle.dn_arrive(theta, m, D, np.full(2, base, np.float32), np.full(2, p, np.float32), 0, 4, 0.9, 0.5, 0.0, weight=w)
    assert np.all(D == np.float32(d_exp)) and np.all(theta == np.float32(th_exp))
    # a power-of-two weight equals feeding the scaled pseudo-gradient (exact)
    r = np.random.default_rng(2)
    g = r.standard_normal(50).astype(np.float32)
    a = [np.ones(50, np.float32), np.zeros(50, np.float32), np.zeros(50, np.float32)]
    b = [np.ones(50, np.float32), np.zeros(50, np.float32), np.zeros(50, np.float32)]
    for t in range(5):
        oracle.dn_arrive(*a, np.zeros(50, np.float32), -g, t, 2, 0.5, 0.5, 0.0, weight=0.25)
        oracle.dn_arrive(*b, np.zeros(50, np.float32), -(g * np.float32(0.25)), t, 2, 0.5, 0.5, 0.0)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))


def test_delay_compensation_comes_before_the_staleness_weight():
    (lam, w, base, p, th_now, d_exp, th_exp), = rows("dcweight")
    theta, m, D = np.full(2, th_now, np.float32), np.zeros(2, np.float32), np.zeros(2, np.float32)
    oracle.dn_arrive(theta, m, D, np.full(2, base, np.float32), np.full(2, p, np.float32), 0, 4, 0.9, 0.5, 0.0,
                     weight=w, dc_lambda=lam)
    assert np.all(D == np.float32(d_exp)) and np.all(theta == np.float32(th_exp))
    # weighting the compensated pseudo-gradient by a power of two == feeding that scaled vector unweighted (exact)
    r = np.random.default_rng(3)
    th = r.standard_normal(40).astype(np.float32)
    b = (th + 0.1 * r.standard_normal(40)).astype(np.float32)
    q = (b - 0.3 * r.standard_normal(40)).astype(np.float32)
    g = b - q
    comp = g + ((np.float32(1.5) * (g * g)) * (th - b))
    a1 = [th.copy(), np.zeros(40, np.float32), np.zeros(40, np.float32)]
    a2 = [th.copy(), np.zeros(40, np.float32), np.zeros(40, np.float32)]
    oracle.dn_arrive(*a1, b, q, 0, 4, 0.9, 0.7, 0.0, weight=0.25, dc_lambda=1.5)
    oracle.dn_arrive(*a2, np.zeros(40, np.float32), -(comp * np.float32(0.25)), 0, 4, 0.9, 0.7, 0.0)
    assert all(np.array_equal(x, y) for x, y in zip(a1, a2))


def test_poly_weights_and_threshold_bookkeeping():
    assert [oracle.poly_weight(s) for s in (0, 3, 15)] == [1.0, 0.5, 0.25]
    assert abs(oracle.poly_weight(8) - 1 / 3) < 1e-7
    srv = oracle.OracleServer(4, 3, 4, 0.5, 0.5)
    srv.set_global(np.ones(4, np.float32))
    for w in range(3):
        srv.pull(w)
        srv.p[w] -= np.float32(0.5)
    srv.arrive([0], poly=True, stale_threshold=1)                     # staleness 0: weight 1
    assert np.all(srv.Delta == 0.5) and srv.t == 1
    srv.p[0] -= np.float32(0.5)
    srv.arrive([0], poly=True, stale_threshold=1)                     # staleness 0 again (re-dispatched at t=1)
    assert srv.t == 2
    before = (srv.theta.copy(), srv.Delta.copy())
    info = srv.arrive([1, 2], poly=True, stale_threshold=1)           # both are 2 ticks stale: discarded
    assert [i["dropped"] for i in info] == [True, True] and srv.t == 2
    assert np.array_equal(srv.theta, before[0]) and np.array_equal(srv.Delta, before[1])
    assert srv.pull_tick == [2, 2, 2]                                  # ... but re-dispatched
    srv.p[1] -= np.float32(0.5)
    srv.t += 0
    srv2 = oracle.OracleServer(4, 2, 8, 0.5, 0.5)
    srv2.set_global(np.ones(4, np.float32))
    srv2.pull(0); srv2.pull(1)
    srv2.p[0] -= np.float32(1.0); srv2.p[1] -= np.float32(1.0)
    for _ in range(3):
        srv2.arrive([0], poly=True)
        srv2.p[0] -= np.float32(1.0)
    d_before = srv2.Delta.copy()
    info = srv2.arrive([1], poly=True)                                 # staleness 3 -> weight 0.5
    assert info[0]["staleness"] == 3 and np.all(srv2.Delta - d_before == 0.5)
