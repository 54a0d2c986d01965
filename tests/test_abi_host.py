"""CPU-only checks of the C-ABI library: it loads, exports every function the header declares, and
its host logic (layout, Eq. 6, Eq. 3, Algorithm 2/5 scheduler, argument validation) agrees with the
oracle.  No compute call is made, so no GPU is needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    text = open(os.path.join(ROOT, "include", "alsgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return set(re.findall(r"\b(alsgd_[a-z0-9_]+)\s*\(", text))


def test_library_exports_every_declared_function():
    L = B.lib()
    declared = header_functions()
    assert declared, "no declarations parsed"
    assert declared == set(B.SIGNATURES), (declared ^ set(B.SIGNATURES))
    for name in declared:
        assert hasattr(L, name), name


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(B.TensorDesc) == 16
    assert C.sizeof(B.Config) == 4 * 4 + 7 * 4 + 4 + 3 * 8
    assert C.sizeof(B.ArrivalInfo) == 40
    assert C.sizeof(B.Ptrs) == 40
    assert C.sizeof(B.WorkerPtrs) == 40
    assert C.sizeof(B.LrSched) == 32


def test_strerror_texts():
    L = B.lib()
    assert L.alsgd_strerror(0) == b"ok"
    for s in range(-7, 0):
        assert L.alsgd_strerror(s) not in (b"ok", b"unknown status")
    assert L.alsgd_strerror(-99) == b"unknown status"


@pytest.mark.parametrize("align", [1, 4, 8, 128, 1000])
def test_layout_offsets_match_oracle(align):
    for tensors in (synth.ragged_tensors(), synth.layout_23m(), synth.flat_tensors(1 << 20)):
        P, offs = B.alsgd_layout_size(tensors, align)
        o_offs, o_P = oracle.layout_offsets([t.numel for t in tensors], align)
        assert (P, offs) == (o_P, o_offs)
        assert P % align == 0


def test_layout_sizes_of_the_transformer_configs():
    assert B.alsgd_layout_size(synth.layout_23m())[0] == 22_914_816
    assert B.alsgd_layout_size(synth.layout_110m())[0] == 109_549_056


def test_layout_rejects_bad_input():
    L = B.lib()
    P = C.c_uint64()
    tab = B.tensor_table([(4, True)])
    assert L.alsgd_layout_size(tab, 0, 4, C.byref(P), None) == B.E_ARG
    assert L.alsgd_layout_size(tab, 1, 0, C.byref(P), None) == B.E_ARG
    assert L.alsgd_layout_size(None, 1, 4, C.byref(P), None) == B.E_ARG
    assert L.alsgd_layout_size(tab, 1, 4, None, None) == B.E_ARG
    zero = B.tensor_table([(4, True)])
    zero[0].numel = 0
    assert L.alsgd_layout_size(zero, 1, 4, C.byref(P), None) == B.E_ARG
    huge = B.tensor_table([(4, True)])
    huge[0].numel = (1 << 64) - 1
    assert L.alsgd_layout_size(huge, 1, 4, C.byref(P), None) == B.E_ARG


def _cfg(**kw):
    cfg = B.Config()
    cfg.n_workers, cfg.N, cfg.pg_base, cfg.flags = 4, 4, B.PG_DISPATCH, B.CFG_REPLICA_BF16
    cfg.beta, cfg.outer_lr, cfg.c = 0.9, 0.7, 0.0
    cfg.adam_b1, cfg.adam_b2, cfg.adam_eps, cfg.adam_wd = 0.9, 0.95, 1e-8, 0.1
    for k, v in kw.items():
        setattr(cfg, k, v)
    return cfg


def test_arena_bytes_accounts_for_every_buffer():
    L = B.lib()
    tab = B.tensor_table(synth.layout_23m())
    P = 22_914_816
    n = C.c_uint64()
    assert L.alsgd_arena_bytes(tab, len(tab), 128, C.byref(_cfg()), C.byref(n)) == 0
    body = 12 * P + 4 * 18 * P          # theta, m, Delta + 4 x (p, snapshot, adam m, adam v, bf16)
    slack = P // 8 + 64 * 1024          # diagnostics partial sums (one double per 512 elements per arrival slot) + tables
    assert body <= n.value <= body + slack
    m = C.c_uint64()
    assert L.alsgd_arena_bytes(tab, len(tab), 128, C.byref(_cfg(pg_base=B.PG_CURRENT, flags=0)), C.byref(m)) == 0
    assert 12 * P + 4 * 12 * P <= m.value <= 12 * P + 4 * 12 * P + slack
    g = C.c_uint64()
    assert L.alsgd_arena_bytes(tab, len(tab), 128, C.byref(_cfg(flags=B.CFG_REPLICA_BF16 | B.CFG_GRAD_STAGING)), C.byref(g)) == 0
    assert g.value - n.value == 4 * P


@pytest.mark.parametrize("bad", [dict(n_workers=0), dict(N=0), dict(beta=1.0), dict(beta=-0.1), dict(c=0.3),
                                 dict(c=-0.01), dict(pg_base=7), dict(flags=64), dict(adam_b1=1.0),
                                 dict(adam_eps=-1.0), dict(adam_wd=-1.0), dict(outer_lr=float("nan"))])
def test_config_domains_are_enforced_before_any_device_work(bad):
    L = B.lib()
    tab = B.tensor_table([(1024, True)])
    n = C.c_uint64()
    assert L.alsgd_arena_bytes(tab, 1, 128, C.byref(_cfg(**bad)), C.byref(n)) == B.E_ARG
    h = C.c_void_p()
    cfg = _cfg(**bad)
    cfg.arena, cfg.arena_bytes = 256, 1 << 30
    assert L.alsgd_init(C.byref(h), tab, 1, 128, C.byref(cfg)) == B.E_ARG
    assert not h


def test_init_rejects_null_misaligned_or_small_arena():
    L = B.lib()
    tab = B.tensor_table([(1024, True)])
    h = C.c_void_p()
    cfg = _cfg()
    assert L.alsgd_init(C.byref(h), tab, 1, 128, C.byref(cfg)) == B.E_ARG          # arena NULL
    cfg.arena, cfg.arena_bytes = 256 + 8, 1 << 30
    assert L.alsgd_init(C.byref(h), tab, 1, 128, C.byref(cfg)) == B.E_ARG          # not 256-aligned
    cfg.arena, cfg.arena_bytes = 256, 1024
    assert L.alsgd_init(C.byref(h), tab, 1, 128, C.byref(cfg)) == B.E_NOMEM
    # c = 1/N is inside the domain
    n = C.c_uint64()
    assert L.alsgd_arena_bytes(tab, 1, 128, C.byref(_cfg(c=0.25)), C.byref(n)) == 0
    assert L.alsgd_arena_bytes(tab, 1, 128, C.byref(_cfg(beta=0.0)), C.byref(n)) == 0


def test_null_context_is_an_argument_error():
    L = B.lib()
    assert L.alsgd_pull(None, 0) == B.E_ARG
    assert L.alsgd_arrive(None, None, 0, 0, None) == B.E_ARG
    assert L.alsgd_sync(None) == B.E_ARG
    assert L.alsgd_counters(None, None, None) == B.E_ARG
    assert L.alsgd_destroy(None) == 0


# ---- Eq. 6, Eq. 3 -------------------------------------------------------------------------------------

def test_dylu_matches_oracle():
    assert B.alsgd_dylu_steps([1, 1.5, 2, 3], 50) == [16, 25, 33, 50]
    r = np.random.default_rng(0)
    for _ in range(200):
        n = int(r.integers(1, 17))
        sp = list(np.exp(r.normal(0, 1.5, n)))
        H = int(r.integers(1, 200))
        assert B.alsgd_dylu_steps(sp, H) == oracle.dylu(sp, H)
    L = B.lib()
    out = (C.c_uint32 * 2)()
    assert L.alsgd_dylu_steps((C.c_double * 2)(1.0, 0.0), 2, 50, out) == B.E_ARG
    assert L.alsgd_dylu_steps((C.c_double * 2)(1.0, 2.0), 2, 0, out) == B.E_ARG


def test_shard_probs_match_oracle():
    r = np.random.default_rng(5)
    for _ in range(200):
        n = int(r.integers(1, 12))
        sizes = list(r.uniform(1, 100, n))
        learned = list(r.uniform(0, 50, n)) if r.integers(0, 4) else [0.0] * n
        assert B.alsgd_shard_probs(sizes, learned) == oracle.shard_probs(sizes, learned)
    assert B.alsgd_shard_probs([1, 3], [5, 15]) == [0.25, 0.75]
    L = B.lib()
    out = (C.c_double * 2)()
    assert L.alsgd_shard_probs((C.c_double * 2)(1.0, 0.0), (C.c_double * 2)(0.0, 0.0), 2, out) == B.E_ARG
    assert L.alsgd_shard_probs((C.c_double * 2)(1.0, 1.0), (C.c_double * 2)(-1.0, 0.0), 2, out) == B.E_ARG


def test_lr_schedule_matches_oracle():
    for (emax, emin, tw, T) in [(0.1, 1e-6, 1000, 88000), (1e-3, 0.0, 0, 100), (0.5, 0.01, 10, 10), (0.5, 0.01, 50, 20)]:
        for t in list(range(0, 130)) + [999, 1000, 1001, 44500, 87999, 88000, 88001, 10**7]:
            assert B.alsgd_lr_at(emax, emin, tw, T, t) == oracle.lr_at(emax, emin, tw, T, t)


# ---- scheduler ---------------------------------------------------------------------------------------------

def run_lib_schedule(durations, local_updates, tau_grace, t_max, max_arrivals):
    W, R = durations.shape
    s = B.Scheduler(W, tau_grace, t_max if t_max < 10**17 else 0)
    rounds = [0] * W
    for w in range(W):
        s.dispatch(w, durations[w, 0], local_updates[w])
    workers, times, batches = [], [], []
    b = 0
    while len(workers) < max_arrivals:
        ids, ts, restart = s.next_batch()
        if not ids:
            break
        for w, t in zip(ids, ts):
            if len(workers) < max_arrivals:
                workers.append(w); times.append(t); batches.append(b)
        b += 1
        stop = False
        for w in ids:
            rounds[w] += 1
            if rounds[w] >= R:
                stop = True
                break
            s.dispatch(w, durations[w, rounds[w]], local_updates[w])
        if stop:
            break
    return workers, times, batches


@pytest.mark.parametrize("tau_grace", [0.0, 0.3, 2.0, 100.0])
def test_scheduler_matches_oracle_on_random_timelines(tau_grace):
    r = np.random.default_rng(int(tau_grace * 10))
    for trial in range(30):
        W = int(r.integers(1, 9))
        R = 40
        speeds = np.exp(r.normal(0, 0.6, W))
        steps = oracle.dylu(list(speeds), 50)
        dur = synth.job_durations(speeds, steps, R, seed=trial)
        if trial % 3 == 0:
            dur = np.round(dur, 0) + 1.0            # provoke ties
        n = 60
        t_max = 10**18 if trial % 2 else 900
        ow, ot, ob = oracle.schedule(dur, steps, tau_grace, t_max, n)
        lw, lt, lb = run_lib_schedule(dur, steps, tau_grace, t_max, n)
        m = min(len(ow), len(lw))
        assert m > 0
        # both stop for the same reason except when the supplied durations run out, which the two
        # drivers notice at slightly different moments; compare the common prefix and its length
        assert abs(len(ow) - len(lw)) <= W
        assert ow[:m] == lw[:m]
        assert ot[:m] == lt[:m]
        assert ob[:m] == lb[:m]


def test_scheduler_homogeneous_workers_are_synchronous():
    dur = np.full((4, 6), 7.0)
    w, t, b = run_lib_schedule(dur, [50] * 4, 0.0, 10**18, 16)
    assert w == [0, 1, 2, 3] * 4 and b == [0] * 4 + [1] * 4 + [2] * 4 + [3] * 4


def test_scheduler_state_errors_and_missing_worker():
    s = B.Scheduler(3, 1.0)
    L = B.lib()
    ids = (C.c_uint32 * 3)()
    k = C.c_uint32()
    assert L.alsgd_sched_next_batch(s._h, ids, None, 3, C.byref(k), None) == B.E_STATE   # nothing in flight
    s.dispatch(0, 1.0, 5)
    assert L.alsgd_sched_dispatch(s._h, 0, 1.0, 5) == B.E_STATE                           # already running
    assert L.alsgd_sched_dispatch(s._h, 3, 1.0, 5) == B.E_RANGE
    assert L.alsgd_sched_dispatch(s._h, 1, 0.0, 5) == B.E_ARG
    s.dispatch(1, 1.5, 5)
    # worker 2 never starts (a failed device): the others keep being scheduled
    assert L.alsgd_sched_next_batch(s._h, ids, None, 1, C.byref(k), None) == B.E_NOMEM    # cap too small
    got, times, restart = s.next_batch()
    assert got == [0, 1] and times == [1.0, 1.5] and restart == 2.0
    s.dispatch(0, 1.0, 5)
    got, times, restart = s.next_batch()
    assert got == [0] and times == [3.0]
    assert s.local_updates() == 15


def test_scheduler_t_max_cuts_a_window():
    s = B.Scheduler(3, 10.0, t_max=25)
    for w in range(3):
        s.dispatch(w, 1.0 + w, 10)
    got, _, _ = s.next_batch()
    assert got == [0, 1, 2][:3] and s.local_updates() == 30
    for w in got:
        s.dispatch(w, 1.0, 10)
    assert s.next_batch()[0] == []


def test_benchmark_reference_arm_needs_only_the_oracle():
    """bench.py --impl reference takes its DyLU steps and arrival order from the oracle alone, and they are the
    ones the library's host scheduler gives the GPU arm."""
    import subprocess
    import sys
    code = ("import sys, json; sys.path.insert(0, %r); import bench; "
            "print(json.dumps([bench.oracle_schedule(40), [m for m in sys.modules if m.endswith('binding')]]))" % ROOT)
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, check=True).stdout
    import json
    (steps, order), loaded = json.loads(out.strip().splitlines()[-1])
    assert loaded == []
    import bench
    lib_steps, lib_order = bench.build_schedule(40)
    assert steps == lib_steps == [16, 25, 33, 50] and order == lib_order


def test_scheduler_checkpoint_continues_the_timeline():
    """Algorithm 2 for 20 windows; export after 9; a fresh scheduler that imports the image produces the
    identical remaining windows (ids, times, restart time, t_local)."""
    W, speeds = 5, [1.0, 1.3, 1.7, 2.2, 3.0]
    steps = B.alsgd_dylu_steps(speeds, 40)
    dur = synth.job_durations(speeds, steps, 64, synth.SEED + 21)

    def drive(s, rounds, n_windows, log):
        for _ in range(n_windows):
            ids, times, restart = s.next_batch()
            log.append((ids, times, restart, s.local_updates()))
            for w in ids:
                rounds[w] += 1
                s.dispatch(w, dur[w, rounds[w]], steps[w])

    full, rounds = [], [0] * W
    a = B.Scheduler(W, 0.35)
    for w in range(W):
        a.dispatch(w, dur[w, 0], steps[w])
    drive(a, rounds, 9, full)
    image = a.export_state()
    rounds_at_9 = list(rounds)
    drive(a, rounds, 11, full)
    assert any(len(ids) > 1 for ids, *_ in full) and any(len(ids) == 1 for ids, *_ in full)

    b = B.Scheduler(W, 0.0)                      # other grace period: the image brings its own
    b.import_state(image)
    resumed = []
    drive(b, rounds_at_9, 11, resumed)
    assert resumed == full[9:]

    L = B.lib()
    c = B.Scheduler(W + 1, 0.35)
    assert L.alsgd_sched_import(c._h, image, len(image)) == B.E_ARG            # other worker count
    assert L.alsgd_sched_import(b._h, image[:20], 20) == B.E_ARG               # truncated
    assert L.alsgd_sched_import(b._h, b"x" * len(image), len(image)) == B.E_ARG
    small = C.create_string_buffer(8)
    assert L.alsgd_sched_export(b._h, small, 8) == B.E_NOMEM
    # a mid-window export: one job consumed, others in flight
    d = B.Scheduler(2, 10.0)
    d.dispatch(0, 1.0, 3)
    img0 = d.export_state()
    d.dispatch(1, 2.0, 4)
    e = B.Scheduler(2, 0.0)
    e.import_state(img0)
    assert L.alsgd_sched_dispatch(e._h, 0, 1.0, 3) == B.E_STATE                # worker 0's job is in flight in the image
    e.dispatch(1, 2.0, 4)
    assert e.next_batch() == d.next_batch()
