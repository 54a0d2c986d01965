"""Benchmark of the asynchronous Local-SGD server path on B200.

One step = one arrival of the seeded heterogeneous schedule on the ~110M-parameter layout: the host
scheduler (Algorithm 2/5) names the arriving worker, that worker runs its DyLU number of inner AdamW
steps (Eq. 6; 16/25/33/50 for speeds 1:1.5:2:3, H = 50), then its pseudo-gradient goes through the
Delayed-Nesterov arrival with the fused re-seed.  Each kernel launch streams the whole flat vector
(3.3-3.7 GB per launch, far larger than L2), so no L2 flush is needed between iterations.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line on rank 0.  At N = 1 the line also carries the reported figures of the other configurations
(`ksweep`: arrival batches k = 1, 2, 4, 8 with 8 resident workers; `layouts`: per-kernel throughput on the 23M /
60M / 110M / 150M layouts), measured after the timed region, and the oracle timed on one and on all host cores.
Further modes: --ksweep, --layouts, --cpu-kernels, --shape-sweep (launch-shape benchmark), --profile-case
(small fixed cases for profiler captures).
"""
import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "params_per_s_dn_arrival_plus_adamw"
UNIT = "params/s"
WORKLOAD = "decoder-110M(12L,d768,ff3072,V32000) W=4 N=4 beta=0.9 outer_lr=0.7 c=0 bf16-replicas"
SPEEDS = [1.0, 1.5, 2.0, 3.0]
H = 50
ADAMW_BYTES = 30          # g,p,m,v read (16) + p,m,v write (12) + bf16 replica write (2)
ARRIVE_RESEED_BYTES = {   # theta, Delta, snapshot, p read / theta, Delta write (+m on a boundary), + new snapshot 4 and bf16 2
    "first": 20 + 6,      # Delta known zero: not read
    "middle": 24 + 6,     # (the re-seeded parameters are not stored twice: until the worker's next AdamW step
    "boundary": 28 + 6,   #  writes them they are read from the snapshot)  + m read and write; Delta zero store elided
}
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per parameter from the committed ncu captures
# (profiles/), valid only for the kernel source they were taken from.
NCU_TRAFFIC = {
    "src_sha256": "a38ecdfa04e6e4fcc6f8673ea58393910425528c24765c0bd2fe7ff66de9691a",
    "adamw_bytes_per_param": 28.90,     # ncu capture at P = 50.3M elements (profiles/adamw_kernel_flat48M.md), scaled by P
    "arrive_bytes_per_param": 28.90,    # same capture, K = 1, average over one Delayed-Nesterov cycle
}


def kernel_source_hash():
    h = hashlib.sha256()
    for name in ("alsgd_kernels_impl.cuh", "alsgd_kernels.cu"):
        with open(os.path.join(ROOT, "paper_2401_09135_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs (read-only)."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.rows:
            if not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            f = [x.strip() for x in line.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except Exception:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def build_schedule(n_arrivals):
    """Arrival order from the library's host scheduler, DyLU steps from Eq. 6."""
    from paper_2401_09135_b200 import binding as B, synth
    steps = B.alsgd_dylu_steps(SPEEDS, H)
    dur = synth.job_durations(SPEEDS, steps, n_arrivals + 2, synth.SEED + 7)
    s = B.Scheduler(len(SPEEDS), 0.0)
    rounds = [0] * len(SPEEDS)
    for w in range(len(SPEEDS)):
        s.dispatch(w, dur[w, 0], steps[w])
    order = []
    while len(order) < n_arrivals:
        ids, _, _ = s.next_batch()
        for w in ids:
            order.append(w)
            rounds[w] += 1
            s.dispatch(w, dur[w, rounds[w]], steps[w])
    return steps, order[:n_arrivals]


def oracle_schedule(n_arrivals):
    """The same schedule from the oracle alone (Eq. 6 and Algorithms 2 + 5 as the oracle states them), so that
    the reference arm needs nothing of the CUDA library."""
    import oracle
    from paper_2401_09135_b200 import synth
    steps = oracle.dylu(SPEEDS, H)
    dur = synth.job_durations(SPEEDS, steps, n_arrivals + 2, synth.SEED + 7)
    workers, _, _ = oracle.schedule(dur, steps, 0.0, 10 ** 18, n_arrivals)
    return steps, workers


# ----------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ----------------------------------------------------------------------------------------------------
def oracle_step(srv, w, n_inner, grads, life, lr=1e-3):
    for _ in range(n_inner):
        life[w] += 1
        srv.inner_adamw(w, grads[life[w] % len(grads)], life[w], lr)
    srv.arrive([w], reseed_after=True)


def run_oracle(n_elems, order, steps, warmup, timed):
    """Times `timed` steps of the same path on the first n_elems elements of the layout."""
    import numpy as np
    import oracle
    from paper_2401_09135_b200 import synth
    tensors = synth.layout_110m()
    offs, P = oracle.layout_offsets([t.numel for t in tensors], 128)
    mask = oracle.decay_mask([t.numel for t in tensors], [t.decay for t in tensors], offs, P)[:n_elems].copy()
    srv = oracle.OracleServer(n_elems, len(SPEEDS), 4, 0.9, 0.7, decay=mask)
    srv.set_global(synth.normal_vec(n_elems, 0.02, synth.SEED, synth.STREAM_THETA0))
    grads = [synth.normal_vec(n_elems, 1e-2, synth.SEED, synth.STREAM_GRAD, sub=i) for i in range(2)]
    for w in range(len(SPEEDS)):
        srv.pull(w)
    life = [0] * len(SPEEDS)
    for w in order[:warmup]:
        oracle_step(srv, w, steps[w], grads, life)
    t0 = time.perf_counter()
    passes = 0
    for w in order[warmup:warmup + timed]:
        oracle_step(srv, w, steps[w], grads, life)
        passes += steps[w] + 1
    dt = time.perf_counter() - t0
    return n_elems * passes / dt, dt, passes


def run_oracle_all_cores(n_elems, w, n_inner, threads):
    """One step of the same path with the oracle's scalar loops range-split over `threads` host threads (exact:
    the path is elementwise; the C functions release the interpreter lock)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    import oracle
    from paper_2401_09135_b200 import synth
    tensors = synth.layout_110m()
    offs, P = oracle.layout_offsets([t.numel for t in tensors], 128)
    mask = oracle.decay_mask([t.numel for t in tensors], [t.decay for t in tensors], offs, P)[:n_elems].copy()
    z = lambda: np.zeros(n_elems, np.float32)
    theta = synth.normal_vec(n_elems, 0.02, synth.SEED, synth.STREAM_THETA0)
    m, D, p, base, am, av, rep = z(), z(), theta.copy(), theta.copy(), z(), z(), np.zeros(n_elems, np.uint16)
    g = synth.normal_vec(n_elems, 1e-2, synth.SEED, synth.STREAM_GRAD)
    cuts = [n_elems * i // threads for i in range(threads + 1)]
    with ThreadPoolExecutor(threads) as ex:
        def every(fn):
            list(ex.map(lambda i: fn(cuts[i], cuts[i + 1]), range(threads)))
        t0 = time.perf_counter()
        for s in range(1, n_inner + 1):
            every(lambda lo, hi: oracle.adamw(p, am, av, g, rep, mask, s, 1e-3, 0.9, 0.95, 1e-8, 0.1, lo=lo, hi=hi))
        every(lambda lo, hi: oracle.dn_arrive(theta, m, D, base, p, 0, 4, 0.9, 0.7, lo=lo, hi=hi))
        every(lambda lo, hi: oracle.reseed(theta, p, base, rep, lo=lo, hi=hi))
        dt = time.perf_counter() - t0
    return n_elems * (n_inner + 1) / dt, dt


def main_reference(args, rank):
    if rank != 0:
        return
    import oracle
    oracle.build()
    steps, order = oracle_schedule(args.warmup + args.steps)
    n_elems = 1 << 22
    value, dt, passes = run_oracle(n_elems, order, steps, args.warmup, args.steps)
    sample = f"first {n_elems} elements of the layout, every step of the schedule (DyLU inner steps + arrival)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "H": H, "speeds": SPEEDS, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------------
def main_ours(args, rank, world, local_rank):
    import numpy as np
    import torch
    from paper_2401_09135_b200 import binding as B, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    tensors = synth.layout_110m()
    ctx = B.Context(tensors, len(SPEEDS), 4, 0.9, 0.7, grad_staging=True, device=local_rank)
    P = ctx.P
    n_total = args.warmup + args.steps
    steps, order = build_schedule(2 * n_total)
    theta0 = synth.theta0(tensors, ctx.offsets, P, synth.SEED + rank)
    ctx.alsgd_set_global(theta0)
    for w in range(len(SPEEDS)):
        ctx.alsgd_pull(w)
    G = 2
    gpool_host = [torch.from_numpy(synth.normal_vec(P, 1e-2, synth.SEED + rank, synth.STREAM_GRAD, sub=i)).pin_memory()
                  for i in range(G)]
    gpool = [g.cuda(non_blocking=True) for g in gpool_host]
    theta_host = torch.empty(P, dtype=torch.float32).pin_memory()
    life = [0] * len(SPEEDS)
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def run(seq, pool, host_io, timers=None):
        """Runs the arrivals in seq; returns the number of kernel launches."""
        launches = 0
        for w in seq:
            if timers is not None:
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record()
            for _ in range(steps[w]):
                life[w] += 1
                ctx.alsgd_inner_adamw(w, pool[synth.grad_pool_index(w, life[w], G)], life[w], 1e-3)
            if timers is not None:
                e1.record()
            ctx.alsgd_arrive([w], B.ARRIVE_RESEED, want_info=False)
            if timers is not None:
                e2.record()
                timers.append((w, e0, e1, e2))
            if host_io:
                ctx.alsgd_get_global(theta_host)          # waits: the worker's next round needs the model
            launches += steps[w] + 1
        return launches

    # ---- device-resident throughput
    run(order[:args.warmup], gpool, False)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    t_wall0 = time.time()
    start_evt, stop_evt = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    timers = []
    start_evt.record()
    launches = run(order[args.warmup:n_total], gpool, False, timers)
    stop_evt.record()
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    ms = start_evt.elapsed_time(stop_evt)
    passes = launches
    adam_ms = sum(e0.elapsed_time(e1) for _, e0, e1, _ in timers)
    adam_launches = sum(steps[w] for w, *_ in timers)
    arr_ms = sum(e1.elapsed_time(e2) for _, _, e1, e2 in timers)
    arr_launches = len(timers)

    # ---- end to end: gradients come from pinned host memory every inner step, theta goes back each arrival
    e2e_seq = order[n_total:n_total + args.steps]
    run(e2e_seq[:1], gpool_host, True)
    barrier()
    s2, t2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    e2e_launches = run(e2e_seq, gpool_host, True)
    t2.record()
    barrier()
    e2e_ms = s2.elapsed_time(t2)
    h2d = sum(steps[w] for w in e2e_seq) * 4 * P / len(e2e_seq)
    d2h = 4 * P

    # ---- the same AdamW step fed bf16 gradients (28 B/param), reported beside the fp32 figures
    g16 = [g.to(torch.bfloat16) for g in gpool]
    for i in range(3):
        life[0] += 1
        ctx.alsgd_inner_adamw_bf16(0, g16[i % G], life[0], 1e-3)
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record()
    for i in range(20):
        life[0] += 1
        ctx.alsgd_inner_adamw_bf16(0, g16[i % G], life[0], 1e-3)
    b1.record()
    torch.cuda.synchronize()
    adam16_ms = b0.elapsed_time(b1) / 20
    del g16

    from paper_2401_09135_b200 import shard
    ms, e2e_ms, adam_avg_ms, arr_avg_ms = shard.max_over_ranks(
        [ms, e2e_ms, adam_ms / adam_launches, arr_ms / arr_launches], device="cuda")

    if rank == 0:
        peak, which = measured_peak()
        value = world * P * passes / (ms * 1e-3)
        e2e_value = world * P * e2e_launches / (e2e_ms * 1e-3)
        adam_gbs = ADAMW_BYTES * P / (adam_avg_ms * 1e-3) / 1e9
        # arrival bytes: by Delayed-Nesterov phase of each timed arrival (N = 4; the warm-up took ticks 0..warmup-1)
        kinds = ["first" if (args.warmup + i) % 4 == 0 else "boundary" if (args.warmup + i) % 4 == 3 else "middle"
                 for i in range(arr_launches)]
        arr_bytes = sum(ARRIVE_RESEED_BYTES[k] for k in kinds) / float(arr_launches)
        arr_gbs = arr_bytes * P / (arr_avg_ms * 1e-3) / 1e9
        traffic_ok = NCU_TRAFFIC["src_sha256"] == kernel_source_hash()
        adam_traffic = NCU_TRAFFIC["adamw_bytes_per_param"] * P if traffic_ok and NCU_TRAFFIC["adamw_bytes_per_param"] else None
        arr_traffic = NCU_TRAFFIC["arrive_bytes_per_param"] * P if traffic_ok and NCU_TRAFFIC["arrive_bytes_per_param"] else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "P": P, "H": H, "speeds": SPEEDS, "dylu_steps": steps,
                       "step": "one scheduled arrival: DyLU inner AdamW steps of the arriving worker + DN arrival with fused re-seed",
                       "l2": "every launch streams 3.3-3.7 GB (inputs larger than the 126 MB L2); no flush. By design consecutive launches walk the "
                             "vectors in opposite directions, so a step re-touches first what the previous step of the same worker left in L2 "
                             "(worth 1.3 % at this size)",
                       "multi_gpu": "each rank holds its own 110M-element range of an N-times larger vector; no exchange"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / len(e2e_seq)},
            "gpu_launches": launches,
            "roofline": {"kernel": "adamw_kernel (fused AdamW + bf16 cast)", "bound": "hbm", "achieved": adam_gbs,
                         "peak": peak, "peak_source": f"of {which}", "unit": "GB/s", "frac": adam_gbs / peak,
                         "frac_of_nominal_8TBs": adam_gbs / NOMINAL_HBM_GBS, "traffic": adam_traffic,
                         "bytes_per_param": ADAMW_BYTES, "launches": adam_launches, "avg_ms": adam_avg_ms},
            "roofline_arrive": {"kernel": "arrive_kernel<K=1> (pseudo-gradient + Delayed Nesterov + re-seed)", "bound": "hbm",
                                "achieved": arr_gbs, "peak": peak, "peak_source": f"of {which}", "unit": "GB/s",
                                "frac": arr_gbs / peak, "frac_of_nominal_8TBs": arr_gbs / NOMINAL_HBM_GBS,
                                "traffic": arr_traffic, "bytes_per_param": arr_bytes, "launches": arr_launches,
                                "avg_ms": arr_avg_ms},
            "params_per_s": {"adamw": P / (adam_avg_ms * 1e-3), "dn_arrival_reseed": P / (arr_avg_ms * 1e-3)},
            "adamw_bf16_grads": {"avg_ms": adam16_ms, "bytes_per_param": 28, "achieved": 28 * P / (adam16_ms * 1e-3) / 1e9,
                                 "unit": "GB/s", "launches": 20, "note": "extra; not part of the timed steps"},
        }
        for key, traffic in (("roofline", adam_traffic), ("roofline_arrive", arr_traffic)):
            if traffic:           # the same launch on the DRAM bytes ncu counted (dirty L2 lines at kernel end are not in them)
                r = line[key]
                r["achieved_on_measured_traffic"] = traffic / (r["avg_ms"] * 1e-3) / 1e9
                r["frac_of_nominal_8TBs_on_measured_traffic"] = r["achieved_on_measured_traffic"] / NOMINAL_HBM_GBS
    ctx.alsgd_sync()
    ctx.close()
    del ctx, gpool
    torch.cuda.empty_cache()
    if rank == 0:
        if world == 1 and not args.no_extras:
            # the reported figures of the other configurations: arrival batches k = 1, 2, 4, 8 with 8 resident
            # workers, and per-kernel throughput on the 23M / 60M / 110M / 150M layouts
            line["ksweep"] = run_ksweep(args, local_rank)
            line["layouts"] = run_layouts(args, local_rank)
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            n_cpu = P // 4
            cpu_order = [order[0]]
            v, dt, p = run_oracle(n_cpu, cpu_order, steps, 0, 1)
            sample = f"first {n_cpu} elements (a quarter) of the layout, one step: {steps[cpu_order[0]]} inner AdamW steps + 1 arrival with re-seed"
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "seconds": dt, "sample": sample}
            cores = os.cpu_count() or 1
            vn, dtn = run_oracle_all_cores(n_cpu, cpu_order[0], steps[cpu_order[0]], cores)
            line["cpu_baseline"]["all_cores"] = {"value": vn, "unit": UNIT, "cores": cores, "seconds": dtn,
                                                 "how": "the oracle's scalar loops range-split over host threads, same sample"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_ksweep(args, device=0):
    """Arrival-batch sweep on the 110M layout with 8 resident workers (N = 8): per k, each round is 8/k
    batches of k through the multi-arrival kernel with fused re-seed, then 10 AdamW steps per worker."""
    import torch
    from paper_2401_09135_b200 import binding as B, synth
    torch.cuda.set_device(device)
    tensors = synth.layout_110m()
    W, N, inner = 8, 8, 10
    diag = bool(getattr(args, "diag", False))
    arrive_flags = B.ARRIVE_RESEED | ((B.ARRIVE_NORM | B.ARRIVE_NANCHECK) if diag else 0)
    peak, which = measured_peak()
    out = []
    gpool = None
    for k in (1, 2, 4, 8):
        ctx = B.Context(tensors, W, N, 0.9, 0.7, device=device)
        P = ctx.P
        if gpool is None:
            gpool = [torch.from_numpy(synth.normal_vec(P, 1e-2, synth.SEED, synth.STREAM_GRAD, sub=i)).cuda() for i in range(2)]
        ctx.alsgd_set_global(synth.theta0(tensors, ctx.offsets, P))
        for w in range(W):
            ctx.alsgd_pull(w)
        order = [int(w) for w in synth.rng(synth.SEED + 8, synth.STREAM_ORDER, k).permutation(W)]
        life = [0] * W
        rounds = args.warmup // 4 + 1 + max(5, args.steps // 3)
        ev = []
        for r in range(rounds):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record()
            for i in range(0, W, k):
                ctx.alsgd_arrive(order[i:i + k], arrive_flags, want_info=False)
            e1.record()
            for w in range(W):
                for _ in range(inner):
                    life[w] += 1
                    ctx.alsgd_inner_adamw(w, gpool[synth.grad_pool_index(w, life[w], 2)], life[w], 1e-3)
            e2.record()
            ev.append((e0, e1, e2))
        torch.cuda.synchronize()
        ev = ev[1:]                                        # first round is warm-up
        arr_ms = sum(a.elapsed_time(b) for a, b, _ in ev) / len(ev)
        adam_ms = sum(b.elapsed_time(c) for _, b, c in ev) / len(ev)
        # one full cycle per round (N = W = 8): theta read+written per batch, Delta read on all batches but the
        # first and written on all but the last, m read+written once; per batch k worker vectors and the one
        # snapshot its workers share are read, k bf16 replicas and one new snapshot are written
        nb = W // k
        arr_bytes = (8 * nb + 8 * (nb - 1) + 8 + nb * (4 * k + 4) + nb * (2 * k + 4)) * P
        adam_bytes = ADAMW_BYTES * P * W * inner
        out.append({"k": k, "arrival_ms_per_round": arr_ms, "arrival_gbs": arr_bytes / arr_ms / 1e6,
                    "arrival_frac": arr_bytes / arr_ms / 1e6 / peak, "arrival_bytes_per_param_per_arrival": arr_bytes / P / W,
                    "arrivals_per_s": W / (arr_ms * 1e-3), "adamw_ms_per_round": adam_ms,
                    "adamw_gbs": adam_bytes / adam_ms / 1e6, "adamw_frac": adam_bytes / adam_ms / 1e6 / peak,
                    "combined_gbs": (arr_bytes + adam_bytes) / (arr_ms + adam_ms) / 1e6,
                    "combined_frac": (arr_bytes + adam_bytes) / (arr_ms + adam_ms) / 1e6 / peak,
                    "arrival_frac_of_8TBs": arr_bytes / arr_ms / 1e6 / NOMINAL_HBM_GBS,
                    "adamw_frac_of_8TBs": adam_bytes / adam_ms / 1e6 / NOMINAL_HBM_GBS})
        ctx.alsgd_sync()
        ctx.close()
        del ctx
        torch.cuda.empty_cache()
    return {"workload": "decoder-110M W=8 N=8 beta=0.9 outer_lr=0.7, k-sweep, 10 inner AdamW steps per worker per round"
                        + (", squared-norm and non-finite diagnostics on every arrival" if diag else ""),
            "peak_gbs": peak, "peak_source": f"of {which}", "unit": "GB/s", "rounds_timed": len(ev), "sweep": out}


def main_ksweep(args):
    print(json.dumps(run_ksweep(args)), flush=True)


def run_layouts(args, device=0):
    """Per-kernel throughput on layouts shaped like the paper's 20M-150M decoder transformers (2 workers, N = 4):
    20 AdamW steps and 20 single arrivals with fused re-seed each, CUDA events, after 4 warm-up launches.
    Below ~30M elements one fp32 buffer fits in L2, so those rows are not HBM-roofline figures."""
    import torch
    from paper_2401_09135_b200 import binding as B, synth
    torch.cuda.set_device(device)
    peak, which = measured_peak()
    out = []
    for name, tensors in (("23M (6L, d384, ff1536)", synth.layout_23m()), ("paper 60M (3L, h896, 16x64)", synth.layout_paper_60m()),
                          ("110M (12L, d768, ff3072)", synth.layout_110m()), ("paper 150M (12L, h896, 16x64)", synth.layout_paper_150m())):
        ctx = B.Context(tensors, 2, 4, 0.9, 0.7, device=device)
        P = ctx.P
        ctx.alsgd_set_global(synth.theta0(tensors, ctx.offsets, P))
        g = [torch.from_numpy(synth.normal_vec(P, 1e-2, synth.SEED, synth.STREAM_GRAD, sub=i)).cuda() for i in range(2)]
        for w in range(2):
            ctx.alsgd_pull(w)
        step = 0

        def adam(n):
            nonlocal step
            for i in range(n):
                step += 1
                ctx.alsgd_inner_adamw(i % 2, g[i % 2], step, 1e-3)

        res = {"layout": name, "P": P}
        adam(4)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); adam(20); e1.record(); torch.cuda.synchronize()
        times = {"adamw": e0.elapsed_time(e1) / 20}
        # arrivals: one AdamW step of the arriving worker (untimed) before each, so that the arrival reads the
        # worker's own parameters and not the snapshot it was dispatched with
        pairs = []
        for i in range(24):
            w = i % 2
            step += 1
            ctx.alsgd_inner_adamw(w, g[w], step, 1e-3)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            ctx.alsgd_arrive([w], B.ARRIVE_RESEED, want_info=False)
            a1.record()
            pairs.append((a0, a1))
        torch.cuda.synchronize()
        times["arrive_reseed"] = sum(x.elapsed_time(y) for x, y in pairs[4:]) / 20
        for key, bpp in (("adamw", ADAMW_BYTES), ("arrive_reseed", 30.0)):
            ms = times[key]
            res[key] = {"ms": ms, "params_per_s": P / (ms * 1e-3), "gbs": bpp * P / (ms * 1e-3) / 1e9,
                        "frac_of_measured": bpp * P / (ms * 1e-3) / 1e9 / peak, "frac_of_8TBs": bpp * P / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS}
        out.append(res)
        ctx.alsgd_sync()
        ctx.close(); del ctx, g
        torch.cuda.empty_cache()
    return {"peak_gbs": peak, "peak_source": f"of {which}", "unit": "GB/s",
            "note": "2 workers, N = 4; 20 AdamW steps and 20 single arrivals with fused re-seed per layout, CUDA events; "
                    "one fp32 vector of the 23M layout (92 MB) fits in the 126 MB L2, so that row is no HBM roofline figure",
            "layouts": out}


def main_layouts(args):
    print(json.dumps(run_layouts(args)), flush=True)


def main_shape_sweep(args):
    """Times many launch shapes of the product's kernel bodies (libalsgd_sweep.so) at the 110M size: threads per
    block, vectors per thread, resident-block caps, one tile per block against a persistent loop, scalar against
    packed two-lane arithmetic, per-arrival against shared dispatch snapshot, with and without diagnostics.
    Prints one JSON object: every row, and the best shape per (kernel, K, snapshot mode, diagnostics)."""
    import torch
    from paper_2401_09135_b200 import sweep
    torch.cuda.set_device(0)
    n = args.sweep_elems
    peak, which = measured_peak()
    segments = None
    if n == 109_549_056:             # the default size: AdamW walks the real weight-decay table of the 110M layout
        from paper_2401_09135_b200 import binding as B, synth
        tensors = synth.layout_110m()
        P, offsets = B.alsgd_layout_size(tensors)
        assert P == n
        segments = sweep.decay_segments(tensors, offsets, P)
    kinds = {"all": None, "adamw": sweep.KIND_ADAMW, "arrive": sweep.KIND_ARRIVE}[args.sweep_kind]
    # --sweep-product-launch: launch the way the library does (programmatic dependent launch; AdamW walking the vector
    # in the opposite direction of the previous launch) instead of plain identical launches
    dep, alt = (0x100, 0x200) if args.sweep_product_launch else (0, 0)
    rows = sweep.run(n, reps=args.sweep_reps, warmup=3, segments=segments, adam_phase=dep | alt,
                     phase_for=(lambda v: (sweep.PHASE_CYCLE if v["K"] == 8 else sweep.PHASE_MIDDLE) | dep) if dep else None,
                     select=(lambda v: v["kind"] == kinds) if kinds is not None else None,
                     log=(lambda r: print(json.dumps(r), file=sys.stderr, flush=True)) if args.verbose else None)
    best = {}
    for r in rows:
        if r["persistent"]:
            continue
        key = ("adamw" if r["kind"] == sweep.KIND_ADAMW else f"arrive K={r['K']} base={sweep.BASE_NAMES[r['base_mode']]}") + (" diag" if r["diag"] else "")
        if key not in best or r["gbs"] > best[key]["gbs"]:
            best[key] = r
    print(json.dumps({"elements": n, "reps": args.sweep_reps, "product_launch": bool(args.sweep_product_launch), "peak_gbs": peak, "peak_source": f"of {which}",
                      "unit": "GB/s on algorithmic bytes", "best": best, "rows": rows}), flush=True)


def main_profile_case(args):
    """Small fixed cases for profiler captures: a few launches of each kernel on vectors larger than L2 but only a
    few GB on the device in total.
      single   2 workers, N = 4, 48Mi elements (2.4 GB): 2 pulls, 3 AdamW steps per worker, then four times (AdamW
               step, single arrival with fused re-seed) through one Delayed-Nesterov cycle (first / middle / middle /
               boundary), one AdamW step per worker, one batch of two
      batches  8 workers, N = 8, 32Mi elements (4.3 GB): pulls, one AdamW step each, two batches of 4, one AdamW step
               each, one batch of 8 (all sharing one dispatch snapshot)
      diag     the batches case with the squared-norm / non-finite diagnostics requested on every arrival"""
    import torch
    from paper_2401_09135_b200 import binding as B, synth
    torch.cuda.set_device(0)
    mode = args.profile_case
    if mode in ("batches", "diag"):
        flags = B.ARRIVE_RESEED | ((B.ARRIVE_NORM | B.ARRIVE_NANCHECK) if mode == "diag" else 0)
        tensors = synth.flat_tensors(32 * 1024 * 1024)
        W = 8
        ctx = B.Context(tensors, W, 8, 0.9, 0.7)
        ctx.alsgd_set_global(synth.theta0(tensors, ctx.offsets, ctx.P))
        g = torch.from_numpy(synth.normal_vec(ctx.P, 1e-2, synth.SEED, synth.STREAM_GRAD)).cuda()
        for w in range(W):
            ctx.alsgd_pull(w)
        for w in range(W):
            ctx.alsgd_inner_adamw(w, g, 1, 1e-3)
        ctx.alsgd_arrive([0, 1, 2, 3], flags, want_info=False)     # first of the cycle, one shared snapshot
        ctx.alsgd_arrive([4, 5, 6, 7], flags, want_info=False)     # ends the cycle of N = 8 (boundary inside)
        for w in range(W):
            ctx.alsgd_inner_adamw(w, g, 2, 1e-3)
        ctx.alsgd_arrive(list(range(W)), flags, want_info=False)   # whole cycle in one pass, two snapshots among the 8
        for w in range(W):
            ctx.alsgd_inner_adamw(w, g, 3, 1e-3)
        ctx.alsgd_arrive(list(range(W)), flags, want_info=False)   # whole cycle in one pass, all 8 share one snapshot
    else:
        n = 48 * 1024 * 1024
        tensors = [synth.Tensor("w0", n // 2, True, "matrix"), synth.Tensor("g0", 4096, False, "gain"),
                   synth.Tensor("w1", n - n // 2 - 4096, True, "matrix")]
        ctx = B.Context(tensors, 2, 4, 0.9, 0.7)
        ctx.alsgd_set_global(synth.theta0(tensors, ctx.offsets, ctx.P))
        g = torch.from_numpy(synth.normal_vec(ctx.P, 1e-2, synth.SEED, synth.STREAM_GRAD)).cuda()
        for w in range(2):
            ctx.alsgd_pull(w)
        for w in range(2):
            for st in range(1, 4):
                ctx.alsgd_inner_adamw(w, g, st, 1e-3)
        step = [3, 3]
        for w in (0, 1, 0, 1):
            step[w] += 1
            ctx.alsgd_inner_adamw(w, g, step[w], 1e-3)
            ctx.alsgd_arrive([w], B.ARRIVE_RESEED, want_info=False)
        for w in range(2):
            step[w] += 1
            ctx.alsgd_inner_adamw(w, g, step[w], 1e-3)
        ctx.alsgd_arrive([0, 1], B.ARRIVE_RESEED, want_info=False)
    ctx.alsgd_sync()
    print(f"profile case {mode} done: P={ctx.P}, t={ctx.alsgd_counters()[0]}")
    ctx.close()


def main_cpu_kernels(args):
    """The oracle's two loops timed per kernel on the host: one core as written, and the same scalar
    loops range-split over all host cores (exact, the path is elementwise)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    import oracle
    from paper_2401_09135_b200 import synth
    oracle.build()
    cores = os.cpu_count() or 1
    n = 109_549_056 // 8
    z = lambda: np.zeros(n, np.float32)
    theta, m, D, p, base, am, av = (synth.normal_vec(n, 0.02, synth.SEED, synth.STREAM_THETA0), z(), z(),
                                    synth.normal_vec(n, 0.02, synth.SEED, synth.STREAM_DELTA), z(), z(), z())
    g = synth.normal_vec(n, 1e-2, synth.SEED, synth.STREAM_GRAD)
    rep = np.zeros(n, np.uint16)
    decay = np.ones(n, np.uint8)

    def arrive(lo, hi, t):
        oracle.dn_arrive(theta, m, D, base, p, t, 4, 0.9, 0.7, lo=lo, hi=hi)
        oracle.reseed(theta, p, base, rep, lo=lo, hi=hi)

    def adam(lo, hi, t):
        oracle.adamw(p, am, av, g, rep, decay, t + 1, 1e-3, 0.9, 0.95, 1e-8, 0.1, lo=lo, hi=hi)

    def rate(fn, threads, reps=3):
        cuts = [n * i // threads for i in range(threads + 1)]
        best = None
        with ThreadPoolExecutor(threads) as ex:
            for r in range(reps + 1):
                t0 = time.perf_counter()
                list(ex.map(lambda i: fn(cuts[i], cuts[i + 1], r), range(threads)))
                dt = time.perf_counter() - t0
                if r > 0:
                    best = dt if best is None else min(best, dt)
        return n / best

    out = {"elements": n, "cores": cores,
           "dn_arrival_reseed": {"1_core": rate(arrive, 1), "n_cores": rate(arrive, cores), "bytes_per_param": 34},
           "adamw_bf16": {"1_core": rate(adam, 1), "n_cores": rate(adam, cores), "bytes_per_param": 30},
           "unit": "params/s", "kind": "oracle"}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the k-sweep and layout tables of the default line")
    ap.add_argument("--ksweep", action="store_true", help="arrival-batch sweep (k = 1, 2, 4, 8) with 8 resident workers")
    ap.add_argument("--diag", action="store_true", help="with --ksweep: request the diagnostics on every arrival")
    ap.add_argument("--layouts", action="store_true", help="per-kernel throughput on 23M / 60M / 110M / 150M layouts")
    ap.add_argument("--cpu-kernels", action="store_true", help="time the oracle's loops per kernel on the host cores")
    ap.add_argument("--profile-case", choices=["single", "batches", "diag"], help="run a small fixed case for a profiler capture")
    ap.add_argument("--shape-sweep", action="store_true", help="time the launch shapes of libalsgd_sweep.so")
    ap.add_argument("--sweep-elems", type=int, default=109_549_056)
    ap.add_argument("--sweep-reps", type=int, default=10)
    ap.add_argument("--sweep-kind", choices=["all", "adamw", "arrive"], default="all")
    ap.add_argument("--sweep-product-launch", action="store_true",
                    help="shape sweep with dependent launches and alternating direction, as the library launches")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.profile_case:
        main_profile_case(args)
    elif args.shape_sweep:
        main_shape_sweep(args)
    elif args.layouts:
        main_layouts(args)
    elif args.cpu_kernels:
        main_cpu_kernels(args)
    elif args.ksweep:
        main_ksweep(args)
    elif args.impl == "reference":
        main_reference(args, rank)
    else:
        main_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
