"""ctypes binding of the launch-shape benchmark library (include/alsgd_sweep.h) and the sweep loop.

The library holds many launch shapes of the product's kernel bodies; this module allocates one set of
buffers with torch, times every shape with CUDA events on the current stream and returns the table.
Marshalling and timing only; used by ``bench.py --shape-sweep``.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libalsgd_sweep.so")

KIND_ADAMW, KIND_ARRIVE = 0, 1
PHASE_MIDDLE, PHASE_CYCLE = 0, 1
BASE_NAMES = {0: "per-arrival", 1: "shared", 2: "current"}


class Variant(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("kind", "K", "base_mode", "V", "block", "min_blocks", "persistent",
                                          "packed", "diag", "staged")]


class Buffers(C.Structure):
    _fields_ = [("n", C.c_uint64), ("theta", C.c_void_p), ("delta", C.c_void_p), ("mom", C.c_void_p),
                ("p", C.c_void_p * 8), ("base", C.c_void_p * 8), ("snapshot", C.c_void_p), ("rep", C.c_void_p * 8),
                ("adam_p", C.c_void_p), ("adam_m", C.c_void_p), ("adam_v", C.c_void_p), ("adam_g", C.c_void_p),
                ("adam_rep", C.c_void_p), ("seg_end", C.c_void_p), ("seg_decay", C.c_void_p),
                ("n_seg", C.c_uint32), ("reserved", C.c_uint32),
                ("diag_scratch", C.c_void_p), ("diag_out", C.c_void_p), ("diag_flags", C.c_void_p), ("diag_state", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        from . import build as _build
        if _build.needs_build("sweep"):
            _build.build(targets=("sweep",))
        L = C.CDLL(LIB_PATH)
        L.alsgd_sweep_count.restype = C.c_int
        L.alsgd_sweep_describe.argtypes = [C.c_int, C.POINTER(Variant)]
        L.alsgd_sweep_describe.restype = C.c_int
        L.alsgd_sweep_launch.argtypes = [C.c_int, C.POINTER(Buffers), C.c_uint32, C.c_void_p]
        L.alsgd_sweep_launch.restype = C.c_int
        _lib = L
    return _lib


def variants():
    L = lib()
    out = []
    for i in range(L.alsgd_sweep_count()):
        v = Variant()
        assert L.alsgd_sweep_describe(i, C.byref(v)) == 0
        out.append({n: int(getattr(v, n)) for n, _ in Variant._fields_})
        out[-1]["index"] = i
    return out


def arrive_bytes_per_param(K, base_mode, phase):
    """Algorithmic bytes per parameter of one arrival pass that also re-seeds its K workers: theta read + written,
    Delta read + written (middle of a cycle) or m read + written (whole cycle in one pass), K worker vectors and
    the snapshots read, one new snapshot and K bf16 replicas written."""
    bases = {0: K, 1: 1, 2: 0}[base_mode]
    return 8 + 8 + 4 * K + 4 * bases + 4 + 2 * K


ADAMW_BYTES_PER_PARAM = 30


def decay_segments(tensors, offsets, P):
    """Maximal runs of equal weight-decay flag over the flat vector (padding is its own undecayed run): the table
    the AdamW kernel walks.  tensors have .numel and .decay."""
    ends, flags = [], []

    def push(end, flag):
        if ends and flags[-1] == flag:
            ends[-1] = end
        else:
            ends.append(end)
            flags.append(flag)
    for i, (t, off) in enumerate(zip(tensors, offsets)):
        end = off + t.numel
        push(end, 1 if t.decay else 0)
        nxt = offsets[i + 1] if i + 1 < len(offsets) else P
        if nxt != end:
            push(nxt, 0)
    return ends, flags


def run(n, select=None, reps=10, warmup=3, phase_for=None, log=None, segments=None, adam_phase=0):
    """Time every variant (or those select(v) accepts) on vectors of n elements.  Returns a list of dicts with
    the variant's fields, the phase, ms per launch and GB/s on the algorithmic bytes."""
    import torch
    L = lib()
    dev = torch.device("cuda", torch.cuda.current_device())
    f32 = lambda scale: torch.randn(n, device=dev, dtype=torch.float32) * scale
    keep = []

    def hold(t):
        keep.append(t)
        return t.data_ptr()

    b = Buffers()
    b.n = n
    b.theta, b.delta, b.mom = hold(f32(0.02)), hold(torch.zeros(n, device=dev)), hold(torch.zeros(n, device=dev))
    for j in range(8):
        b.p[j] = hold(f32(0.02))
        b.base[j] = hold(f32(0.02))
        b.rep[j] = hold(torch.empty(n, device=dev, dtype=torch.int16))
    b.snapshot = hold(torch.empty(n, device=dev))
    b.adam_p, b.adam_m, b.adam_v = hold(f32(0.02)), hold(torch.zeros(n, device=dev)), hold(torch.zeros(n, device=dev))
    b.adam_g, b.adam_rep = hold(f32(0.01)), hold(torch.empty(n, device=dev, dtype=torch.int16))
    seg_end, seg_decay = segments if segments is not None else ([n], [1])
    assert seg_end[-1] == n
    b.seg_end = hold(torch.tensor(seg_end, device=dev, dtype=torch.int64))
    b.seg_decay = hold(torch.tensor(seg_decay, device=dev, dtype=torch.int32))
    b.n_seg = len(seg_end)
    b.diag_scratch = hold(torch.zeros(8 * (n // 256 + 66), device=dev, dtype=torch.float64))
    b.diag_out = hold(torch.zeros(8, device=dev, dtype=torch.float64))
    keep_flags = torch.zeros(8, device=dev, dtype=torch.int32)
    b.diag_flags = hold(keep_flags)
    b.diag_state = hold(torch.zeros(16, device=dev, dtype=torch.int32))
    stream = torch.cuda.current_stream().cuda_stream
    rows = []
    for v in variants():
        if select is not None and not select(v):
            continue
        if v["kind"] == KIND_ARRIVE:
            phase = phase_for(v) if phase_for else (PHASE_CYCLE if v["K"] == 8 else PHASE_MIDDLE)
            bpp = arrive_bytes_per_param(v["K"], v["base_mode"], phase & 0xFF)
        else:
            phase, bpp = adam_phase, ADAMW_BYTES_PER_PARAM
        for _ in range(warmup):
            rc = L.alsgd_sweep_launch(v["index"], C.byref(b), phase, stream)
            if rc != 0:
                raise RuntimeError(f"sweep variant {v}: cudaError {rc}")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            L.alsgd_sweep_launch(v["index"], C.byref(b), phase, stream)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        if v["staged"] and int(keep_flags[7].item()) != 0:
            raise RuntimeError(f"sweep variant {v}: a bounded wait ran out")
        row = dict(v, phase=phase, bytes_per_param=bpp, ms=ms, gbs=bpp * n / ms / 1e6)
        rows.append(row)
        if log:
            log(row)
    return rows
