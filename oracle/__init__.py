"""CPU oracle (test infrastructure only).

Plain single-threaded C++ (``alsgd_oracle.cpp``) reached through ctypes, plus ``OracleServer``: the
bookkeeping around it (server tick, Delayed-Nesterov phase, pull ticks, staleness) written out as
ordinary Python over numpy arrays.  Nothing here imports, links or reads the CUDA library; only the
test-suite, the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "alsgd_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no FMA contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math",
                               "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_f32p = C.POINTER(C.c_float)
_u16p = C.POINTER(C.c_uint16)
_u8p = C.POINTER(C.c_uint8)
_u32p = C.POINTER(C.c_uint32)
_f64p = C.POINTER(C.c_double)


def _configure(L):
    """Declare the argument and result types of every oracle function on a loaded library."""
    L.orc_bf16_rne.argtypes = [C.c_uint32]
    L.orc_bf16_rne.restype = C.c_uint16
    L.orc_cast_bf16.argtypes = [_f32p, _u16p, C.c_uint64, C.c_uint64]
    L.orc_cast_bf16.restype = None
    L.orc_inv_n.argtypes = [C.c_uint32]
    L.orc_inv_n.restype = C.c_float
    L.orc_boundary_weight.argtypes = [C.c_uint32, C.c_float, C.c_float]
    L.orc_boundary_weight.restype = C.c_float
    L.orc_between_weight.argtypes = [C.c_float, C.c_float]
    L.orc_between_weight.restype = C.c_float
    L.orc_dn_arrive.argtypes = [_f32p, _f32p, _f32p, _f32p, _f32p, C.c_uint64, C.c_uint64, C.c_uint64,
                                C.c_uint32, C.c_float, C.c_float, C.c_float, C.c_int, C.c_float,
                                C.c_float, C.c_int]
    L.orc_dn_arrive.restype = C.c_int
    L.orc_pg_norm2.argtypes = [_f32p, _f32p, _f32p, C.c_uint64, C.c_uint64, C.c_int, _u32p]
    L.orc_pg_norm2.restype = C.c_double
    L.orc_reseed.argtypes = [_f32p, _f32p, _f32p, _u16p, C.c_uint64, C.c_uint64]
    L.orc_reseed.restype = None
    L.orc_adamw.argtypes = [_f32p, _f32p, _f32p, _f32p, _u16p, _u8p, C.c_uint64, C.c_uint64, C.c_uint64,
                            C.c_float, C.c_float, C.c_float, C.c_float, C.c_float]
    L.orc_adamw.restype = None
    L.orc_dylu.argtypes = [_f64p, C.c_uint32, C.c_uint32, _u32p]
    L.orc_dylu.restype = None
    L.orc_lr_at.argtypes = [C.c_double, C.c_double, C.c_uint64, C.c_uint64, C.c_uint64]
    L.orc_lr_at.restype = C.c_double
    L.orc_poly_weight.argtypes = [C.c_uint64]
    L.orc_poly_weight.restype = C.c_float
    L.orc_shard_probs.argtypes = [_f64p, _f64p, C.c_uint32, _f64p]
    L.orc_shard_probs.restype = None
    L.orc_schedule.argtypes = [C.c_uint32, _f64p, C.c_uint32, _u32p, C.c_double, C.c_uint64, C.c_uint32,
                               _u32p, _f64p, _u32p]
    L.orc_schedule.restype = C.c_uint32
    return L


def lib():
    global _lib
    if _lib is None:
        _lib = _configure(C.CDLL(build()))
    return _lib


def _p(a, ty):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ty)


# ---- thin array-level wrappers ------------------------------------------------------------------

def bf16_rne_bits(bits: int) -> int:
    return int(lib().orc_bf16_rne(int(bits) & 0xFFFFFFFF))


def cast_bf16(src: np.ndarray) -> np.ndarray:
    src = np.ascontiguousarray(src, dtype=np.float32)
    out = np.empty(src.shape[0], dtype=np.uint16)
    lib().orc_cast_bf16(_p(src, _f32p), _p(out, _u16p), 0, src.shape[0])
    return out


OUTER_DN, OUTER_BUFFERED, OUTER_SGDM = 0, 1, 2


def dn_arrive(theta, m, Delta, base, p, t, N, beta, eps, c=0.0, pg_current=False, weight=1.0,
              dc_lambda=0.0, buffered=False, lo=0, hi=None) -> bool:
    """One arrival of Algorithm 3 in place on float32 arrays; returns the boundary flag.

    buffered: False / OUTER_DN = Delayed Nesterov; True / OUTER_BUFFERED = "Async. Buffer" (Nesterov step
    on the buffer mean at every N-th arrival); OUTER_SGDM = the same with the SGD Momentum step."""
    hi = theta.shape[0] if hi is None else hi
    for a in (theta, m, Delta, p):
        assert a.dtype == np.float32
    if base is None:
        assert pg_current
        base = theta
    return bool(lib().orc_dn_arrive(_p(theta, _f32p), _p(m, _f32p), _p(Delta, _f32p), _p(base, _f32p),
                                    _p(p, _f32p), lo, hi, int(t), int(N), float(beta), float(eps),
                                    float(c), int(bool(pg_current)), float(weight), float(dc_lambda),
                                    int(buffered)))


def pg_norm2(theta, base, p, pg_current=False, lo=0, hi=None):
    hi = theta.shape[0] if hi is None else hi
    bad = C.c_uint32(0)
    if base is None:
        base = theta
    s = lib().orc_pg_norm2(_p(theta, _f32p), _p(base, _f32p), _p(p, _f32p), lo, hi, int(bool(pg_current)),
                           C.byref(bad))
    return float(s), int(bad.value)


def reseed(theta, p, base, replica, lo=0, hi=None):
    hi = theta.shape[0] if hi is None else hi
    lib().orc_reseed(_p(theta, _f32p), _p(p, _f32p), _p(base, _f32p), _p(replica, _u16p), lo, hi)


def adamw(p, m, v, g, replica, decay, step, lr, b1, b2, eps, wd, lo=0, hi=None):
    hi = p.shape[0] if hi is None else hi
    assert g.dtype == np.float32 and p.dtype == np.float32
    lib().orc_adamw(_p(p, _f32p), _p(m, _f32p), _p(v, _f32p), _p(g, _f32p), _p(replica, _u16p),
                    _p(decay, _u8p), lo, hi, int(step), float(lr), float(b1), float(b2), float(eps), float(wd))


def dylu(speeds, H):
    sp = np.ascontiguousarray(speeds, dtype=np.float64)
    out = np.zeros(sp.shape[0], dtype=np.uint32)
    lib().orc_dylu(_p(sp, _f64p), sp.shape[0], int(H), _p(out, _u32p))
    return [int(x) for x in out]


def lr_at(eta_max, eta_min, t_warmup, T, t) -> float:
    return float(lib().orc_lr_at(float(eta_max), float(eta_min), int(t_warmup), int(T), int(t)))


def poly_weight(staleness: int) -> float:
    return float(lib().orc_poly_weight(int(staleness)))


def shard_probs(sizes, learned):
    """Eq. 2: sampling probability of every data shard."""
    s = np.ascontiguousarray(sizes, dtype=np.float64)
    l = np.ascontiguousarray(learned, dtype=np.float64)
    out = np.zeros(s.shape[0], dtype=np.float64)
    lib().orc_shard_probs(_p(s, _f64p), _p(l, _f64p), s.shape[0], _p(out, _f64p))
    return [float(x) for x in out]


def schedule(durations, local_updates, tau_grace, t_max, max_arrivals):
    """Algorithm 2 + 5 on faked time.  Returns (workers, times, batch_index) lists."""
    d = np.ascontiguousarray(durations, dtype=np.float64)
    W, R = d.shape
    lu = np.ascontiguousarray(local_updates, dtype=np.uint32)
    ow = np.zeros(max_arrivals, dtype=np.uint32)
    ot = np.zeros(max_arrivals, dtype=np.float64)
    ob = np.zeros(max_arrivals, dtype=np.uint32)
    n = lib().orc_schedule(W, _p(d, _f64p), R, _p(lu, _u32p), float(tau_grace), int(t_max), int(max_arrivals),
                           _p(ow, _u32p), _p(ot, _f64p), _p(ob, _u32p))
    return [int(x) for x in ow[:n]], [float(x) for x in ot[:n]], [int(x) for x in ob[:n]]


def layout_offsets(numels, align_elems: int):
    """Flat offsets of a tensor list: each tensor starts at the next multiple of align_elems; the
    total is rounded up the same way.  Returns (offsets, P)."""
    offs, cur = [], 0
    for n in numels:
        offs.append(cur)
        cur += int(n)
        cur = (cur + align_elems - 1) // align_elems * align_elems
    return offs, cur


def decay_mask(numels, decays, offsets, P) -> np.ndarray:
    """Per-element weight-decay flag (padding is never decayed)."""
    mask = np.zeros(int(P), dtype=np.uint8)
    for n, d, off in zip(numels, decays, offsets):
        if d:
            mask[int(off):int(off) + int(n)] = 1
    return mask


# ---- the server, as the paper states it -----------------------------------------------------------

class OracleServer:
    """Server state of Algorithm 3 (theta, m, Delta, t) and W worker replicas (parameters, dispatch
    snapshot, AdamW moments, bf16 copy), advanced one call at a time with the scalar oracle."""

    def __init__(self, P, n_workers, N, beta, outer_lr, c=0.0, pg_current=False, decay=None,
                 adam=(0.9, 0.95, 1e-8, 0.1), replica=True):
        self.P, self.W, self.N = int(P), int(n_workers), int(N)
        self.beta, self.eps, self.c = np.float32(beta), np.float32(outer_lr), np.float32(c)
        self.pg_current = bool(pg_current)
        self.adam = tuple(np.float32(x) for x in adam)
        self.decay = decay if decay is not None else np.zeros(self.P, dtype=np.uint8)
        z = lambda: np.zeros(self.P, dtype=np.float32)
        self.theta, self.m, self.Delta = z(), z(), z()
        self.t = 0
        self.p = [z() for _ in range(self.W)]
        self.base = [z() for _ in range(self.W)]
        self.am = [z() for _ in range(self.W)]
        self.av = [z() for _ in range(self.W)]
        self.replica = [np.zeros(self.P, dtype=np.uint16) for _ in range(self.W)] if replica else [None] * self.W
        self.pull_tick = [None] * self.W

    def set_global(self, theta0):
        self.theta[:] = theta0

    def pull(self, w):
        reseed(self.theta, self.p[w], self.base[w], self.replica[w])
        self.pull_tick[w] = self.t

    def inner_adamw(self, w, grads, step, lr):
        b1, b2, eps, wd = self.adam
        adamw(self.p[w], self.am[w], self.av[w], grads, self.replica[w], self.decay, step, lr, b1, b2, eps, wd)

    def arrive(self, ids, reseed_after=True, norm=False, weights=None, dc_lambda=0.0, buffered=False,
               poly=False, stale_threshold=None):
        """Apply the arrivals of one grace window in the given order, then (optionally) re-dispatch
        all of them with the final global model.  Returns one info dict per arrival.

        poly: weight each pseudo-gradient by (1 + staleness)^-0.5 (Section 4, "Async. DiLoCo + Poly").
        stale_threshold: with poly, discard updates whose staleness exceeds it ("PolyThres"); a
        discarded update is not a server update (t does not advance) but its worker is re-dispatched."""
        infos = []
        for j, w in enumerate(ids):
            stale = self.t - self.pull_tick[w]
            info = {"worker": w, "tick": self.t, "staleness": stale, "dropped": False, "boundary": False}
            if poly and stale_threshold is not None and stale > stale_threshold:
                info["dropped"] = True                 # never looked at: no diagnostics either
                info["gnorm2"], info["nonfinite"] = 0.0, 0
                infos.append(info)
                continue
            if norm:
                info["gnorm2"], info["nonfinite"] = pg_norm2(self.theta, self.base[w], self.p[w], self.pg_current)
            wt = 1.0 if weights is None else weights[j]
            if poly:
                wt = poly_weight(stale)
            info["boundary"] = dn_arrive(self.theta, self.m, self.Delta, self.base[w], self.p[w], self.t, self.N,
                                         self.beta, self.eps, self.c, self.pg_current, wt, dc_lambda, buffered)
            self.t += 1
            infos.append(info)
        if reseed_after:
            for w in ids:
                self.pull(w)
        return infos
