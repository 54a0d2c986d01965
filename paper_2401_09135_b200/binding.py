"""Thin ctypes binding of the C ABI declared in include/alsgd.h.

Argument marshalling only: every step of the server path and of the inner optimizer runs in the
library's CUDA kernels.  There is no CPU fallback; loading fails loudly when libalsgd.so is missing
and cannot be built.  PyTorch is used for the device arena, the stream and tensor views of the
borrowed device pointers.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libalsgd.so")

OK, E_ARG, E_RANGE, E_STATE, E_CUDA, E_NOMEM, E_UNSUPPORTED, E_BOUNDS = 0, -1, -2, -3, -4, -5, -6, -7
TENSOR_DECAY = 1
PG_DISPATCH, PG_CURRENT = 0, 1
CFG_REPLICA_BF16, CFG_GRAD_STAGING, CFG_OUTER_BUFFERED, CFG_OUTER_SGDM, CFG_STABLE_PTRS = 1, 2, 4, 8, 16
STALE_NONE, STALE_POLY, STALE_POLY_THRES = 0, 1, 2
ARRIVE_RESEED, ARRIVE_NORM, ARRIVE_NANCHECK = 1, 2, 4


class TensorDesc(C.Structure):
    _fields_ = [("numel", C.c_uint64), ("flags", C.c_uint32), ("reserved", C.c_uint32)]


class Config(C.Structure):
    _fields_ = [("n_workers", C.c_uint32), ("N", C.c_uint32), ("pg_base", C.c_uint32), ("flags", C.c_uint32),
                ("beta", C.c_float), ("outer_lr", C.c_float), ("c", C.c_float),
                ("adam_b1", C.c_float), ("adam_b2", C.c_float), ("adam_eps", C.c_float), ("adam_wd", C.c_float),
                ("device", C.c_int32), ("stream", C.c_void_p), ("arena", C.c_void_p), ("arena_bytes", C.c_uint64)]


class ArrivalInfo(C.Structure):
    _fields_ = [("tick", C.c_uint64), ("staleness", C.c_uint64), ("gnorm2", C.c_double),
                ("worker", C.c_uint32), ("boundary", C.c_uint32), ("nonfinite", C.c_uint32), ("dropped", C.c_uint32)]


class ArriveOpts(C.Structure):
    _fields_ = [("weights", C.POINTER(C.c_float)), ("dc_lambda", C.c_float), ("staleness_rule", C.c_uint32),
                ("stale_threshold", C.c_uint32), ("reserved", C.c_uint32)]


class Ptrs(C.Structure):
    _fields_ = [("theta", C.c_void_p), ("m", C.c_void_p), ("delta", C.c_void_p), ("P", C.c_uint64),
                ("n_workers", C.c_uint32), ("reserved", C.c_uint32)]


class WorkerPtrs(C.Structure):
    _fields_ = [("p", C.c_void_p), ("base", C.c_void_p), ("adam_m", C.c_void_p), ("adam_v", C.c_void_p),
                ("replica", C.c_void_p)]


class LrSched(C.Structure):
    _fields_ = [("eta_max", C.c_double), ("eta_min", C.c_double), ("t_warmup", C.c_uint64), ("T", C.c_uint64)]


_vp = C.c_void_p
_u32p = C.POINTER(C.c_uint32)
_u64p = C.POINTER(C.c_uint64)
_f64p = C.POINTER(C.c_double)

# name -> (restype, argtypes): every function include/alsgd.h declares
SIGNATURES = {
    "alsgd_strerror": (C.c_char_p, [C.c_int]),
    "alsgd_layout_size": (C.c_int, [C.POINTER(TensorDesc), C.c_uint32, C.c_uint32, _u64p, _u64p]),
    "alsgd_arena_bytes": (C.c_int, [C.POINTER(TensorDesc), C.c_uint32, C.c_uint32, C.POINTER(Config), _u64p]),
    "alsgd_init": (C.c_int, [C.POINTER(_vp), C.POINTER(TensorDesc), C.c_uint32, C.c_uint32, C.POINTER(Config)]),
    "alsgd_destroy": (C.c_int, [_vp]),
    "alsgd_set_global": (C.c_int, [_vp, _vp, C.c_int]),
    "alsgd_get_global": (C.c_int, [_vp, _vp, C.c_int]),
    "alsgd_set_worker_params": (C.c_int, [_vp, C.c_uint32, _vp, C.c_int]),
    "alsgd_get_worker_params": (C.c_int, [_vp, C.c_uint32, _vp, C.c_int]),
    "alsgd_pull": (C.c_int, [_vp, C.c_uint32]),
    "alsgd_inner_adamw": (C.c_int, [_vp, C.c_uint32, _vp, C.c_int, C.c_uint64, C.c_float]),
    "alsgd_inner_adamw_bf16": (C.c_int, [_vp, C.c_uint32, _vp, C.c_int, C.c_uint64, C.c_float]),
    "alsgd_arrive": (C.c_int, [_vp, _u32p, C.c_uint32, C.c_uint32, C.POINTER(ArrivalInfo)]),
    "alsgd_arrive_ex": (C.c_int, [_vp, _u32p, C.c_uint32, C.c_uint32, C.POINTER(ArriveOpts), C.POINTER(ArrivalInfo)]),
    "alsgd_counters": (C.c_int, [_vp, _u64p, _u32p]),
    "alsgd_state_ptrs": (C.c_int, [_vp, C.POINTER(Ptrs)]),
    "alsgd_worker_state_ptrs": (C.c_int, [_vp, C.c_uint32, C.POINTER(WorkerPtrs)]),
    "alsgd_state_bytes": (C.c_int, [_vp, _u64p]),
    "alsgd_export_state": (C.c_int, [_vp, _vp, C.c_uint64]),
    "alsgd_import_state": (C.c_int, [_vp, _vp, C.c_uint64]),
    "alsgd_sync": (C.c_int, [_vp]),
    "alsgd_debug_word_ptr": (C.c_int, [_vp, C.POINTER(_vp)]),
    "alsgd_debug_guard_limit": (C.c_int, [_vp, C.c_uint64]),
    "alsgd_last_cuda_error": (C.c_int, [_vp]),
    "alsgd_dylu_steps": (C.c_int, [_f64p, C.c_uint32, C.c_uint32, _u32p]),
    "alsgd_shard_probs": (C.c_int, [_f64p, _f64p, C.c_uint32, _f64p]),
    "alsgd_lr_at": (C.c_int, [C.POINTER(LrSched), C.c_uint64, _f64p]),
    "alsgd_sched_create": (C.c_int, [C.POINTER(_vp), C.c_uint32, C.c_double, C.c_uint64]),
    "alsgd_sched_destroy": (C.c_int, [_vp]),
    "alsgd_sched_dispatch": (C.c_int, [_vp, C.c_uint32, C.c_double, C.c_uint32]),
    "alsgd_sched_next_batch": (C.c_int, [_vp, _u32p, _f64p, C.c_uint32, _u32p, _f64p]),
    "alsgd_sched_local_updates": (C.c_int, [_vp, _u64p]),
    "alsgd_sched_state_bytes": (C.c_int, [_vp, _u64p]),
    "alsgd_sched_export": (C.c_int, [_vp, _vp, C.c_uint64]),
    "alsgd_sched_import": (C.c_int, [_vp, _vp, C.c_uint64]),
    "alsgd_pg_norm_static": (C.c_int, [_vp, _vp, C.c_uint64, C.c_int32, _vp, _vp, _vp]),
}
STATIC_MAX_ELEMS = 1 << 27

_lib = None
_variant = "main"


def use_debug_library(on: bool = True):
    """Route every later call through libalsgd_dbg.so (kernels with bounds checks; alsgd_sync reports refused
    accesses) instead of libalsgd.so.  Must be chosen before the first call that loads a library."""
    global _variant
    want = "debug" if on else "main"
    if _lib is not None and want != _variant:
        raise RuntimeError("a library is already loaded in this process")
    _variant = want


class AlsgdError(RuntimeError):
    def __init__(self, status, where, cuda=0):
        self.status = status
        msg = f"{where}: status {status}"
        try:
            msg += f" ({lib().alsgd_strerror(status).decode()})"
        except Exception:
            pass
        if cuda:
            msg += f", cudaError {cuda}"
        super().__init__(msg)


def lib():
    """Load libalsgd.so (building it in-tree first if the sources are newer)."""
    global _lib
    if _lib is None:
        from . import build as _build
        if _build.needs_build(_variant):
            _build.build(targets=(_variant,))
        path = LIB_PATH if _variant == "main" else _build.LIB_DBG
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: the CUDA library is required, there is no fallback")
        L = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)      # AttributeError if the library does not export a declared symbol
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status, where, ctx=None):
    if status != OK:
        cuda = lib().alsgd_last_cuda_error(ctx) if ctx else 0
        raise AlsgdError(status, where, cuda)


def tensor_table(tensors):
    """ctypes array from an iterable of (numel, decay) pairs or objects with .numel / .decay."""
    items = [(t.numel, t.decay) if hasattr(t, "numel") else t for t in tensors]
    arr = (TensorDesc * len(items))()
    for i, (n, d) in enumerate(items):
        arr[i].numel, arr[i].flags = int(n), TENSOR_DECAY if d else 0
    return arr


def alsgd_layout_size(tensors, align_elems=128):
    tab = tensor_table(tensors)
    P = C.c_uint64()
    offs = (C.c_uint64 * len(tab))()
    _check(lib().alsgd_layout_size(tab, len(tab), align_elems, C.byref(P), offs), "alsgd_layout_size")
    return int(P.value), [int(x) for x in offs]


def alsgd_dylu_steps(speeds, H):
    sp = (C.c_double * len(speeds))(*[float(x) for x in speeds])
    out = (C.c_uint32 * len(speeds))()
    _check(lib().alsgd_dylu_steps(sp, len(speeds), int(H), out), "alsgd_dylu_steps")
    return [int(x) for x in out]


def alsgd_shard_probs(sizes, learned):
    n = len(sizes)
    s = (C.c_double * n)(*[float(x) for x in sizes])
    l = (C.c_double * n)(*[float(x) for x in learned])
    out = (C.c_double * n)()
    _check(lib().alsgd_shard_probs(s, l, n, out), "alsgd_shard_probs")
    return [float(x) for x in out]


def alsgd_lr_at(eta_max, eta_min, t_warmup, T, t):
    s = LrSched(float(eta_max), float(eta_min), int(t_warmup), int(T))
    out = C.c_double()
    _check(lib().alsgd_lr_at(C.byref(s), int(t), C.byref(out)), "alsgd_lr_at")
    return float(out.value)


class Scheduler:
    """alsgd_sched_*: Algorithm 2 / Algorithm 5 on faked time."""

    def __init__(self, n_workers, tau_grace, t_max=0):
        self._h = _vp()
        self.n = int(n_workers)
        _check(lib().alsgd_sched_create(C.byref(self._h), self.n, float(tau_grace), int(t_max)), "alsgd_sched_create")

    def dispatch(self, worker, duration, local_updates):
        _check(lib().alsgd_sched_dispatch(self._h, int(worker), float(duration), int(local_updates)), "alsgd_sched_dispatch")

    def next_batch(self):
        ids = (C.c_uint32 * self.n)()
        times = (C.c_double * self.n)()
        k = C.c_uint32()
        restart = C.c_double()
        _check(lib().alsgd_sched_next_batch(self._h, ids, times, self.n, C.byref(k), C.byref(restart)), "alsgd_sched_next_batch")
        return [int(ids[i]) for i in range(k.value)], [float(times[i]) for i in range(k.value)], float(restart.value)

    def local_updates(self):
        out = C.c_uint64()
        _check(lib().alsgd_sched_local_updates(self._h, C.byref(out)), "alsgd_sched_local_updates")
        return int(out.value)

    def export_state(self) -> bytes:
        n = C.c_uint64()
        _check(lib().alsgd_sched_state_bytes(self._h, C.byref(n)), "alsgd_sched_state_bytes")
        buf = C.create_string_buffer(int(n.value))
        _check(lib().alsgd_sched_export(self._h, buf, int(n.value)), "alsgd_sched_export")
        return buf.raw

    def import_state(self, image: bytes):
        _check(lib().alsgd_sched_import(self._h, image, len(image)), "alsgd_sched_import")

    def close(self):
        if self._h:
            lib().alsgd_sched_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Context:
    """One alsgd_ctx with a torch-owned arena on one CUDA device.  Method names follow the ABI."""

    def __init__(self, tensors, n_workers, N, beta, outer_lr, c=0.0, pg_base=PG_DISPATCH,
                 adam=(0.9, 0.95, 1e-8, 0.1), replica=True, grad_staging=False, align_elems=128,
                 device=0, stream=None, buffered=False, sgdm=False, stable_ptrs=False):
        import torch
        self.torch = torch
        if not torch.cuda.is_available():
            raise RuntimeError("alsgd needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self.tab = tensor_table(tensors)
        self.align = int(align_elems)
        self.P, self.offsets = alsgd_layout_size(tensors, self.align)
        cfg = Config()
        cfg.n_workers, cfg.N, cfg.pg_base = int(n_workers), int(N), int(pg_base)
        cfg.flags = ((CFG_REPLICA_BF16 if replica else 0) | (CFG_GRAD_STAGING if grad_staging else 0)
                     | (CFG_OUTER_BUFFERED if buffered else 0) | (CFG_OUTER_SGDM if sgdm else 0)
                     | (CFG_STABLE_PTRS if stable_ptrs else 0))
        cfg.beta, cfg.outer_lr, cfg.c = float(beta), float(outer_lr), float(c)
        cfg.adam_b1, cfg.adam_b2, cfg.adam_eps, cfg.adam_wd = [float(x) for x in adam]
        cfg.device = device
        nbytes = C.c_uint64()
        _check(lib().alsgd_arena_bytes(self.tab, len(self.tab), self.align, C.byref(cfg), C.byref(nbytes)), "alsgd_arena_bytes")
        self.arena_bytes = int(nbytes.value)
        with torch.cuda.device(self.device):
            self.arena = torch.empty(self.arena_bytes + 256, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        pad = (-self.arena.data_ptr()) % 256
        cfg.arena, cfg.arena_bytes = self.arena.data_ptr() + pad, self.arena_bytes
        cfg.stream = self.stream.cuda_stream
        self.cfg = cfg
        self.n_workers = int(n_workers)
        self._h = _vp()
        _check(lib().alsgd_init(C.byref(self._h), self.tab, len(self.tab), self.align, C.byref(cfg)), "alsgd_init")

    # -- views of borrowed device memory ---------------------------------------------------------
    def _view(self, ptr, dtype):
        if not ptr:
            return None
        torch = self.torch
        off = int(ptr) - self.arena.data_ptr()
        size = self.P * (2 if dtype in (torch.int16, torch.bfloat16) else 4)
        return self.arena[off:off + size].view(dtype)

    def alsgd_state_ptrs(self):
        """(theta, m, Delta) as fp32 torch views of the arena."""
        p = Ptrs()
        _check(lib().alsgd_state_ptrs(self._h, C.byref(p)), "alsgd_state_ptrs", self._h)
        f = self.torch.float32
        return self._view(p.theta, f), self._view(p.m, f), self._view(p.delta, f)

    def alsgd_worker_state_ptrs(self, w):
        """dict of torch views: p, base, adam_m, adam_v (fp32), replica (int16 bit patterns)."""
        p = WorkerPtrs()
        _check(lib().alsgd_worker_state_ptrs(self._h, int(w), C.byref(p)), "alsgd_worker_state_ptrs", self._h)
        f = self.torch.float32
        return {"p": self._view(p.p, f), "base": self._view(p.base, f), "adam_m": self._view(p.adam_m, f),
                "adam_v": self._view(p.adam_v, f), "replica": self._view(p.replica, self.torch.int16)}

    # -- the ABI calls ---------------------------------------------------------------------------------
    def _ptr(self, t):
        """(address, is_device) of a contiguous fp32 torch tensor or numpy array of P elements."""
        if hasattr(t, "data_ptr"):
            assert t.is_contiguous() and t.dtype == self.torch.float32 and t.numel() == self.P
            return t.data_ptr(), int(t.is_cuda)
        assert t.flags["C_CONTIGUOUS"] and t.dtype.name == "float32" and t.size == self.P
        return t.ctypes.data, 0

    def alsgd_set_global(self, src):
        a, d = self._ptr(src)
        _check(lib().alsgd_set_global(self._h, a, d), "alsgd_set_global", self._h)

    def alsgd_get_global(self, dst):
        a, d = self._ptr(dst)
        _check(lib().alsgd_get_global(self._h, a, d), "alsgd_get_global", self._h)

    def alsgd_set_worker_params(self, w, src):
        a, d = self._ptr(src)
        _check(lib().alsgd_set_worker_params(self._h, int(w), a, d), "alsgd_set_worker_params", self._h)

    def alsgd_get_worker_params(self, w, dst):
        a, d = self._ptr(dst)
        _check(lib().alsgd_get_worker_params(self._h, int(w), a, d), "alsgd_get_worker_params", self._h)

    def alsgd_pull(self, w):
        _check(lib().alsgd_pull(self._h, int(w)), "alsgd_pull", self._h)

    def alsgd_inner_adamw(self, w, grads, step, lr):
        a, d = self._ptr(grads)
        _check(lib().alsgd_inner_adamw(self._h, int(w), a, d, int(step), float(lr)), "alsgd_inner_adamw", self._h)

    @staticmethod
    def _infos(info, k):
        return [{"worker": int(i.worker), "tick": int(i.tick), "staleness": int(i.staleness),
                 "boundary": bool(i.boundary), "gnorm2": float(i.gnorm2), "nonfinite": int(i.nonfinite),
                 "dropped": bool(i.dropped)} for i in info[:k]]

    def alsgd_inner_adamw_bf16(self, w, grads, step, lr):
        """grads: contiguous torch tensor of P bf16 (or int16 bit patterns), on the device or pinned on the host."""
        assert grads.is_contiguous() and grads.numel() == self.P and grads.element_size() == 2
        _check(lib().alsgd_inner_adamw_bf16(self._h, int(w), grads.data_ptr(), int(grads.is_cuda), int(step), float(lr)),
               "alsgd_inner_adamw_bf16", self._h)

    def alsgd_arrive(self, worker_ids, flags=ARRIVE_RESEED, want_info=True):
        k = len(worker_ids)
        ids = (C.c_uint32 * max(k, 1))(*[int(x) for x in worker_ids])
        info = (ArrivalInfo * max(k, 1))() if want_info else None
        _check(lib().alsgd_arrive(self._h, ids, k, int(flags), info), "alsgd_arrive", self._h)
        return self._infos(info, k) if want_info else None

    def alsgd_arrive_ex(self, worker_ids, flags=ARRIVE_RESEED, weights=None, dc_lambda=0.0,
                        staleness_rule=STALE_NONE, stale_threshold=0, want_info=True):
        k = len(worker_ids)
        ids = (C.c_uint32 * max(k, 1))(*[int(x) for x in worker_ids])
        info = (ArrivalInfo * max(k, 1))() if want_info else None
        opts = ArriveOpts()
        wbuf = (C.c_float * max(k, 1))(*[float(x) for x in weights]) if weights is not None else None
        opts.weights = wbuf
        opts.dc_lambda, opts.staleness_rule, opts.stale_threshold = float(dc_lambda), int(staleness_rule), int(stale_threshold)
        _check(lib().alsgd_arrive_ex(self._h, ids, k, int(flags), C.byref(opts), info), "alsgd_arrive_ex", self._h)
        return self._infos(info, k) if want_info else None

    def alsgd_counters(self):
        t, ph = C.c_uint64(), C.c_uint32()
        _check(lib().alsgd_counters(self._h, C.byref(t), C.byref(ph)), "alsgd_counters", self._h)
        return int(t.value), int(ph.value)

    def alsgd_state_bytes(self):
        n = C.c_uint64()
        _check(lib().alsgd_state_bytes(self._h, C.byref(n)), "alsgd_state_bytes", self._h)
        return int(n.value)

    def alsgd_export_state(self):
        """The state image as a numpy uint8 array."""
        import numpy as np
        buf = np.empty(self.alsgd_state_bytes(), dtype=np.uint8)
        _check(lib().alsgd_export_state(self._h, buf.ctypes.data, buf.size), "alsgd_export_state", self._h)
        return buf

    def alsgd_import_state(self, image):
        assert image.dtype.name == "uint8" and image.flags["C_CONTIGUOUS"]
        _check(lib().alsgd_import_state(self._h, image.ctypes.data, image.size), "alsgd_import_state", self._h)

    def alsgd_sync(self):
        _check(lib().alsgd_sync(self._h), "alsgd_sync", self._h)

    def alsgd_debug_word_ptr(self):
        """Device address of the debug build's violation record (raises E_UNSUPPORTED on the normal build)."""
        out = _vp()
        _check(lib().alsgd_debug_word_ptr(self._h, C.byref(out)), "alsgd_debug_word_ptr", self._h)
        return int(out.value)

    def raw(self, name, *args):
        """Call an ABI function on this context and return its status without raising."""
        return getattr(lib(), name)(self._h, *args)

    def close(self):
        if self._h:
            lib().alsgd_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
