"""Drives the CUDA library (through the C-ABI binding) and the CPU oracle with the same seeded inputs
and compares them element by element.

Every step of the path is elementwise over the flat index, so at sizes where the oracle would take
minutes it runs on a sorted sample of indices (random picks plus every tensor's first and last
elements): the library processes the full vectors, the oracle processes the gathered sub-vectors,
and the comparison covers exactly the sampled positions.
"""
import numpy as np
import torch

import oracle
from paper_2401_09135_b200 import binding as B

RTOL = 2e-6          # stated bar: max |err| <= 2e-6 * max(1, |ref|) per fp32 element


def sample_indices(tensors, offsets, P, n_random, seed=1234):
    """Sorted unique sample: n_random uniform picks + 8 elements at both ends of every tensor + the tail of P."""
    r = np.random.default_rng(seed)
    parts = [r.integers(0, P, size=n_random, dtype=np.int64)]
    for t, off in zip(tensors, offsets):
        lo, hi = int(off), int(off) + t.numel
        parts.append(np.arange(lo, min(lo + 8, hi), dtype=np.int64))
        parts.append(np.arange(max(hi - 8, lo), hi, dtype=np.int64))
    parts.append(np.arange(max(P - 16, 0), P, dtype=np.int64))
    return np.unique(np.concatenate(parts))


def assert_fp32(name, got, ref, strict=True):
    got = np.asarray(got, dtype=np.float32)
    ref = np.asarray(ref, dtype=np.float32)
    assert got.shape == ref.shape, name
    with np.errstate(invalid="ignore"):
        err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
        tol = RTOL * np.maximum(1.0, np.abs(ref.astype(np.float64)))
        bad = ~((err <= tol) | (np.isnan(got) & np.isnan(ref)) | (got == ref))
    assert not bad.any(), f"{name}: {int(bad.sum())} elements beyond 2e-6*max(1,|ref|); worst {np.nanmax(err):.3e}"
    if strict:
        # The two sides perform the same IEEE operations in the same order, so they agree bit for bit.
        # (NaN payload and sign are not part of the contract: any NaN matches any NaN.)
        same = (got.view(np.uint32) == ref.view(np.uint32)) | (np.isnan(got) & np.isnan(ref))
        assert same.all(), f"{name}: {int((~same).sum())} elements differ in their bits"


class Pair:
    def __init__(self, tensors, n_workers, N, beta, outer_lr, c=0.0, pg_current=False, replica=True,
                 adam=(0.9, 0.95, 1e-8, 0.1), align=128, n_sample=None, grad_staging=False, strict=True,
                 buffered=False, sgdm=False, stable_ptrs=False):
        self.tensors = tensors
        self.W = n_workers
        self.strict = strict
        self.ctx = B.Context(tensors, n_workers, N, beta, outer_lr, c=c,
                             pg_base=B.PG_CURRENT if pg_current else B.PG_DISPATCH, adam=adam, replica=replica,
                             grad_staging=grad_staging, align_elems=align, buffered=buffered, sgdm=sgdm,
                             stable_ptrs=stable_ptrs)
        self.buffered = oracle.OUTER_SGDM if sgdm else (oracle.OUTER_BUFFERED if buffered else oracle.OUTER_DN)
        self.P, self.offsets = self.ctx.P, self.ctx.offsets
        o_offs, o_P = oracle.layout_offsets([t.numel for t in tensors], align)
        assert (o_P, o_offs) == (self.P, self.offsets)
        mask = oracle.decay_mask([t.numel for t in tensors], [t.decay for t in tensors], o_offs, o_P)
        if n_sample is None or n_sample >= self.P:
            self.idx = None
            n = self.P
        else:
            self.idx = sample_indices(tensors, self.offsets, self.P, n_sample)
            self.idx_dev = torch.from_numpy(self.idx).cuda()
            mask = mask[self.idx]
            n = self.idx.shape[0]
        self.orc = oracle.OracleServer(n, n_workers, N, beta, outer_lr, c=c, pg_current=pg_current,
                                       decay=np.ascontiguousarray(mask), adam=adam, replica=replica)
        self.pg_current = pg_current

    # -- sampling ---------------------------------------------------------------------------------
    def take(self, full_np):
        return np.ascontiguousarray(full_np if self.idx is None else full_np[self.idx])

    def fetch(self, dev_tensor):
        t = dev_tensor if self.idx is None else dev_tensor[self.idx_dev]
        return t.cpu().numpy()

    # -- mirrored calls ----------------------------------------------------------------------------
    def set_global(self, theta0_np):
        self.ctx.alsgd_set_global(theta0_np)
        self.orc.set_global(self.take(theta0_np))

    def pull(self, w):
        self.ctx.alsgd_pull(w)
        self.orc.pull(w)

    def perturb(self, w, z_dev, z_np, scale_dev=None, scale_np=None):
        """p_w <- p_w - scale*z : the stand-in for a round of local training (test harness arithmetic,
        one IEEE multiply and one IEEE subtract per element on both sides)."""
        p = self.ctx.alsgd_worker_state_ptrs(w)["p"]
        zs = self.take(z_np)
        if scale_dev is not None:
            p.sub_(scale_dev * z_dev)
            self.orc.p[w] -= self.take(scale_np) * zs
        else:
            p.sub_(z_dev)
            self.orc.p[w] -= zs

    def inner_adamw(self, w, g_dev, g_np, step, lr):
        self.ctx.alsgd_inner_adamw(w, g_dev, step, lr)
        self.orc.inner_adamw(w, self.take(g_np), step, lr)

    def arrive(self, ids, reseed=True, norm=False, weights=None, dc_lambda=0.0, poly=False, stale_threshold=None):
        flags = (B.ARRIVE_RESEED if reseed else 0) | ((B.ARRIVE_NORM | B.ARRIVE_NANCHECK) if norm else 0)
        plain = weights is None and dc_lambda == 0.0 and not poly
        if plain:
            got = self.ctx.alsgd_arrive(ids, flags)
        else:
            rule = B.STALE_NONE if not poly else (B.STALE_POLY if stale_threshold is None else B.STALE_POLY_THRES)
            got = self.ctx.alsgd_arrive_ex(ids, flags, weights=weights, dc_lambda=dc_lambda, staleness_rule=rule,
                                           stale_threshold=stale_threshold or 0)
        w32 = None if weights is None else [float(np.float32(x)) for x in weights]
        ref = self.orc.arrive(ids, reseed_after=reseed, norm=norm and self.idx is None, weights=w32,
                              dc_lambda=float(np.float32(dc_lambda)), buffered=self.buffered, poly=poly,
                              stale_threshold=stale_threshold)
        for g, r in zip(got, ref):                 # bookkeeping: bit-exact
            assert g["worker"] == r["worker"] and g["tick"] == r["tick"]
            assert g["boundary"] == r["boundary"] and g["staleness"] == r["staleness"]
            assert g["dropped"] == r["dropped"]
            if norm and self.idx is None:
                assert g["nonfinite"] == r["nonfinite"]
                if not r["nonfinite"]:
                    # the library accumulates squares in binary32 per thread before widening: entries beyond
                    # 1.8e19 in magnitude overflow that partial, and the documented result is then +inf
                    if r["gnorm2"] >= 1e37 and np.isinf(g["gnorm2"]):
                        continue
                    assert abs(g["gnorm2"] - r["gnorm2"]) <= 1e-6 * max(r["gnorm2"], 1e-30)
        return got

    # -- comparison ---------------------------------------------------------------------------------
    def check_server(self, where=""):
        theta, m, delta = self.ctx.alsgd_state_ptrs()
        self.ctx.alsgd_sync()
        assert_fp32(f"theta {where}", self.fetch(theta), self.orc.theta, self.strict)
        assert_fp32(f"m {where}", self.fetch(m), self.orc.m, self.strict)
        assert_fp32(f"Delta {where}", self.fetch(delta), self.orc.Delta, self.strict)
        t, phase = self.ctx.alsgd_counters()
        assert t == self.orc.t and phase == self.orc.t % self.orc.N

    def check_worker(self, w, where=""):
        v = self.ctx.alsgd_worker_state_ptrs(w)
        self.ctx.alsgd_sync()
        assert_fp32(f"p[{w}] {where}", self.fetch(v["p"]), self.orc.p[w], self.strict)
        assert_fp32(f"adam_m[{w}] {where}", self.fetch(v["adam_m"]), self.orc.am[w], self.strict)
        assert_fp32(f"adam_v[{w}] {where}", self.fetch(v["adam_v"]), self.orc.av[w], self.strict)
        if v["base"] is not None:
            assert_fp32(f"base[{w}] {where}", self.fetch(v["base"]), self.orc.base[w], self.strict)
        if v["replica"] is not None:
            got = self.fetch(v["replica"]).view(np.uint16)
            ref = self.orc.replica[w]
            nan = np.isnan(self.orc.p[w])            # a NaN's sign is not part of the contract
            assert np.array_equal(got[~nan], ref[~nan]), f"bf16 replica[{w}] {where}: bits differ"
            assert np.all((got[nan] & 0x7FFF) == 0x7FC0)

    def check_all(self, where=""):
        self.check_server(where)
        for w in range(self.W):
            self.check_worker(w, where)

    def close(self):
        self.ctx.close()
