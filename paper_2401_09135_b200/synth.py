"""Seeded synthetic inputs shared by the CUDA path's tests/bench and by the CPU oracle's tests.

This module holds input *recipes* only: tensor lists shaped like the paper's decoder-only
transformers (Table 6: layers / hidden width / 32 000-token vocabulary), random vectors, worker
perturbations, job durations and arrival orders.  None of the method's arithmetic (Algorithm 3,
AdamW, bf16 rounding, Eq. 6, Algorithm 2) lives here, and the module imports neither the CUDA
binding nor the oracle.  Every random number comes from numpy's Philox counter-based generator
keyed by ``(seed, stream)``, so the same call gives the same bytes on every machine.

Streams: 0 = initial global parameters, 1 = worker perturbations, 2 = gradients,
3 = job-duration jitter, 4 = staleness draws, 5 = arrival-order draws, 6 = per-tensor scales.
"""
from __future__ import annotations

from collections import namedtuple

import numpy as np

SEED = 20240109

STREAM_THETA0 = 0
STREAM_DELTA = 1
STREAM_GRAD = 2
STREAM_JITTER = 3
STREAM_STALENESS = 4
STREAM_ORDER = 5
STREAM_SCALE = 6

#: kind is "matrix" (weight-decayed, N(0, 0.02^2) init), "gain" (init 1) or "bias" (init 0).
Tensor = namedtuple("Tensor", ["name", "numel", "decay", "kind"])


def rng(seed: int, stream: int, sub: int = 0) -> np.random.Generator:
    """Counter-based generator for one (seed, stream, sub-stream) triple."""
    return np.random.Generator(np.random.Philox(key=[(int(seed) << 8) ^ int(sub) & 0xFFFFFFFF, int(stream)]))


def flat_tensors(P: int):
    """One undifferentiated weight vector of P elements (the small flat-vector configuration)."""
    return [Tensor("flat", int(P), True, "matrix")]


def transformer_tensors(vocab: int, d_model: int, d_ff: int, n_layers: int):
    """Tensor list of a decoder-only transformer with a tied embedding, no linear biases, no
    positional table and LayerNorm gain+bias, in flat-buffer order.  Matrices are weight-decayed,
    gains and biases are not."""
    t = [Tensor("tok_emb", vocab * d_model, True, "matrix")]
    for l in range(n_layers):
        t.append(Tensor(f"l{l}.ln1.g", d_model, False, "gain"))
        t.append(Tensor(f"l{l}.ln1.b", d_model, False, "bias"))
        for w in ("wq", "wk", "wv", "wo"):
            t.append(Tensor(f"l{l}.{w}", d_model * d_model, True, "matrix"))
        t.append(Tensor(f"l{l}.ln2.g", d_model, False, "gain"))
        t.append(Tensor(f"l{l}.ln2.b", d_model, False, "bias"))
        t.append(Tensor(f"l{l}.w_ff1", d_model * d_ff, True, "matrix"))
        t.append(Tensor(f"l{l}.w_ff2", d_ff * d_model, True, "matrix"))
    t.append(Tensor("lnf.g", d_model, False, "gain"))
    t.append(Tensor("lnf.b", d_model, False, "bias"))
    return t


def paper_tensors(vocab: int, hidden: int, n_heads: int, kv_size: int, n_layers: int, ff_mult: int = 4):
    """Tensor list with the numbers of the paper's Table 6 (layers, hidden dim, heads, K/V size, vocab):
    attention width n_heads * kv_size (which differs from the hidden dim for the 60M / 150M models),
    feed-forward width ff_mult * hidden, tied embedding, LayerNorm gain+bias, no linear biases."""
    d_attn = n_heads * kv_size
    t = [Tensor("tok_emb", vocab * hidden, True, "matrix")]
    for l in range(n_layers):
        t.append(Tensor(f"l{l}.ln1.g", hidden, False, "gain"))
        t.append(Tensor(f"l{l}.ln1.b", hidden, False, "bias"))
        for w in ("wq", "wk", "wv"):
            t.append(Tensor(f"l{l}.{w}", hidden * d_attn, True, "matrix"))
        t.append(Tensor(f"l{l}.wo", d_attn * hidden, True, "matrix"))
        t.append(Tensor(f"l{l}.ln2.g", hidden, False, "gain"))
        t.append(Tensor(f"l{l}.ln2.b", hidden, False, "bias"))
        t.append(Tensor(f"l{l}.w_ff1", hidden * ff_mult * hidden, True, "matrix"))
        t.append(Tensor(f"l{l}.w_ff2", ff_mult * hidden * hidden, True, "matrix"))
    t.append(Tensor("lnf.g", hidden, False, "gain"))
    t.append(Tensor("lnf.b", hidden, False, "bias"))
    return t


def layout_paper_60m():
    """Table 6, 60M column: 3 layers, hidden 896, 16 heads of size 64, vocab 32000 (~59M elements)."""
    return paper_tensors(32000, 896, 16, 64, 3)


def layout_paper_150m():
    """Table 6, 150M column: 12 layers, hidden 896, 16 heads of size 64, vocab 32000 (~150M elements)."""
    return paper_tensors(32000, 896, 16, 64, 12)


def layout_23m():
    """~23M-parameter layout: 6 layers, d_model 384, d_ff 1536, vocab 32000 (22 914 816 elements)."""
    return transformer_tensors(32000, 384, 1536, 6)


def layout_110m():
    """~110M-parameter layout: 12 layers, d_model 768, d_ff 3072, vocab 32000 (109 549 056 elements)."""
    return transformer_tensors(32000, 768, 3072, 12)


def ragged_tensors():
    """A small layout whose tensor sizes are not multiples of any vector width, with decayed and
    undecayed tensors interleaved; used to exercise padding, tails and segment edges."""
    sizes = [(1037, True), (5, False), (3, False), (4099, True), (1, False), (257, True), (130, False), (7001, True)]
    return [Tensor(f"r{i}", n, d, "matrix" if d else "gain") for i, (n, d) in enumerate(sizes)]


def theta0(tensors, offsets, P: int, seed: int = SEED) -> np.ndarray:
    """Initial global parameters: matrices N(0, 0.02^2), gains 1, biases 0, padding 0."""
    out = np.zeros(int(P), dtype=np.float32)
    g = rng(seed, STREAM_THETA0)
    for t, off in zip(tensors, offsets):
        off = int(off)
        if t.kind == "matrix":
            out[off:off + t.numel] = g.standard_normal(t.numel, dtype=np.float32) * np.float32(0.02)
        elif t.kind == "gain":
            out[off:off + t.numel] = 1.0
    return out


def normal_vec(n: int, std: float, seed: int, stream: int, sub: int = 0) -> np.ndarray:
    """n float32 draws from N(0, std^2)."""
    return rng(seed, stream, sub).standard_normal(int(n), dtype=np.float32) * np.float32(std)


def zero_padding(vec: np.ndarray, tensors, offsets) -> np.ndarray:
    """Zero every element of a flat vector that lies in alignment padding between tensors."""
    mask = np.zeros(vec.shape[0], dtype=bool)
    for t, off in zip(tensors, offsets):
        mask[int(off):int(off) + t.numel] = True
    vec[~mask] = 0.0
    return vec


def round_robin_order(n_workers: int, n_arrivals: int, seed: int = SEED):
    """Round-robin arrival order whose first worker and direction come from the seed."""
    g = rng(seed, STREAM_ORDER)
    start = int(g.integers(0, n_workers))
    step = 1 if int(g.integers(0, 2)) == 0 else -1
    return [(start + step * i) % n_workers for i in range(n_arrivals)]


def job_durations(speeds, steps, n_rounds: int, seed: int = SEED, amp: float = 0.05) -> np.ndarray:
    """Faked training time of every job: durations[w, r] = steps[w] / speeds[w] * (1 + amp*u) with
    u ~ U[-1, 1) seeded.  Stands in for the paper's real-world device statistics (not published)."""
    W = len(speeds)
    u = rng(seed, STREAM_JITTER).uniform(-1.0, 1.0, size=(W, n_rounds))
    base = np.asarray(steps, dtype=np.float64) / np.asarray(speeds, dtype=np.float64)
    return base[:, None] * (1.0 + amp * u)


def staleness_batches(n_workers: int, k: int, n_batches: int, max_stale: int = 15, seed: int = SEED):
    """Arrival batches whose order realises a random staleness: at each (re)start a worker draws
    s ~ U{0..max_stale} and becomes due at (tick of that start) + s; each batch is the k workers
    with the smallest (due, id), in that order, and all k restart when the batch has been applied
    (the server tick advances by one per arrival)."""
    g = rng(seed, STREAM_STALENESS)
    due = [(int(g.integers(0, max_stale + 1)), w) for w in range(n_workers)]
    tick = 0
    out = []
    for _ in range(n_batches):
        due.sort()
        batch = [w for _, w in due[:k]]
        rest = due[k:]
        tick += k
        due = rest + [(tick + int(g.integers(0, max_stale + 1)), w) for w in batch]
        out.append(batch)
    return out


def lognormal_tensor_scales(n_tensors: int, visit: int, mu: float = -7.0, sigma: float = 1.0, seed: int = SEED):
    """One perturbation magnitude per tensor for one worker visit: exp(N(mu, sigma^2))."""
    z = rng(seed, STREAM_SCALE, visit).standard_normal(n_tensors)
    return np.exp(mu + sigma * z)


def per_element_scale(tensors, offsets, P: int, scales) -> np.ndarray:
    """Expand one scale per tensor to a flat float32 vector (0 in padding)."""
    out = np.zeros(int(P), dtype=np.float32)
    for t, off, s in zip(tensors, offsets, scales):
        out[int(off):int(off) + t.numel] = np.float32(s)
    return out


def grad_pool_index(worker: int, step: int, pool: int) -> int:
    """Which pre-generated gradient vector a worker uses at a given lifetime step."""
    h = (worker * 0x9E3779B1 + step * 0x85EBCA77) & 0xFFFFFFFF
    h ^= h >> 15
    h = (h * 0x2C1B3C6D) & 0xFFFFFFFF
    h ^= h >> 12
    return h % pool
