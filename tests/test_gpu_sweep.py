"""The launch-shape benchmark library (include/alsgd_sweep.h): every shape of a kernel body computes the same
bits.  Results must not depend on threads per block, vectors per thread, resident-block caps, persistent loops
or on whether operands move through registers or through bulk copies into shared memory; the packed-arithmetic
shapes are the documented exception (benchmark only) and are left out."""
import ctypes as C

import pytest
import torch

from paper_2401_09135_b200 import sweep


def test_sweep_library_loads_and_describes_its_variants():
    vs = sweep.variants()
    assert len(vs) > 100
    assert {v["kind"] for v in vs} == {sweep.KIND_ADAMW, sweep.KIND_ARRIVE}
    assert any(v["staged"] for v in vs) and any(v["persistent"] for v in vs) and any(v["diag"] for v in vs)
    bad = sweep.Variant()
    assert sweep.lib().alsgd_sweep_describe(len(vs), C.byref(bad)) == -1
    assert sweep.lib().alsgd_sweep_launch(0, None, 0, None) != 0


def _buffers(n, seed):
    dev = torch.device("cuda")
    g = torch.Generator(device=dev).manual_seed(seed)
    r = lambda s: torch.randn(n, device=dev, generator=g) * s
    t = {"theta": r(0.02), "delta": r(1e-3), "mom": r(1e-3), "snapshot": torch.zeros(n, device=dev),
         "adam_p": r(0.02), "adam_m": r(1e-3), "adam_v": torch.rand(n, device=dev, generator=g) * 1e-5, "adam_g": r(0.01),
         "adam_rep": torch.zeros(n, device=dev, dtype=torch.int16)}
    for j in range(8):
        t[f"p{j}"], t[f"base{j}"] = r(0.02), r(0.02)
        t[f"rep{j}"] = torch.zeros(n, device=dev, dtype=torch.int16)
    t["seg_end"] = torch.tensor([1000, 5000, 5001, n // 2 + 3, n], device=dev, dtype=torch.int64)
    t["seg_decay"] = torch.tensor([1, 0, 1, 0, 1], device=dev, dtype=torch.int32)
    t["diag_scratch"] = torch.zeros(8 * (n // 256 + 66), device=dev, dtype=torch.float64)
    t["diag_out"] = torch.zeros(8, device=dev, dtype=torch.float64)
    t["diag_flags"] = torch.zeros(8, device=dev, dtype=torch.int32)
    t["diag_state"] = torch.zeros(16, device=dev, dtype=torch.int32)
    b = sweep.Buffers()
    b.n = n
    for name in ("theta", "delta", "mom", "snapshot", "adam_p", "adam_m", "adam_v", "adam_g", "adam_rep", "seg_end",
                 "seg_decay", "diag_scratch", "diag_out", "diag_flags", "diag_state"):
        setattr(b, name, t[name].data_ptr())
    for j in range(8):
        b.p[j], b.base[j], b.rep[j] = t[f"p{j}"].data_ptr(), t[f"base{j}"].data_ptr(), t[f"rep{j}"].data_ptr()
    b.n_seg = 5
    return t, b


def _bits(x):
    return x.view(torch.int32) if x.dtype == torch.float32 else x


@pytest.mark.gpu
def test_every_adamw_shape_gives_the_same_bits():
    n = 2 * 1024 * 1024 + 1536                     # ragged last tile for every tile size; a multiple of 8
    L = sweep.lib()
    stream = torch.cuda.current_stream().cuda_stream
    ref = None
    for v in sweep.variants():
        if v["kind"] != sweep.KIND_ADAMW:
            continue
        t, b = _buffers(n, 5)
        assert L.alsgd_sweep_launch(v["index"], C.byref(b), 0, stream) == 0
        torch.cuda.synchronize()
        assert int(t["diag_flags"][7].item()) == 0, f"a bounded wait ran out in {v}"
        out = [_bits(t[k]).clone() for k in ("adam_p", "adam_m", "adam_v", "adam_rep")]
        if ref is None:
            ref = out
        else:
            assert all(torch.equal(a, r) for a, r in zip(out, ref)), v


@pytest.mark.gpu
@pytest.mark.parametrize("phase", [sweep.PHASE_MIDDLE, sweep.PHASE_CYCLE])
def test_every_arrival_shape_gives_the_same_bits(phase):
    n = 512 * 1024 + 3                             # scalar tail
    L = sweep.lib()
    stream = torch.cuda.current_stream().cuda_stream
    ref = {}
    for v in sweep.variants():
        if v["kind"] != sweep.KIND_ARRIVE or v["packed"]:
            continue
        t, b = _buffers(n, 6)
        assert L.alsgd_sweep_launch(v["index"], C.byref(b), phase, stream) == 0
        torch.cuda.synchronize()
        K = v["K"]
        out = [_bits(t[k]).clone() for k in ["theta", "delta", "mom", "snapshot"] + [f"rep{j}" for j in range(K)]]
        key = (K, v["base_mode"])
        if key not in ref:
            ref[key] = (out, None)
        assert all(torch.equal(a, r) for a, r in zip(out, ref[key][0])), v
        if v["diag"]:                               # the norms agree across shapes to rounding of the partial sums
            norms = t["diag_out"][:K].clone()
            if ref[key][1] is None:
                ref[key] = (ref[key][0], norms)
            assert torch.allclose(norms, ref[key][1], rtol=1e-6, atol=0.0), v
            assert not t["diag_flags"][:K].any() and not t["diag_state"].any()
    assert len(ref) >= 7
