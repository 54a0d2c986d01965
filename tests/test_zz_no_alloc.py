"""The allocation-free diagnostics entry point against the regular one.

alsgd_pg_norm_static exists for embedders that cannot get device memory of their own (code living
inside another framework's memory plan, or a process whose memory was all handed out at start-up):
its working memory is a fixed array inside the library.  This file checks, through the C ABI, that it
reports the same squared pseudo-gradient norm and non-finite flag as alsgd_arrive does with its
NORM | NANCHECK flags, on two calls in a row (the second call sees the array as the first left it),
and that it refuses vectors larger than its fixed working memory.  The file name sorts last so that a
run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2401_09135_b200 import binding as B
from paper_2401_09135_b200 import synth

pytestmark = pytest.mark.gpu


def static_norm(start, p, n, out_norm, out_flag):
    return B.lib().alsgd_pg_norm_static(start.data_ptr(), p.data_ptr(), n, 0,
                                        torch.cuda.current_stream().cuda_stream,
                                        out_norm.data_ptr(), out_flag.data_ptr())


@pytest.mark.parametrize("P", [4096 * 5 + 1237, 1 << 20])
def test_static_entry_point_matches_arrive_diagnostics_twice(P):
    tensors = synth.flat_tensors(P)
    ctx = B.Context(tensors, 2, 4, 0.9, 0.7, align_elems=1)
    ctx.alsgd_set_global(synth.theta0(tensors, ctx.offsets, ctx.P, synth.SEED))
    out_norm = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    out_flag = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    for call, w in enumerate((0, 1)):
        ctx.alsgd_pull(w)
        z = synth.normal_vec(ctx.P, 1e-3 * (call + 1), synth.SEED, synth.STREAM_DELTA, sub=call)
        if call == 1:
            z[ctx.P // 2] = np.inf                  # second call: poisoned worker, flag must flip to 1
        v = ctx.alsgd_worker_state_ptrs(w)
        v["p"].sub_(torch.from_numpy(z).cuda())
        assert static_norm(v["base"], v["p"], ctx.P, out_norm, out_flag) == B.OK
        repeat = torch.empty_like(out_norm)
        assert static_norm(v["base"], v["p"], ctx.P, repeat, out_flag) == B.OK
        o_norm, o_flag = oracle.pg_norm2(v["base"].cpu().numpy(), v["base"].cpu().numpy(), v["p"].cpu().numpy())
        info = ctx.alsgd_arrive([w], B.ARRIVE_NORM | B.ARRIVE_NANCHECK)[0]
        torch.cuda.synchronize()
        assert int(out_flag.item()) == info["nonfinite"] == o_flag == call
        if call == 0:
            got, ref = float(out_norm.item()), info["gnorm2"]
            assert ref > 0 and abs(got - ref) <= 1e-6 * ref          # same tolerance as the norm parity tests
            assert abs(got - o_norm) <= 1e-6 * o_norm                # and directly against the CPU oracle's double sum
            assert float(repeat.item()) == got                       # fixed summation order: same bits
    ctx.close()


def test_static_entry_point_limits_and_arguments():
    x = torch.zeros(4096, dtype=torch.float32, device="cuda")
    n64 = torch.zeros(1, dtype=torch.float64, device="cuda")
    f32 = torch.zeros(1, dtype=torch.int32, device="cuda")
    L = B.lib()
    s = torch.cuda.current_stream().cuda_stream
    too_big = B.STATIC_MAX_ELEMS + 1                                  # refused before anything is read
    assert L.alsgd_pg_norm_static(x.data_ptr(), x.data_ptr(), too_big, 0, s, n64.data_ptr(), f32.data_ptr()) == B.E_NOMEM
    assert L.alsgd_pg_norm_static(x.data_ptr(), x.data_ptr(), 0, 0, s, n64.data_ptr(), f32.data_ptr()) == B.E_ARG
    assert L.alsgd_pg_norm_static(None, x.data_ptr(), 16, 0, s, n64.data_ptr(), f32.data_ptr()) == B.E_ARG
    assert L.alsgd_pg_norm_static(x.data_ptr() + 4, x.data_ptr(), 16, 0, s, n64.data_ptr(), f32.data_ptr()) == B.E_ARG
    assert L.alsgd_pg_norm_static(x.data_ptr(), x.data_ptr(), 16, 64, s, n64.data_ptr(), f32.data_ptr()) == B.E_RANGE
    assert L.alsgd_pg_norm_static(x.data_ptr(), x.data_ptr(), 4096, 0, s, n64.data_ptr(), f32.data_ptr()) == B.OK
    torch.cuda.synchronize()
    assert float(n64.item()) == 0.0 and int(f32.item()) == 0


@pytest.mark.parametrize("n", [B.STATIC_MAX_ELEMS, B.STATIC_MAX_ELEMS - 3])
def test_static_entry_point_at_its_size_limit(n):
    """The largest accepted vector uses every slot of the fixed working memory (n = limit), and limit - 3 ends in a
    ragged tile.  Every pseudo-gradient entry is +-2^-10, so the exact sum is n * 2^-20 and every partial sum is
    exact in double: the result must match to the last bit.  1 GiB of inputs."""
    free, _ = torch.cuda.mem_get_info()
    if free < 3 * (1 << 30):
        pytest.skip("needs 3 GiB of free device memory")
    start = torch.ones(n, dtype=torch.float32, device="cuda")
    p = torch.ones(n, dtype=torch.float32, device="cuda")
    p[0::2] += 2.0 ** -10
    p[1::2] -= 2.0 ** -10
    out_norm = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    out_flag = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    for _ in range(2):
        assert static_norm(start, p, n, out_norm, out_flag) == B.OK
        torch.cuda.synchronize()
        assert float(out_norm.item()) == n * 2.0 ** -20 and int(out_flag.item()) == 0
    # the oracle on the last ragged tile plus a sampled stretch agrees with the per-element value
    lo = n - 5000
    o_norm, o_flag = oracle.pg_norm2(start[lo:].cpu().numpy(), start[lo:].cpu().numpy(), p[lo:].cpu().numpy())
    assert o_norm == 5000 * 2.0 ** -20 and o_flag == 0
    p[n - 1] = float("nan")                                            # the very last element, in the last tile
    assert static_norm(start, p, n, out_norm, out_flag) == B.OK
    torch.cuda.synchronize()
    assert int(out_flag.item()) == 1
    del start, p
    torch.cuda.empty_cache()
