"""The debug build of the library (libalsgd_dbg.so, -DALSGD_DEBUG_BOUNDS): its kernels check every access to an
arena-owned vector against the arena's byte range and alignment, skip and record what falls outside, and
alsgd_sync returns the record as ALSGD_E_BOUNDS.  A process can load only one build, so the cases run in a child
process (tests/debug_bounds_child.py): parity cases with ragged sizes, scalar tails and a batch split over
launches must record nothing; the status must follow the record; and with the accepted range narrowed to exclude
one slice, exactly the accesses to that slice must be refused, recorded and not performed."""
import os
import subprocess
import sys

import pytest

from paper_2401_09135_b200 import binding as B

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.mark.gpu
def test_debug_build_records_refused_accesses_and_stays_silent_on_clean_runs():
    r = subprocess.run([sys.executable, os.path.join(HERE, "debug_bounds_child.py")], capture_output=True, text=True,
                       timeout=900)
    assert r.returncode == 0 and "DEBUG-BOUNDS-OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


@pytest.mark.gpu
def test_normal_build_has_no_debug_hooks():
    from paper_2401_09135_b200 import synth
    ctx = B.Context(synth.flat_tensors(256), 1, 1, 0.9, 0.7)
    import ctypes as C
    out = C.c_void_p(1)
    assert ctx.raw("alsgd_debug_word_ptr", C.byref(out)) == B.E_UNSUPPORTED and not out.value
    assert ctx.raw("alsgd_debug_guard_limit", 0) == B.E_UNSUPPORTED
    ctx.close()


def test_debug_library_exports_the_same_symbols():
    import ctypes as C
    from paper_2401_09135_b200 import build
    if build.needs_build("debug"):
        build.build(targets=("debug",))
    L = C.CDLL(build.LIB_DBG)
    for name in B.SIGNATURES:
        assert hasattr(L, name), name
