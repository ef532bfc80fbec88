"""llvq_gemv_static, the entry point for callers that cannot allocate device memory (a process whose
pool owns the GPU, a plug-in without an allocator, code inside a stream capture): it must give what
llvq_gemv gives, call after call, with nothing but the caller's buffers and the library's built-in
scratch.  Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from helpers import GAIN, TOL_NORMALISED, make_case

pytestmark = pytest.mark.gpu


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    from paper_2609_02652_b200 import binding as B

    B.load()
    torch.cuda.set_device(0)
    ctx = B.create(0)
    try:
        # two different shapes back to back: the second call finds the shared scratch as the first left it
        for rows, k, seed in [(1000, 2560, 31), (4096, 4096, 32), (1000, 2560, 31)]:
            case = make_case(rows, k, seed=seed)
            buf = B.expand(ctx, B.PLANES, case.d_codes, rows, case.nb)
            ref = B.gemv(ctx, B.PLANES, buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24)
            for _ in range(2):
                y = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
                B.gemv_static(buf, case.d_scale, GAIN, case.d_x, rows, case.nb * 24, y)
                torch.cuda.synchronize()
                yv, rv = y.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
                assert np.isfinite(yv).all()
                # same tolerance as the parity tests, relative to ||W_row|| ||x||; ||W_row|| = r * sqrt(sum gain^2) >= r * 0.75 * sqrt(nb)
                bound = case.row_scale.astype(np.float64) * 0.75 * np.sqrt(case.nb) * np.linalg.norm(case.x.astype(np.float64))
                assert (np.abs(yv - rv) <= TOL_NORMALISED * bound + 1e-30).all()
                assert torch.equal(y, ref)          # same kernel, order-free reduction: in fact identical
        # more rows than the built-in scratch holds: a clear error, nothing launched
        rows = 65536 + 32
        dummy = torch.zeros(B.layout_bytes(B.PLANES, rows, 24), dtype=torch.uint8, device="cuda")
        sc = torch.zeros(rows, dtype=torch.float16, device="cuda")
        xx = torch.zeros(24, dtype=torch.float16, device="cuda")
        yy = torch.zeros(rows, dtype=torch.float32, device="cuda")
        with pytest.raises(B.LlvqError) as e:
            B.gemv_static(dummy, sc, GAIN, xx, rows, 24, yy)
        assert e.value.code == -3
        # exactly the maximum is accepted
        rows = 65536
        B.gemv_static(dummy[: B.layout_bytes(B.PLANES, rows, 24)], sc[:rows], GAIN, xx, rows, 24, yy[:rows])
        torch.cuda.synchronize()
        assert (yy[:rows] == 0).all()
        # none of those launches gave up on a wait: the built-in flag is clear
        B.static_status()
        # ... and the calls after the first allocated nothing on the device: the free memory is what it was
        case = make_case(1000, 2560, seed=31)
        buf = B.expand(ctx, B.PLANES, case.d_codes, 1000, case.nb)
        y = torch.empty(1000, dtype=torch.float32, device="cuda")
        B.gemv_static(buf, case.d_scale, GAIN, case.d_x, 1000, case.nb * 24, y)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        for _ in range(3):
            B.gemv_static(buf, case.d_scale, GAIN, case.d_x, 1000, case.nb * 24, y)
        B.static_status()
        assert torch.cuda.mem_get_info()[0] == free_before
    finally:
        ctx.close()


def test_static_time_out_is_reported_and_repaired():
    """A wait that runs out (the one-warp self-test kernel: nothing faults) raises the static entry point's flag;
    llvq_static_status reports it once, clears flag and scratch, and the next launch is right again."""
    from paper_2609_02652_b200 import binding as B

    B.load()
    torch.cuda.set_device(0)
    ctx = B.create(0)
    try:
        case = make_case(257, 960, seed=33)
        buf = B.expand(ctx, B.PLANES, case.d_codes, case.rows, case.nb)
        ref = B.gemv(ctx, B.PLANES, buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24)
        B.static_selftest_wait_limit()
        with pytest.raises(B.LlvqError) as e:
            B.static_status()
        assert e.value.code == -5
        B.static_status()                               # reported once, then clear
        y = torch.empty(case.rows, dtype=torch.float32, device="cuda")
        B.gemv_static(buf, case.d_scale, GAIN, case.d_x, case.rows, case.nb * 24, y)
        B.static_status()
        assert torch.equal(y, ref)
    finally:
        ctx.close()


_FIRST_CALL_FROM_TWO_THREADS = r"""
import sys, threading
import numpy as np, torch
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
from helpers import GAIN, make_case
from paper_2609_02652_b200 import binding as B
B.load(); torch.cuda.set_device(0)
ctx = B.create(0)
cases = [make_case(513, 1200, seed=41 + i) for i in range(2)]
bufs = [B.expand(ctx, B.PLANES, c.d_codes, c.rows, c.nb) for c in cases]
refs = [B.gemv(ctx, B.PLANES, b, c.d_scale, GAIN, c.d_x, c.rows, c.nb * 24) for b, c in zip(bufs, cases)]
ys = [torch.empty(c.rows, dtype=torch.float32, device="cuda") for c in cases]
torch.cuda.synchronize()
gate, rcs = threading.Barrier(2), [None, None]
def first_call(i):
    # the process's first llvq_gemv_static calls, from two host threads at once: one sets the device up, the other
    # waits for it; the launches themselves are serialised on one stream (they share the built-in scratch)
    gate.wait()
    try:
        B.gemv_static(bufs[i], cases[i].d_scale, GAIN, cases[i].d_x, cases[i].rows, cases[i].nb * 24, ys[i], stream=torch.cuda.default_stream())
        rcs[i] = 0
    except Exception as e:
        rcs[i] = repr(e)
ts = [threading.Thread(target=first_call, args=(i,)) for i in range(2)]
[t.start() for t in ts]; [t.join() for t in ts]
B.static_status()
assert rcs == [0, 0], rcs
assert all(torch.equal(y, r) for y, r in zip(ys, refs))
print("ok")
"""


def test_first_call_from_two_host_threads_at_once():
    """The set-up the first call on a device does is guarded: two threads that make that first call together both
    succeed and both get llvq_gemv's results.  Needs a process that has not called the entry point yet: a child."""
    import os
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", _FIRST_CALL_FROM_TWO_THREADS, root], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and r.stdout.strip().endswith("ok"), r.stdout + r.stderr
