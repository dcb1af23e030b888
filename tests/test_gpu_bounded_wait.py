"""The bounded barrier wait of the persistent kernels, run to its limit on the GPU.

Every wait in the encode, decode and transcode kernels is a loop of `mbarrier.try_wait` with a
time limit; a CTA whose wait runs out reports KVH_ERR_TIMEOUT, raises its abort flag so that its
other warps stop waiting too, and returns.  In a healthy run none of that code executes, so a
test-only kernel (its own library, not part of the C ABI) calls the very same wait routine on a
barrier nobody arrives at, with a limit of a millisecond.  Nothing hangs and nothing faults: the
launch must come back by itself, quickly, with status 8."""
import ctypes
import time

import pytest
import torch

from test_gpu_parity import kvh  # noqa: F401

pytestmark = pytest.mark.gpu


def test_a_wait_nobody_answers_runs_out_and_reports_timeout(kvh):
    from paper_2509_00105_b200 import _build
    L = ctypes.CDLL(str(_build.build(variant="selftest")))
    L.kvh_selftest_bounded_wait.restype = ctypes.c_int
    L.kvh_selftest_bounded_wait.argtypes = [ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((6,), -1, dtype=torch.int64, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    limit_ns = 1_000_000
    # arguments are checked first: no limit, or one long enough to look like a hang, is refused
    assert L.kvh_selftest_bounded_wait(0, status.data_ptr(), out.data_ptr(), stream) == 1
    assert L.kvh_selftest_bounded_wait(10**9, status.data_ptr(), out.data_ptr(), stream) == 1
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    assert L.kvh_selftest_bounded_wait(limit_ns, status.data_ptr(), out.data_ptr(), stream) == 0
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    assert status.item() == 8 and kvh.status_string(8) == "device wait timed out"
    ok0, ns0, ok1, ns1, ok2, ns2 = out.tolist()
    # warp 0: ran out, after the limit and not long after it
    assert ok0 == 0 and limit_ns <= ns0 < 50 * limit_ns
    # warp 1: had the library's 2 s limit but left through the abort flag warp 0 raised
    assert ok1 == 0 and ns1 < 100 * limit_ns
    # warp 2: its barrier was arrived at, so the wait succeeded (and took no time to speak of)
    assert ok2 == 1 and ns2 < limit_ns
    assert wall < 1.0                                   # the launch ended by itself, far below the 2 s limit
    # the context is intact: an ordinary call works afterwards
    status.zero_()
    kv = torch.zeros((1, 2, 64, 64), dtype=torch.bfloat16, device="cuda")
    kvh.encode(kv, 3, dev_status=status)
    assert status.item() == 0
