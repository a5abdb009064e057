"""gcaps_rta_batch_static: the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not theirs to call (a plug-in whose host owns
the allocator, a process that must not allocate after start-up).  For them the library carries
its own fixed scratch array.  This test calls that entry point through the C-ABI twice in a row
and requires exactly the outputs of the ordinary entry point (all values are integers, so the
tolerance is zero), with the second call finding the first call's left-overs in the scratch.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2406_05221_b200 import binding, taskgen

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def _both(batch, policy, L, ovh):
    ts = binding.DeviceTasksets.from_host(batch)
    ref_w, ref_s = binding.rta_batch(ts, policy, L, ovh)
    torch.cuda.synchronize()
    out_w = torch.full((ts.n_tasks,), 12345, dtype=torch.int64, device="cuda")
    out_s = torch.full((ts.n_tasksets,), 77, dtype=torch.uint8, device="cuda")
    binding.rta_batch_static(ts, policy, L, ovh, out_wcrt=out_w, out_sched=out_s)
    torch.cuda.synchronize()
    assert torch.equal(out_w, ref_w) and torch.equal(out_s, ref_s)


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first call: a ragged batch that fills several size bins and most of the scratch
    big = taskgen.WORKLOADS["divergence"].generate(0, 60_000)
    _both(big, binding.POLICY_GCAPS, 1024, 50)
    # second call straight after it: another shape, another policy, a much smaller plan, so the
    # scratch still holds most of the first call's permutation
    small = taskgen.WORKLOADS["sweep"].generate(0, 3_000, stream=1)
    _both(small, binding.POLICY_RR | binding.BUSY, 512, 25)
    # and the first batch again, now with the other policy
    _both(big, binding.POLICY_RR, 1024, 50)


def test_limit_is_enforced_without_enqueuing_anything():
    lib = binding.load_library()
    full = taskgen.WORKLOADS["pr1"].generate(0, 10)
    ts = binding.DeviceTasksets.from_host(full)
    out_w = torch.zeros(ts.n_tasks, dtype=torch.int64, device="cuda")
    out_s = torch.zeros(ts.n_tasksets, dtype=torch.uint8, device="cuda")
    rc = lib.gcaps_rta_batch_static(ctypes.byref(ts.c), binding.STATIC_MAX_TASKSETS + 1, 0, 1024, 0,
                                    out_w.data_ptr(), out_s.data_ptr(), None)
    assert rc == binding.ERR_TOO_LARGE
    assert b"GCAPS_RTA_STATIC_MAX_TASKSETS" in lib.gcaps_rta_strerror(rc)
    torch.cuda.synchronize()
    assert int(out_w.abs().sum()) == 0 and int(out_s.sum()) == 0
    # exactly at the limit it runs
    edge = taskgen.WORKLOADS["pr1"].generate(0, 1000)
    reps = binding.STATIC_MAX_TASKSETS // 1000 + 1
    at_limit = taskgen.TasksetBatch.concat([edge] * reps).slice(0, binding.STATIC_MAX_TASKSETS)
    _both(at_limit, binding.POLICY_GCAPS, 1024, 50)
