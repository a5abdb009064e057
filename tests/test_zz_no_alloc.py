"""gcaps_rta_batch_static: the entry point for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not theirs to call (a plug-in whose host owns
the allocator, a process that must not allocate after start-up).  For them the library carries
its own fixed scratch array.  This test calls that entry point through the C-ABI twice in a row
and requires exactly the outputs of the ordinary entry point and of the CPU oracle (all values
are integers, so the tolerance is zero), with the second call finding the first call's
left-overs in the scratch; it also checks that such a call leaves the amount of free device
memory untouched.
"""
import ctypes

import numpy as np
import pytest

from oracle import rta
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
    # the oracle itself, not only the other entry point
    w_cpu, s_cpu, _ = rta.analyse(batch, policy, L, ovh)
    assert np.array_equal(out_w.cpu().numpy(), w_cpu)
    assert np.array_equal(out_s.cpu().numpy(), s_cpu)


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


def test_a_call_allocates_and_frees_nothing():
    """With the outputs in place beforehand, a call through the C-ABI must change neither the
    driver's count of free device memory nor what torch's allocator holds."""
    lib = binding.load_library()
    batch = taskgen.WORKLOADS["sweep"].generate(3, 20_000)
    ts = binding.DeviceTasksets.from_host(batch)
    out_w = torch.zeros(ts.n_tasks, dtype=torch.int64, device="cuda")
    out_s = torch.zeros(ts.n_tasksets, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call(policy):
        rc = lib.gcaps_rta_batch_static(ctypes.byref(ts.c), ts.n_tasksets, policy, 1024, 50,
                                        out_w.data_ptr(), out_s.data_ptr(), ctypes.c_void_p(stream))
        assert rc == 0
        torch.cuda.synchronize()

    call(binding.POLICY_GCAPS)  # the first call on a device looks the scratch address up
    free0, _ = torch.cuda.mem_get_info()
    torch0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    call(binding.POLICY_RR)
    call(binding.POLICY_GCAPS)
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == torch0 and torch.cuda.memory_reserved() == reserved0
    w_cpu, s_cpu, _ = rta.analyse(batch, binding.POLICY_GCAPS, 1024, 50)
    assert np.array_equal(out_w.cpu().numpy(), w_cpu) and np.array_equal(out_s.cpu().numpy(), s_cpu)
