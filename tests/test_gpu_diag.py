"""The two measurement aids of the library through the C-ABI: the planning step on its own and
the integer issue-rate probe."""
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


def test_planning_alone_leaves_a_permutation_grouped_by_size():
    """gcaps_rta_plan_batch writes what gcaps_rta_batch's own planning writes: a permutation of
    the taskset indices in which the tasksets of a size bin are contiguous; a following analysis
    call on the same workspace still matches the oracle."""
    w = taskgen.WORKLOADS["divergence"]
    b = w.generate(3, 20_000)
    ts = binding.DeviceTasksets.from_host(b)
    ws = torch.zeros(binding.workspace_bytes(ts.n_tasksets), dtype=torch.uint8, device="cuda")
    binding.rta_plan(ts, ws)
    torch.cuda.synchronize()
    raw = ws.cpu().numpy()
    hdr = raw[:144].view(np.uint32)                    # bin_start[12], bin_count[12], next[12]
    start, count = hdr[:12], hdr[12:24]
    assert int(count.sum()) == ts.n_tasksets and (hdr[24:36] == 0).all()
    plan_blocks = (ts.n_tasksets + 1023) // 1024
    perm_off = 256 + (plan_blocks * 12 * 4 + 255) // 256 * 256
    perm = raw[perm_off:perm_off + 4 * ts.n_tasksets].view(np.uint32)
    assert np.array_equal(np.sort(perm), np.arange(ts.n_tasksets, dtype=np.uint32))
    n = np.diff(b.task_off)[perm]
    limits = [8, 16, 24, 32, 64, 96, 128, 192, 256]
    for k, hi in enumerate(limits):
        lo = limits[k - 1] if k else -1
        part = n[start[k]:start[k] + count[k]]
        assert ((part > lo) & (part <= hi)).all(), k
    wc, sc = binding.rta_batch(ts, binding.POLICY_GCAPS, w.timeslice_us, w.overhead_us, workspace=ws)
    torch.cuda.synchronize()
    w_ref, s_ref, _ = rta.analyse(b, binding.POLICY_GCAPS, w.timeslice_us, w.overhead_us)
    assert np.array_equal(wc.cpu().numpy(), w_ref) and np.array_equal(sc.cpu().numpy(), s_ref)


def test_integer_issue_probe_counts_and_rates():
    lib = binding.load_library()
    scratch = torch.zeros(1, dtype=torch.int32, device="cuda")
    ops = ctypes.c_int64(0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for kind, per_step in ((0, 1), (1, 2), (2, 2)):
        assert lib.gcaps_rta_int_issue_probe(kind, 64, scratch.data_ptr(), ctypes.byref(ops), None) == 0
        assert ops.value == sms * 8 * 256 * 8 * 16 * 64 * per_step
    torch.cuda.synchronize()
    assert int(scratch.item()) == 0                      # the guard word is never written
    for bad in ((3, 64), (-1, 64), (0, 0), (0, (1 << 24) + 1)):
        assert lib.gcaps_rta_int_issue_probe(bad[0], bad[1], scratch.data_ptr(), ctypes.byref(ops), None) \
            == binding.ERR_INVALID_ARG
    assert lib.gcaps_rta_int_issue_probe(0, 64, None, ctypes.byref(ops), None) == binding.ERR_INVALID_ARG
    rates = [binding.int_issue_rate(kind, trips=1024, repeats=3) for kind in (0, 1, 2)]
    # between a tenth of and a little above 148 SMs x 128 lanes x 2 GHz
    for r in rates:
        assert 3e12 < r < 5e13, rates
    assert rates[1] > rates[0]                           # adds issue faster than multiply-adds
