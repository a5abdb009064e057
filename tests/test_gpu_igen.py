"""On-device taskset generation (gcaps_gen_count / gcaps_gen_fill) through the C-ABI: bit-exact
against the generator's oracle (oracle/igen_oracle.py, plain Python integers, no code in common
with the library) on samples of every workload, against the host build of the library's own
generator on larger ranges, and the analysis of tasksets that were generated on the device against
the CPU oracle on their host-generated twins."""
import ctypes

import numpy as np
import pytest

from oracle import rta
from oracle.igen_oracle import reference_taskset
from paper_2406_05221_b200 import binding, taskgen

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def assert_same(ts, batch, what):
    for f in taskgen.ARRAY_FIELDS:
        got = ts.t[f].cpu().numpy()
        assert got.shape == getattr(batch, f).shape, (what, f)
        assert np.array_equal(got, getattr(batch, f)), (what, f)


@pytest.mark.parametrize("name,stream,first,count", [
    ("pr1", 0, 0, 300), ("sweep", 0, 77, 200), ("sweep", 4, 50_000, 200), ("sweep", 8, 99_900, 100),
    ("large", 0, 999_950, 50), ("rr_model", 0, 123_456, 200), ("divergence", 0, 9_999_900, 100),
    ("divergence", 0, 31, 150)])
def test_device_generation_equals_the_generator_oracle(name, stream, first, count):
    """The device output against the plain-integer oracle of the generator, taskset by taskset."""
    w = taskgen.WORKLOADS[name]
    ts = binding.generate_device(w.streams[stream], first, count)
    torch.cuda.synchronize()
    p = w.streams[stream].int_params()
    want = taskgen.TasksetBatch.from_tasksets([reference_taskset(p, first + t) for t in range(count)])
    assert_same(ts, want, "%s/%d against the oracle" % (name, stream))


def test_device_generation_at_the_range_ends_equals_the_generator_oracle():
    params = taskgen.GenParams(seed=42, cores=(1, 3), tasks_per_core=(1, 3), util_per_core=(0.5, 0.99),
                               period_us=(1e6, 1.07e9), gpu_mode=1, gpu_segments=(0, 16),
                               gpu_ratio=(0.0, 0.99), harmonic_frac=0.5, wfd=True)
    ts = binding.generate_device(params, 3, 400)
    torch.cuda.synchronize()
    p = params.int_params()
    want = taskgen.TasksetBatch.from_tasksets([reference_taskset(p, 3 + t) for t in range(400)])
    assert_same(ts, want, "range ends against the oracle")


@pytest.mark.parametrize("name,stream,first,count", [
    ("pr1", 0, 0, 1000), ("sweep", 0, 5, 4097), ("sweep", 8, 99_000, 1000), ("large", 0, 17, 2500),
    ("rr_model", 0, 123_456, 3000), ("divergence", 0, 9_990_000, 5001), ("divergence", 0, 0, 1)])
def test_device_generation_equals_host_generation(name, stream, first, count):
    w = taskgen.WORKLOADS[name]
    ts = binding.generate_device(w.streams[stream], first, count)
    torch.cuda.synchronize()
    assert_same(ts, w.generate(first, count, stream=stream, integer=True), name)


def test_device_generation_at_the_ends_of_the_parameter_ranges():
    """Periods up to 2^30 us with most of a core's utilisation in one or two tasks (quotients of
    the segment split near 2^29), up to 16 segments, harmonic periods, per-task segment counts,
    worst-fit allocation over many cores, cores without tasks."""
    cases = [
        taskgen.GenParams(seed=41, cores=(1, 3), tasks_per_core=(1, 2), util_per_core=(0.9, 0.99),
                          period_us=(5e8, 1.07e9), gpu_frac=1.0, gpu_segments=(1, 16), gpu_ratio=(0.5, 0.95)),
        taskgen.GenParams(seed=42, cores=(1, 3), tasks_per_core=(1, 3), util_per_core=(0.5, 0.99),
                          period_us=(1e6, 1.07e9), gpu_mode=1, gpu_segments=(0, 16), gpu_ratio=(0.0, 0.99),
                          harmonic_frac=0.5, wfd=True),
        taskgen.GenParams(seed=43, cores=(33, 64), tasks_per_core=(0, 4), util_per_core=(0.01, 0.2),
                          period_us=(1.0, 50.0), gpu_frac=0.7, gpu_segments=(2, 9), gpu_ratio=(0.3, 0.9), wfd=True),
    ]
    for k, params in enumerate(cases):
        ts = binding.generate_device(params, 3, 3000)
        torch.cuda.synchronize()
        twin = taskgen.generate(params, 3, 3000, integer=True)
        assert_same(ts, twin, "case %d" % k)
        if k == 0:
            assert twin.cseg_wcet.max() > 1 << 26 and twin.gseg_exec.max() > 1 << 26


def test_analysis_of_device_generated_tasksets():
    for name, count in (("sweep", 3000), ("large", 800), ("divergence", 2500)):
        w = taskgen.WORKLOADS[name]
        ts = binding.generate_device(w.streams[0], 7, count)
        twin = w.generate(7, count, integer=True)
        for policy in (0, 1, 0x101):
            wc, sc = binding.rta_batch(ts, policy, w.timeslice_us, w.overhead_us)
            torch.cuda.synchronize()
            w_ref, s_ref, _ = rta.analyse(twin, policy, w.timeslice_us, w.overhead_us)
            assert np.array_equal(sc.cpu().numpy(), s_ref), (name, policy)
            assert np.array_equal(wc.cpu().numpy(), w_ref), (name, policy)
        if name == "sweep":
            assert s_ref.max() == 1


def test_full_size_large_stream_sampled():
    """1,000,000 tasksets of the bench shape generated on the device; slices regenerated on the
    host are compared through the offsets, and the array lengths through the totals."""
    w = taskgen.WORKLOADS["large"]
    timing = {}
    ts = binding.generate_device(w.streams[0], 0, w.n_tasksets, timing=timing)
    assert ts.n_tasksets == w.n_tasksets and ts.n_tasks == 80 * w.n_tasksets
    off = {f: ts.t[f] for f in ("task_off", "cseg_off", "gseg_off")}
    for first in (0, 499_990, 999_000):
        twin = w.generate(first, 1000, integer=True)
        k0 = int(off["task_off"][first]); k1 = int(off["task_off"][first + 1000])
        c0 = int(off["cseg_off"][k0]); c1 = int(off["cseg_off"][k1])
        g0 = int(off["gseg_off"][k0]); g1 = int(off["gseg_off"][k1])
        assert k1 - k0 == twin.n_tasks and c1 - c0 == twin.n_csegs and g1 - g0 == twin.n_gsegs
        for f, (a, b) in (("period", (k0, k1)), ("priority", (k0, k1)), ("core", (k0, k1)),
                          ("deadline", (k0, k1)), ("cseg_wcet", (c0, c1)), ("gseg_misc", (g0, g1)),
                          ("gseg_exec", (g0, g1))):
            assert np.array_equal(ts.t[f][a:b].cpu().numpy(), getattr(twin, f)), (first, f)
        assert np.array_equal(ts.t["cseg_off"][k0:k1 + 1].cpu().numpy() - c0, twin.cseg_off)
        assert np.array_equal(ts.t["gseg_off"][k0:k1 + 1].cpu().numpy() - g0, twin.gseg_off)
    assert int(off["cseg_off"][-1]) == ts.n_csegs and int(off["gseg_off"][-1]) == ts.n_gsegs


def test_empty_and_argument_errors():
    w = taskgen.WORKLOADS["pr1"]
    ts = binding.generate_device(w.streams[0], 0, 0)
    assert ts.n_tasksets == 0 and ts.n_tasks == 0
    lib = binding.load_library()
    good = w.streams[0].int_params()
    totals = torch.zeros(3, dtype=torch.int64, device="cuda")
    ws = torch.empty(int(lib.gcaps_gen_workspace_bytes(ctypes.byref(good), 100)), dtype=torch.uint8, device="cuda")
    bad = w.streams[0].int_params()
    bad.tpc_hi = 300
    assert lib.gcaps_gen_count(ctypes.byref(bad), 0, 100, totals.data_ptr(), ws.data_ptr(), ws.numel(), None) == binding.ERR_INVALID_ARG
    bad = w.streams[0].int_params()
    bad.seg_hi = 17
    assert lib.gcaps_gen_count(ctypes.byref(bad), 0, 100, totals.data_ptr(), ws.data_ptr(), ws.numel(), None) == binding.ERR_INVALID_ARG
    assert lib.gcaps_gen_count(ctypes.byref(good), 0, 100, totals.data_ptr(), ws.data_ptr(), 64, None) == binding.ERR_WORKSPACE
    assert lib.gcaps_gen_count(ctypes.byref(good), -1, 100, totals.data_ptr(), ws.data_ptr(), ws.numel(), None) == binding.ERR_INVALID_ARG
    assert lib.gcaps_gen_count(ctypes.byref(good), 0, 100, None, ws.data_ptr(), ws.numel(), None) == binding.ERR_INVALID_ARG


def test_arrays_that_are_too_short_are_not_overrun():
    """gcaps_gen_fill with capacities below the totals leaves out what does not fit and writes
    nothing behind the capacities (guard words stay intact)."""
    w = taskgen.WORKLOADS["sweep"]
    lib = binding.load_library()
    cp = w.streams[0].int_params()
    count = 500
    twin = w.generate(0, count, integer=True)
    ws = torch.empty(int(lib.gcaps_gen_workspace_bytes(ctypes.byref(cp), count)), dtype=torch.uint8, device="cuda")
    totals = torch.zeros(3, dtype=torch.int64, device="cuda")
    assert lib.gcaps_gen_count(ctypes.byref(cp), 0, count, totals.data_ptr(), ws.data_ptr(), ws.numel(), None) == 0
    assert totals.cpu().tolist() == [twin.n_tasks, twin.n_csegs, twin.n_gsegs]
    cap_t, cap_c, cap_g = twin.n_tasks // 2, twin.n_csegs // 2, twin.n_gsegs // 2
    guard = -77
    sizes = {"task_off": count + 1, "period": cap_t, "deadline": cap_t, "priority": cap_t, "core": cap_t,
             "cseg_off": cap_t + 1, "cseg_wcet": cap_c, "gseg_off": cap_t + 1, "gseg_misc": cap_g, "gseg_exec": cap_g}
    t = {f: torch.full((sizes[f] + 64,), guard, dtype=torch.int64, device="cuda") for f in taskgen.ARRAY_FIELDS}
    c = binding.CTasksets(cap_t, cap_c, cap_g, *[t[f].data_ptr() for f in taskgen.ARRAY_FIELDS])
    assert lib.gcaps_gen_fill(ctypes.byref(cp), 0, count, ctypes.byref(c), ws.data_ptr(), ws.numel(), None) == 0
    torch.cuda.synchronize()
    for f in taskgen.ARRAY_FIELDS:
        assert (t[f][sizes[f]:] == guard).all(), f
    fit = int((twin.task_off[1:] <= cap_t).sum())     # tasksets that fit all three capacities
    fit = min(fit, int((twin.cseg_off[twin.task_off[1:fit + 1]] <= cap_c).sum()),
              int((twin.gseg_off[twin.task_off[1:fit + 1]] <= cap_g).sum()))
    k = int(twin.task_off[fit])
    assert np.array_equal(t["period"][:k].cpu().numpy(), twin.period[:k])
