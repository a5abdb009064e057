"""Stream order and host threads: what a caller may do without synchronising.

The kernels of the size bins of one call overlap one another (dependent launches).  Whatever the
caller enqueues on the same stream afterwards -- a copy of the results, the next call on the same
workspace -- must still find the whole call completed, also when the long-running kernel is the
first of the chain (a batch of small tasksets only: the kernels of the larger bins have nothing
to do and would finish at once).  Every check is against the CPU oracle.
"""
import threading

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


@pytest.fixture(scope="module")
def small_heavy():
    """300,000 tasksets of 20 tasks: everything lands in the bins of at most 32 tasks."""
    w = taskgen.WORKLOADS["sweep"]
    batch = w.generate(11, 300_000, stream=1)
    ref = {pol: rta.analyse(batch, pol, w.timeslice_us, w.overhead_us)[:2]
           for pol in (binding.POLICY_GCAPS, binding.POLICY_RR)}
    return w, batch, ref


def test_consumers_in_stream_order_see_finished_results(small_heavy):
    w, batch, ref = small_heavy
    ts = binding.DeviceTasksets.from_host(batch)
    side = torch.cuda.Stream()
    ws = torch.empty(binding.workspace_bytes(ts.n_tasksets), dtype=torch.uint8, device="cuda")
    out_w = torch.full((ts.n_tasks,), 12345, dtype=torch.int64, device="cuda")
    out_s = torch.full((ts.n_tasksets,), 77, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    got = {}
    with torch.cuda.stream(side):
        for rep in range(3):
            for pol in (binding.POLICY_GCAPS, binding.POLICY_RR):
                # same outputs, same workspace, no synchronisation anywhere in this loop: the copy
                # must see this call finished, the next call's plan must not disturb this one,
                # and the fill must not be overtaken by a kernel that is still writing
                binding.rta_batch(ts, pol, w.timeslice_us, w.overhead_us, out_wcrt=out_w,
                                  out_sched=out_s, workspace=ws, stream=side)
                got[(rep, pol)] = (out_w.clone(), out_s.clone())
                out_w.fill_(12345)
                out_s.fill_(77)
    side.synchronize()
    for (rep, pol), (gw, gs) in got.items():
        assert np.array_equal(gs.cpu().numpy(), ref[pol][1]), (rep, pol)
        assert np.array_equal(gw.cpu().numpy(), ref[pol][0]), (rep, pol)
    assert int((out_w != 12345).sum()) == 0 and int((out_s != 77).sum()) == 0


def test_static_calls_back_to_back_without_synchronising(small_heavy):
    w, batch, ref = small_heavy
    part = batch.slice(0, binding.STATIC_MAX_TASKSETS)
    n_tasks = int(part.task_off[-1])
    ts = binding.DeviceTasksets.from_host(part)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    got = []
    with torch.cuda.stream(side):
        for pol in (binding.POLICY_GCAPS, binding.POLICY_RR, binding.POLICY_GCAPS, binding.POLICY_RR):
            got.append((pol, binding.rta_batch_static(ts, pol, w.timeslice_us, w.overhead_us, stream=side)))
    side.synchronize()
    for pol, (gw, gs) in got:
        assert np.array_equal(gs.cpu().numpy(), ref[pol][1][:part.n_tasksets]), pol
        assert np.array_equal(gw.cpu().numpy(), ref[pol][0][:n_tasks]), pol


def test_priority_search_in_stream_order(small_heavy):
    w, batch, _ = small_heavy
    part = batch.slice(0, 60_000)
    ts = binding.DeviceTasksets.from_host(part)
    side = torch.cuda.Stream()
    ws = torch.empty(binding.workspace_bytes(ts.n_tasksets), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        first = binding.rta_gpu_priority(ts, binding.ASSIGN, w.overhead_us, workspace=ws, stream=side)
        first = tuple(x.clone() for x in first)
        second = binding.rta_batch(ts, binding.POLICY_GCAPS, w.timeslice_us, w.overhead_us,
                                   workspace=ws, stream=side)
    side.synchronize()
    want = rta.analyse_gpu_priority(part, rta.FLAG_ASSIGN, w.overhead_us)
    for x, y in zip(first, want):
        assert np.array_equal(x.cpu().numpy(), y)
    w_cpu, s_cpu, _ = rta.analyse(part, binding.POLICY_GCAPS, w.timeslice_us, w.overhead_us)
    assert np.array_equal(second[0].cpu().numpy(), w_cpu) and np.array_equal(second[1].cpu().numpy(), s_cpu)


def test_host_buffer_calls_from_two_threads():
    """The host-buffer entry points share one set of staging buffers; concurrent calls are
    serialised inside the library and each must still return its own batch's results."""
    jobs = []
    for seed, name, pol in ((1, "sweep", binding.POLICY_GCAPS), (2, "divergence", binding.POLICY_RR)):
        w = taskgen.WORKLOADS[name]
        b = w.generate(seed, 40_000)
        jobs.append((w, b, pol, rta.analyse(b, pol, w.timeslice_us, w.overhead_us)[:2]))
    results = [None, None]
    errors = []

    def run(k):
        try:
            w, b, pol, _ = jobs[k]
            arrays = {f: np.ascontiguousarray(getattr(b, f)) for f in binding.ARRAY_FIELDS}
            for _ in range(3):
                results[k] = binding.rta_batch_host(arrays, pol, w.timeslice_us, w.overhead_us)
        except Exception as exc:  # surfaced below, in the main thread
            errors.append(exc)

    threads = [threading.Thread(target=run, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    binding.release_host()
    assert not errors, errors
    for k in range(2):
        assert np.array_equal(results[k][0], jobs[k][3][0]) and np.array_equal(results[k][1], jobs[k][3][1])


def test_device_calls_from_two_threads_on_their_own_streams():
    w = taskgen.WORKLOADS["rr_model"]
    b = w.generate(5, 50_000)
    ts = binding.DeviceTasksets.from_host(b)
    want = {pol: rta.analyse(b, pol, w.timeslice_us, w.overhead_us)[:2] for pol in (0, 1)}
    out, errors = {}, []

    def run(pol):
        try:
            st = torch.cuda.Stream()
            for _ in range(5):
                out[pol] = binding.rta_batch(ts, pol, w.timeslice_us, w.overhead_us, stream=st)
            st.synchronize()
        except Exception as exc:
            errors.append(exc)

    threads = [threading.Thread(target=run, args=(pol,)) for pol in (0, 1)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for pol in (0, 1):
        assert np.array_equal(out[pol][0].cpu().numpy(), want[pol][0])
        assert np.array_equal(out[pol][1].cpu().numpy(), want[pol][1])
