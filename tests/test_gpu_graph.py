"""The analysis calls only enqueue work on the caller's stream (no allocation, no host
synchronisation), so a caller can record one into a CUDA graph and replay it on new data held in
the same buffers.  Replays must give the oracle's values for whatever the buffers hold then."""
import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import binding, taskgen
from tests.helpers import BUSY

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def capture(fn):
    """One plain call (first use sets kernel attributes), then the same call recorded in a graph."""
    fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


@pytest.mark.parametrize("name,count", [("pr1", 1000), ("divergence", 1500), ("large", 300)])
def test_replayed_batch_call_follows_the_buffers(name, count):
    w = taskgen.WORKLOADS[name]
    b = w.generate(17, count)
    ts = binding.DeviceTasksets.from_host(b)
    ws = torch.empty(max(binding.workspace_bytes(ts.n_tasksets), 256), dtype=torch.uint8, device="cuda")
    wc = torch.empty(ts.n_tasks, dtype=torch.int64, device="cuda")
    sc = torch.empty(ts.n_tasksets, dtype=torch.uint8, device="cuda")
    for policy in (0, 1, 1 | BUSY):
        g = capture(lambda: binding.rta_batch(ts, policy, w.timeslice_us, w.overhead_us, out_wcrt=wc,
                                              out_sched=sc, workspace=ws))
        # same structure, other execution times: CPU segments grow by a half, in place
        cur = b
        for scale_num in (2, 3):
            wc.fill_(binding.WCRT_INVALID)
            sc.fill_(binding.SCHED_INVALID)
            g.replay()
            torch.cuda.synchronize()
            w_ref, s_ref = rta.analyse(cur, policy, w.timeslice_us, w.overhead_us)[:2]
            assert (sc.cpu().numpy() == s_ref).all(), (name, policy)
            assert (wc.cpu().numpy() == w_ref).all(), (name, policy)
            cur = b.select(np.arange(b.n_tasksets))
            cur.cseg_wcet = (b.cseg_wcet * (scale_num + 1)) // 2
            ts.t["cseg_wcet"].copy_(torch.from_numpy(cur.cseg_wcet))
        ts.t["cseg_wcet"].copy_(torch.from_numpy(b.cseg_wcet))
        torch.cuda.synchronize()


def test_replayed_sweep_and_gpu_priority_calls():
    w = taskgen.WORKLOADS["rr_model"]
    b = w.generate(5, 1200)
    ts = binding.DeviceTasksets.from_host(b)
    Ls = [L for L in w.timeslices for _ in w.overheads]
    th = [t for _ in w.timeslices for t in w.overheads]
    ws = torch.empty(max(binding.workspace_bytes(ts.n_tasksets), 256), dtype=torch.uint8, device="cuda")
    wc = torch.empty((len(Ls), ts.n_tasks), dtype=torch.int64, device="cuda")
    sc = torch.empty((len(Ls), ts.n_tasksets), dtype=torch.uint8, device="cuda")
    g = capture(lambda: binding.rta_sweep(ts, 1, Ls, th, out_wcrt=wc, out_sched=sc, workspace=ws))
    wc.fill_(binding.WCRT_INVALID)
    sc.fill_(binding.SCHED_INVALID)
    g.replay()
    torch.cuda.synchronize()
    w_ref, s_ref = rta.analyse_sweep(b, 1, Ls, th)
    assert (sc.cpu().numpy() == s_ref).all() and (wc.cpu().numpy() == w_ref).all()

    # the priority search allocates its result tensors itself: inside a capture they come from the
    # graph's own pool and stay valid for as long as the graph does
    out = {}
    g2 = capture(lambda: out.update(r=binding.rta_gpu_priority(ts, binding.ASSIGN, 100, None, workspace=ws)))
    g2.replay()
    torch.cuda.synchronize()
    ref = rta.analyse_gpu_priority(b, rta.FLAG_ASSIGN, 100)
    for got, want in zip(out["r"], ref):
        assert (got.cpu().numpy() == want).all()
