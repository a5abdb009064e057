"""GPU parity of the analysis with separate GPU-segment priorities and of the priority search
(paper Sec. 5.3, 6.4) against the CPU oracle, through the C-ABI; bit-exact."""
import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import binding, taskgen
from tests.helpers import BUSY, LITERAL, batch_of, parse_vectors, random_tasksets
from tests.test_oracle_gpu_priority import gp_cases

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
ASSIGN = binding.ASSIGN


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def gpu_gp(batch, flags, eps, gpu_priority=None):
    ts = binding.DeviceTasksets.from_host(batch)
    gp = None if gpu_priority is None else torch.from_numpy(np.asarray(gpu_priority, np.int64)).cuda()
    w, s, out = binding.rta_gpu_priority(ts, flags, eps, gp)
    torch.cuda.synchronize()
    return w.cpu().numpy(), s.cpu().numpy(), out.cpu().numpy()


def assert_gp_parity(batch, flags, eps, gpu_priority=None, what=""):
    w_ref, s_ref, g_ref = rta.analyse_gpu_priority(batch, flags, eps, gpu_priority=gpu_priority)
    w, s, g = gpu_gp(batch, flags, eps, gpu_priority)
    assert (s == s_ref).all(), what
    assert (w == w_ref).all(), what
    if flags & ASSIGN:
        assert (g == g_ref).all(), what
    return w, s, g


def test_table2_vectors():
    tasks, _ = parse_vectors("table2_vectors.txt")
    b = batch_of([tasks])
    for c in gp_cases():
        flags = (BUSY if c["busy"] else 0) | (ASSIGN if c["gpu"] is None else 0)
        w, s, g = gpu_gp(b, flags, c["eps"], c["gpu"])
        assert w.tolist() == c["expect"] and s[0] == c["sched"], c["name"]
        if c["levels"]:
            assert g.tolist() == c["levels"], c["name"]


@pytest.mark.parametrize("flags", [0, BUSY, BUSY | LITERAL])
def test_random_small_tasksets(flags):
    rng = np.random.default_rng(51 + flags)
    sets = random_tasksets(rng, 2500, max_tasks=12, max_cores=4, wcet_hi=7)
    sets += random_tasksets(rng, 300, max_tasks=10, unique_prio=False)
    b = batch_of(sets)
    for eps in (0, 1, 3):
        assert_gp_parity(b, flags | ASSIGN, eps, what="assign")
        assert_gp_parity(b, flags, eps, gpu_priority=b.priority, what="cpu priorities as gpu priorities")
    # arbitrary GPU priorities: many break the same-core rule and must come back INVALID
    gp = rng.integers(0, 6, b.n_tasks)
    w, s, _ = assert_gp_parity(b, flags, 1, gpu_priority=gp, what="random gpu priorities")
    assert (s == 2).any() and (s != 2).any()


def test_workload_samples_and_edges():
    for name, count in (("pr1", 1000), ("sweep", 2000), ("rr_model", 1500), ("large", 300), ("divergence", 1500)):
        w = taskgen.WORKLOADS[name]
        b = w.generate(3, count, stream=min(2, len(w.streams) - 1))
        for flags in (0, BUSY):
            assert_gp_parity(b, flags | ASSIGN, w.overhead_us, what=name)
            assert_gp_parity(b, flags, w.overhead_us, gpu_priority=b.priority, what=name)
    big = 1 << 40
    sets = [[], [dict(T=10, D=11, prio=1, core=0, cseg=[1])], [dict(T=10, prio=1, core=0, cseg=[-1])],
            [dict(T=big, prio=2, core=0, cseg=[big // 8], gseg=[(big // 16, big // 16)]),
             dict(T=big, prio=1, core=1, cseg=[big // 4], gseg=[(1, big // 8)] * 3)],
            [dict(T=2, prio=2, core=0, cseg=[2]), dict(T=1 << 23, prio=1, core=0, cseg=[1])],
            [dict(T=100000 + i, prio=i, core=i % 5, cseg=[3] * 3, gseg=[(1, 2)] * (i % 4)) for i in range(256)],
            [dict(T=100, prio=i, core=0, cseg=[1]) for i in range(257)]]
    b = batch_of(sets)
    for flags in (ASSIGN, ASSIGN | BUSY):
        for eps in (0, 5, big):
            assert_gp_parity(b, flags, eps, what="edges")
    assert_gp_parity(b, 0, 5, gpu_priority=b.priority, what="edges given")


def test_search_rescues_tasksets_on_the_sweep_workload():
    """The paper's experiment (Sec. 7.1): run the default test, then the priority search on what
    fails.  On a mid-utilisation point of the sweep some tasksets are rescued."""
    w = taskgen.WORKLOADS["sweep"]
    b = w.generate(0, 20000, stream=1)
    ts = binding.DeviceTasksets.from_host(b)
    _, s_default = binding.rta_batch(ts, 0, w.timeslice_us, w.overhead_us)
    _, s_search, _ = binding.rta_gpu_priority(ts, ASSIGN, w.overhead_us)
    torch.cuda.synchronize()
    s_default, s_search = s_default.cpu().numpy(), s_search.cpu().numpy()
    either = (s_default == 1) | (s_search == 1)
    assert either.sum() >= (s_default == 1).sum()
    _, s_ref, _ = rta.analyse_gpu_priority(b.slice(0, 3000), ASSIGN, w.overhead_us)
    assert (s_search[:3000] == s_ref).all()
