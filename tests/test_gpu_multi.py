"""GPU parity of gcaps_rta_multi_batch (several analyses of a batch in one pass) against the CPU
oracle: by definition one independent oracle run per analysis and per (timeslice, overhead)
pair; bit-exact."""
import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import binding, taskgen
from tests.helpers import BEST_EFFORT, LITERAL, batch_of, random_tasksets
from tests.test_oracle_best_effort import _demote

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
B = binding


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def multi_parity(batch, analyses, Ls, ovhs, flags=0, what=""):
    ts = binding.DeviceTasksets.from_host(batch)
    pols = [B.ANALYSIS_POLICY[a] | flags for a in (1, 2, 4, 8) if analyses & a]
    n, k = len(ovhs), len(pols)
    wc = torch.full((n, k, ts.n_tasks), B.WCRT_INVALID, dtype=torch.int64, device="cuda")
    sc = torch.full((n, k, max(ts.n_tasksets, 0)), B.SCHED_INVALID, dtype=torch.uint8, device="cuda")
    binding.rta_multi(ts, analyses, Ls, ovhs, flags, out_wcrt=wc, out_sched=sc)
    torch.cuda.synchronize()
    w_ref, s_ref = rta.analyse_multi(batch, pols, Ls, ovhs)
    wc, sc = wc.cpu().numpy(), sc.cpu().numpy()
    for q in range(n):
        for j in range(k):
            bad = np.nonzero(sc[q, j] != s_ref[q, j])[0]
            assert bad.size == 0, "%s pair %d analysis %d: out_sched differs at %s" % (what, q, j, bad[:5])
            bad = np.nonzero(wc[q, j] != w_ref[q, j])[0]
            assert bad.size == 0, "%s pair %d analysis %d: out_wcrt differs at %s: %s vs %s" % (
                what, q, j, bad[:5], wc[q, j][bad[:5]], w_ref[q, j][bad[:5]])
    _, sc2 = binding.rta_multi(ts, analyses, Ls, ovhs, flags, want_wcrt=False)
    torch.cuda.synchronize()
    assert (sc2.cpu().numpy() == s_ref).all(), what
    return wc, sc


@pytest.mark.parametrize("analyses", [5, 10, 15, 3, 12, 6, 9, 7, 14, 1, 8])
def test_every_combination_of_analyses_on_random_tasksets(analyses):
    rng = np.random.default_rng(analyses)
    sets = random_tasksets(rng, 2000, max_tasks=12, max_cores=4, wcet_hi=8)
    sets += random_tasksets(rng, 300, max_tasks=40, max_cores=5, unique_prio=False)
    multi_parity(batch_of(sets), analyses, [3, 3, 7], [0, 2, 1], 0, "random")


@pytest.mark.parametrize("name,count", [("pr1", 1000), ("sweep", 3000), ("large", 1500),
                                        ("rr_model", 2500), ("divergence", 6000)])
def test_the_two_policies_of_a_bench_step_in_one_call(name, count):
    """GCAPS and round robin, self-suspension, at the workload's constants: what one bench step
    computes; then all four analyses at two pairs."""
    w = taskgen.WORKLOADS[name]
    best = 0
    for stream in sorted({0, len(w.streams) - 1}):
        b = w.generate(11, count - 5, stream=stream)
        _, sc = multi_parity(b, 5, [w.timeslice_us], [w.overhead_us], 0, name)
        best = max(best, int(sc.max()))
        multi_parity(b, 15, [w.timeslice_us, 256], [w.overhead_us, 0], 0, name + " all four")
    if name in ("pr1", "sweep"):
        assert best == 1  # the easy end of the sweep has schedulable tasksets


def test_flags_and_values_that_leave_the_32_bit_path():
    rng = np.random.default_rng(12)
    sets, _ = _demote(random_tasksets(rng, 1500, max_tasks=12, max_cores=4, wcet_hi=8), rng)
    b = batch_of(sets)
    multi_parity(b, 15, [4, 9], [1, 0], BEST_EFFORT, "best effort")
    multi_parity(b, 15, [4], [1], LITERAL, "literal")
    multi_parity(b, 5, [5, 1 << 30], [1 << 21, 3], 0, "huge overhead: exact path")
    big = 1 << 30
    wide = [[dict(T=big, prio=2, core=0, cseg=[big // 8], gseg=[(big // 16, big // 16)]),
             dict(T=big, prio=1, core=0, cseg=[big // 4], gseg=[(1, big // 8)] * 3)]] * 40
    multi_parity(batch_of(sets[:300] + wide), 15, [1000], [5], 0, "wide values")


def test_invalid_empty_and_argument_errors():
    rng = np.random.default_rng(2)
    b = batch_of(random_tasksets(rng, 300, max_tasks=10))
    b.period = b.period.copy()
    b.period[7] = -1
    _, sc = multi_parity(b, 15, [4], [0], 0, "invalid")
    assert (sc == B.SCHED_INVALID).sum() == 4
    ts = binding.DeviceTasksets.from_host(batch_of([]))
    wc, sc = binding.rta_multi(ts, 5, [4], [0])
    assert sc.shape == (1, 2, 0)
    ts = binding.DeviceTasksets.from_host(batch_of(random_tasksets(rng, 5)))
    for bad in (dict(analyses=0), dict(analyses=16), dict(analyses=5, flags=0x100),
                dict(analyses=4, timeslices_us=None), dict(analyses=4, timeslices_us=[0])):
        kw = dict(analyses=5, timeslices_us=[4], overheads_us=[0], flags=0)
        kw.update(bad)
        with pytest.raises(binding.GcapsError) as e:
            binding.rta_multi(ts, kw["analyses"], kw["timeslices_us"], kw["overheads_us"], kw["flags"])
        assert e.value.code == binding.ERR_INVALID_ARG


def test_full_size_large_workload_in_the_bench_call_sampled():
    """1,000,000 tasksets of 80 tasks, GCAPS + round robin in the one call the benchmark times."""
    w = taskgen.WORKLOADS["large"]
    b = w.generate(0, w.n_tasksets)
    ts = binding.DeviceTasksets.from_host(b)
    wc, sc = binding.rta_multi(ts, 5, [w.timeslice_us], [w.overhead_us])
    torch.cuda.synchronize()
    wc, sc = wc.cpu().numpy()[0].reshape(2, -1, 80), sc.cpu().numpy()[0]
    rng = np.random.default_rng(4)
    sample = np.sort(rng.choice(w.n_tasksets, 2500, replace=False))
    sub = b.select(sample)
    for j, policy in enumerate((0, 1)):
        w_ref, s_ref, _ = rta.analyse(sub, policy, w.timeslice_us, w.overhead_us)
        assert (sc[j][sample] == s_ref).all()
        assert (wc[j][sample].reshape(-1) == w_ref).all()
        assert sc[j].max() <= 1
        has_neg = (wc[j] < 0).any(axis=1)
        assert ((sc[j] == 1) == ~has_neg).all()
        ok = wc[j] >= 0
        assert (wc[j][ok] <= b.deadline.reshape(-1, 80)[ok]).all()
