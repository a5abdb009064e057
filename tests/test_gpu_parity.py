"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C-ABI.

All times are integer microseconds, so the bar is bit-exact equality of every out_wcrt value
(including the sentinels) and every out_sched flag.
"""
import copy
import ctypes

import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import binding, taskgen
from tests.helpers import ALL_MODES, BUSY, LITERAL, batch_of, parse_vector_sets, random_tasksets

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MODES4 = [0, BUSY, 1, 1 | BUSY]


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    binding.load_library()


def gpu_run(batch, policy, L=1024, ovh=0):
    ts = binding.DeviceTasksets.from_host(batch)
    wcrt = torch.full((ts.n_tasks,), binding.WCRT_INVALID, dtype=torch.int64, device="cuda")
    sched = torch.full((max(ts.n_tasksets, 0),), binding.SCHED_INVALID, dtype=torch.uint8, device="cuda")
    binding.rta_batch(ts, policy, L, ovh, out_wcrt=wcrt, out_sched=sched)
    torch.cuda.synchronize()
    return wcrt.cpu().numpy(), sched.cpu().numpy()


def assert_parity(batch, policy, L=1024, ovh=0, what=""):
    w_ref, s_ref, _ = rta.analyse(batch, policy, L, ovh)
    w, s = gpu_run(batch, policy, L, ovh)
    bad_s = np.nonzero(s != s_ref)[0]
    assert bad_s.size == 0, "%s: out_sched differs at tasksets %s" % (what, bad_s[:5])
    bad_w = np.nonzero(w != w_ref)[0]
    assert bad_w.size == 0, "%s: out_wcrt differs at tasks %s: %s vs oracle %s" % (
        what, bad_w[:5], w[bad_w[:5]], w_ref[bad_w[:5]])
    return w, s


@pytest.mark.parametrize("fixture", ["table2_vectors.txt", "indirect_delay_vectors.txt",
                                     "same_core_jitter_vectors.txt"])
def test_hand_derived_vectors(fixture):
    for set_name, tasks, cases in parse_vector_sets(fixture):
        b = batch_of([tasks])
        for c in cases:
            w, s = gpu_run(b, c["policy"], c["L"], c["ovh"])
            assert w.tolist() == c["expect"], (set_name, c["name"])
            assert s[0] == (1 if min(c["expect"]) >= 0 else 0), (set_name, c["name"])


@pytest.mark.parametrize("policy", ALL_MODES)
def test_random_small_tasksets_all_modes(policy):
    rng = np.random.default_rng(policy + 11)
    sets = random_tasksets(rng, 3000, max_tasks=12, max_cores=4, wcet_hi=8)
    sets += random_tasksets(rng, 500, max_tasks=12, unique_prio=False)
    b = batch_of(sets)
    for L, ovh in ((1, 0), (3, 1), (7, 2)):
        assert_parity(b, policy, L, ovh, "random small")


@pytest.mark.parametrize("name,count", [("pr1", 1000), ("sweep", 3000), ("large", 1500),
                                        ("rr_model", 3000), ("divergence", 6000)])
def test_workload_samples(name, count):
    """The five benchmark workloads, several tiles and a ragged tail each."""
    w = taskgen.WORKLOADS[name]
    for stream in sorted({0, len(w.streams) // 2, len(w.streams) - 1}):
        b = w.generate(7, count - 3, stream=stream)
        modes = MODES4 if "gcaps" in w.policies else [1, 1 | BUSY]
        for policy in modes:
            wc, s = assert_parity(b, policy, w.timeslice_us, w.overhead_us, "%s/%d" % (name, stream))
        if name in ("pr1", "sweep") and stream == 0:
            assert s.max() == 1  # the easy end of the sweep has schedulable tasksets


def test_converging_large_tasksets():
    """Tasksets of 80 tasks that are schedulable under GCAPS: the recurrence runs for every task
    (two to three ranks per lane), every bound is a converged value."""
    w = taskgen.WORKLOADS["large_light"]
    b = w.generate(5, 1200)
    for policy in MODES4:
        wc, s = assert_parity(b, policy, w.timeslice_us, w.overhead_us, "large_light")
        if policy == 0:
            assert s.min() == 1 and wc.min() > 0


def test_rr_driver_model_grid():
    w = taskgen.WORKLOADS["rr_model"]
    b = w.generate(0, 1500)
    for L in w.timeslices:
        for theta in w.overheads:
            assert_parity(b, 1, L, theta, "rr grid L=%d theta=%d" % (L, theta))


def test_zero_overhead_and_literal_on_workloads():
    b = taskgen.WORKLOADS["sweep"].generate(0, 1500, stream=2)
    for policy in ALL_MODES:
        assert_parity(b, policy, 1024, 0, "sweep ovh=0")
        assert_parity(b, policy, 1000, 200, "sweep ovh=200")


def test_priorities_that_are_not_a_dense_numbering():
    """Sparse, tied and negative priority values on tasksets of every size bin: the kernels then
    count the tasks that come before instead of subtracting from the largest priority."""
    for name, count in (("sweep", 1500), ("large", 400), ("divergence", 2500)):
        w = taskgen.WORKLOADS[name]
        base = w.generate(29, count)
        for what, f in (("sparse", lambda p: p * 3 + 5), ("tied", lambda p: p // 2),
                        ("negative", lambda p: p * 7 - 1000)):
            b = base.select(np.arange(base.n_tasksets))
            b.priority = f(base.priority)
            for policy in (0, 1, BUSY, 1 | BUSY):
                assert_parity(b, policy, w.timeslice_us, w.overhead_us, "%s %s" % (name, what))
            ts = binding.DeviceTasksets.from_host(b)
            got = binding.rta_gpu_priority(ts, binding.ASSIGN, w.overhead_us)
            torch.cuda.synchronize()
            ref = rta.analyse_gpu_priority(b, rta.FLAG_ASSIGN, w.overhead_us)
            for x, y in zip(got, ref):
                assert np.array_equal(x.cpu().numpy(), y), "%s %s search" % (name, what)


def test_size_bins_and_edges():
    """Sizes around every bin boundary, empty tasksets, the maximum size, in one batch."""
    rng = np.random.default_rng(5)
    sets = []
    for n in (0, 1, 2, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 95, 96, 97, 128, 200, 255, 256, 0, 3):
        ts = []
        for i in range(n):
            T = int(rng.integers(2000, 200000))
            ng = int(rng.integers(0, 3))
            ts.append(dict(T=T, D=T - int(rng.integers(0, T // 4)), prio=int(rng.integers(0, 50)),
                           core=int(rng.integers(0, 9)),
                           cseg=[int(rng.integers(0, max(2, T // (40 * max(n, 1))))) for _ in range(ng + 1)],
                           gseg=[(int(rng.integers(0, 5)), int(rng.integers(0, max(2, T // (60 * max(n, 1))))))
                                 for _ in range(ng)]))
        sets.append(ts)
    b = batch_of(sets)
    for policy in ALL_MODES:
        assert_parity(b, policy, 64, 3, "bins")
    # reversed order exercises another permutation of the plan
    b2 = batch_of(sets[::-1])
    assert_parity(b2, 0, 64, 3, "bins reversed")


def test_empty_batch_and_empty_arrays():
    b = batch_of([])
    w, s = gpu_run(b, 0)
    assert w.size == 0 and s.size == 0
    b = batch_of([[], [], []])
    w, s = gpu_run(b, 1, 5, 1)
    assert s.tolist() == [1, 1, 1]


def test_invalid_tasksets_are_flagged_not_trapped():
    good = [dict(T=10, prio=1, core=0, cseg=[1], gseg=[(1, 2)])]
    sets = [good,
            [dict(T=10, D=11, prio=1, core=0, cseg=[1]), dict(T=10, prio=0, core=0, cseg=[1])],
            [dict(T=10, prio=1, core=0, cseg=[-1])],
            [],
            [dict(T=10, prio=1, core=-1, cseg=[1])],
            [dict(T=0, D=0, prio=1, core=0, cseg=[1])],
            [dict(T=(1 << 40) + 1, prio=1, core=0, cseg=[1])],
            [dict(T=100, prio=1, core=0, cseg=[1], gseg=[(0, (1 << 40) + 1)])],
            [dict(T=100, prio=i, core=0, cseg=[1]) for i in range(257)],
            good]
    b = batch_of(sets)
    for policy in (0, 1 | BUSY):
        w, s = assert_parity(b, policy, 4, 0, "invalid")
    assert s.tolist() == [1, 2, 2, 1, 2, 2, 2, 2, 2, 1]
    err = binding.rta_validate(binding.DeviceTasksets.from_host(b)).cpu().numpy()
    assert err.tolist() == rta.validate(b).tolist()
    # broken offsets: the oracle and the library agree and nothing faults
    for field, idx, val in (("task_off", 2, 9999), ("task_off", 3, -4), ("cseg_off", 2, -1),
                            ("gseg_off", 1, 1 << 50), ("cseg_off", 5, 0)):
        bb = copy.deepcopy(b)
        getattr(bb, field)[idx] = val
        w_ref, s_ref, _ = rta.analyse(bb, 0, 4, 0)
        w, s = gpu_run(bb, 0, 4, 0)
        assert (s == s_ref).all(), (field, idx)
        assert (w == w_ref).all(), (field, idx)
        err = binding.rta_validate(binding.DeviceTasksets.from_host(bb)).cpu().numpy()
        assert err.tolist() == rta.validate(bb).tolist()


def test_iteration_cap_and_extreme_values():
    B = 1 << 40
    sets = [
        [dict(T=2, prio=2, core=0, cseg=[2]), dict(T=1 << 23, prio=1, core=0, cseg=[1])],  # ITER_LIMIT
        [dict(T=2, prio=2, core=0, cseg=[2]), dict(T=1001, prio=1, core=0, cseg=[1])],     # slow miss
        [dict(T=B, prio=3, core=0, cseg=[B // 8], gseg=[(B // 16, B // 16)]),
         dict(T=B, prio=2, core=0, cseg=[B // 16], gseg=[(1, B // 16)]),
         dict(T=B, prio=1, core=1, cseg=[B // 2], gseg=[(0, 1)])],
        [dict(T=B, prio=1, core=0, cseg=[B >> 10] * 512, gseg=[(B >> 12, B >> 12)] * 512)],
        [dict(T=1, prio=2, core=0, cseg=[1]), dict(T=5, prio=1, core=0, cseg=[1])],
        [dict(T=50, prio=2, core=0, cseg=[0]), dict(T=50, prio=1, core=0, cseg=[0], gseg=[(0, 0)])],
    ]
    b = batch_of(sets)
    for policy in ALL_MODES:
        w, s = assert_parity(b, policy, 1, 0, "extreme")
        assert_parity(b, policy, 1, B, "extreme ovh")
        assert_parity(b, policy, B, 1, "extreme L")
    w, s = gpu_run(b, 0, 1, 0)
    assert w[1] == binding.WCRT_ITER_LIMIT and w[3] == binding.WCRT_MISS


def test_values_around_the_32_bit_path_limit():
    """Tasksets whose times sit just below, at and above 2^26 us (where the kernels switch from
    32-bit to exact 64-bit arithmetic), mixed in one batch; also small periods down to 2 and 1,
    priorities that are dense, sparse, negative, huge or tied, and tasks with many segments."""
    rng = np.random.default_rng(21)
    lim = 1 << 26
    sets = []
    for top in (lim - 1, lim, lim + 1, 3 * lim, lim // 2):
        for n in (3, 20, 33, 70):
            ts = []
            for i in range(n):
                T = int(top if i % 3 == 0 else rng.integers(top // 8, top))
                ng = int(rng.integers(0, 3))
                ts.append(dict(T=T, D=T - int(rng.integers(0, 3)), prio=0, core=int(rng.integers(0, 4)),
                               cseg=[int(rng.integers(0, T // (8 * n) + 2)) for _ in range(ng + 1)],
                               gseg=[(int(rng.integers(0, T // (16 * n) + 2)), int(rng.integers(0, T // (10 * n) + 2)))
                                     for _ in range(ng)]))
            style = len(sets) % 5
            for i, tk in enumerate(ts):
                tk["prio"] = [n - i, 1000 * (n - i) - 7, -(i + 1), (1 << 40) + (n - i), (n - i) // 3][style]
            sets.append(ts)
    # tiny periods, and one task with 70 segments of each kind (beyond the per-task fast limit)
    sets.append([dict(T=2, prio=3, core=0, cseg=[1]), dict(T=3, prio=2, core=0, cseg=[1]),
                 dict(T=40, prio=1, core=0, cseg=[1], gseg=[(0, 1)])])
    sets.append([dict(T=1, prio=3, core=0, cseg=[1]), dict(T=7, prio=2, core=0, cseg=[1])])
    sets.append([dict(T=100000, prio=2, core=0, cseg=[3] * 71, gseg=[(1, 2)] * 70),
                 dict(T=200000, prio=1, core=0, cseg=[5], gseg=[(1, 7)])])
    sets.append([dict(T=50000 + i, prio=i, core=i % 3, cseg=[2] * 12, gseg=[(1, 1)] * 11) for i in range(30)])
    b = batch_of(sets)
    for policy in ALL_MODES:
        for L, ovh in ((1024, 50), (1, 0), (lim, 1), (lim - 1, lim - 1), (3, 1 << 21)):
            assert_parity(b, policy, L, ovh, "limit L=%d ovh=%d" % (L, ovh))


def test_every_class_of_period_as_a_divisor():
    """The kernels divide by each interferer's period with a precomputed reciprocal.  Periods of
    every magnitude (powers of two and their neighbours, small values, random ones up to the
    32-bit path's limit) against dividends from a few thousand up to 2^26."""
    rng = np.random.default_rng(33)
    lim = 1 << 26
    periods = [2, 3, 4, 5, 6, 7, 8, 9, 15, 16, 17, 31, 33, 1000, 1023, 1024, 1025]
    periods += [(1 << k) + d for k in range(5, 26) for d in (-1, 0, 1)]
    periods += [lim - 1, lim - 2, lim - 3] + [int(x) for x in rng.integers(2, lim, 3000)]
    periods += [int(x) for x in np.exp(rng.uniform(np.log(2), np.log(lim), 3000))]
    sets = []
    for T in periods:
        T = max(2, min(lim - 1, T))
        own = int(rng.choice([5000, 1 << 20, 1 << 25]))
        ch = max(1, T // int(rng.integers(3, 9)))
        sets.append([dict(T=T, prio=3, core=0, cseg=[ch]),
                     dict(T=max(2, T // 2 + 1), prio=2, core=1, cseg=[1], gseg=[(0, max(1, T // 7))]),
                     dict(T=lim - 1, prio=1, core=0, cseg=[own], gseg=[(1, 1)])])
    b = batch_of(sets)
    for policy in MODES4:
        w, s = assert_parity(b, policy, 1024, 0, "divisors")
    assert (w[2::3] > 0).mean() > 0.5   # most of the low-priority tasks converge (many sweeps)


def test_arrays_that_start_on_odd_8_byte_boundaries():
    """Input arrays that are views starting 8 bytes into an allocation (so 16-byte loads cannot
    start at their first element), for batches whose slices touch both ends of the arrays."""
    for name, count in (("large", 40), ("sweep", 70), ("divergence", 300), ("pr1", 1)):
        w = taskgen.WORKLOADS[name]
        b = w.generate(11, count)
        tens = {}
        for f, arr in b.arrays().items():
            for shift in (1,):
                pad = torch.full((arr.shape[0] + 3,), (1 << 62) + 12345, dtype=torch.int64, device="cuda")
                pad[shift:shift + arr.shape[0]] = torch.from_numpy(arr).cuda()
                tens[f] = pad[shift:shift + arr.shape[0]]
        ts = binding.DeviceTasksets(tens)
        for policy in MODES4:
            w_ref, s_ref, _ = rta.analyse(b, policy, w.timeslice_us, w.overhead_us)
            wc, sc = binding.rta_batch(ts, policy, w.timeslice_us, w.overhead_us)
            torch.cuda.synchronize()
            assert (sc.cpu().numpy() == s_ref).all() and (wc.cpu().numpy() == w_ref).all(), (name, policy)


def test_determinism_and_output_reuse():
    b = taskgen.WORKLOADS["divergence"].generate(1000, 4000)
    ts = binding.DeviceTasksets.from_host(b)
    outs = []
    for _ in range(3):
        w, s = binding.rta_batch(ts, 0, 1024, 50)
        torch.cuda.synchronize()
        outs.append((w.cpu().numpy().copy(), s.cpu().numpy().copy()))
    for w, s in outs[1:]:
        assert (w == outs[0][0]).all() and (s == outs[0][1]).all()


def test_streams_and_workspace_errors():
    b = taskgen.WORKLOADS["pr1"].generate(0, 300)
    ts = binding.DeviceTasksets.from_host(b)
    w_ref, s_ref, _ = rta.analyse(b, 0, 1024, 50)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        w, s = binding.rta_batch(ts, 0, 1024, 50)
    side.synchronize()
    assert (w.cpu().numpy() == w_ref).all() and (s.cpu().numpy() == s_ref).all()
    tiny = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.GcapsError) as e:
        binding.rta_batch(ts, 0, 1024, 50, workspace=tiny)
    assert e.value.code == binding.ERR_WORKSPACE
    with pytest.raises(binding.GcapsError):
        binding.rta_batch(ts, 1, 0, 0)


def test_host_buffer_entry_point():
    """gcaps_rta_batch_host: chunked copies in, analysis, copies out -- same results."""
    b = taskgen.WORKLOADS["divergence"].generate(0, 150_000)   # several chunks
    for policy in (0, 1):
        w_ref, s_ref, _ = rta.analyse(b, policy, 1024, 50)
        w, s = binding.rta_batch_host(b.arrays(), policy, 1024, 50)
        assert (s == s_ref).all() and (w == w_ref).all()
    # pinned buffers, and a batch with malformed offsets in the middle
    small = taskgen.WORKLOADS["sweep"].generate(0, 500)
    pinned = {f: torch.from_numpy(a.copy()).pin_memory().numpy() for f, a in small.arrays().items()}
    w_ref, s_ref, _ = rta.analyse(small, 1 | BUSY, 512, 25)
    w, s = binding.rta_batch_host(pinned, 1 | BUSY, 512, 25)
    assert (s == s_ref).all() and (w == w_ref).all()
    broken = copy.deepcopy(small)
    broken.cseg_off[broken.task_off[200] + 3] = -7
    broken.task_off[400] = broken.task_off[399] - 1
    w_ref, s_ref, _ = rta.analyse(broken, 0, 512, 25)
    w, s = binding.rta_batch_host(broken.arrays(), 0, 512, 25)
    assert (s == s_ref).all() and (w == w_ref).all()
    # several analyses of one copy of the inputs
    pols = [0, 1, BUSY, 1 | BUSY | LITERAL]
    ws, ss = binding.rta_batch_host_multi(b.arrays(), pols, 1024, 50)
    for q, policy in enumerate(pols):
        w_ref, s_ref, _ = rta.analyse(b, policy, 1024, 50)
        assert (ss[q] == s_ref).all() and (ws[q] == w_ref).all(), policy
    ws, ss = binding.rta_batch_host_multi(broken.arrays(), [0, 1], 512, 25)
    for q, policy in enumerate([0, 1]):
        w_ref, s_ref, _ = rta.analyse(broken, policy, 512, 25)
        assert (ss[q] == s_ref).all() and (ws[q] == w_ref).all(), policy
    with pytest.raises(binding.GcapsError):
        binding.rta_batch_host_multi(small.arrays(), [0] * 9, 512, 25)
    binding.release_host()


def test_full_size_large_workload_sampled():
    """The benchmark's own configuration (1,000,000 tasksets of 80 tasks): outputs of sampled
    tasksets against the oracle, and properties that hold at any size for the rest."""
    w = taskgen.WORKLOADS["large"]
    b = w.generate(0, w.n_tasksets)
    ts = binding.DeviceTasksets.from_host(b)
    rng = np.random.default_rng(9)
    sample = np.sort(rng.choice(w.n_tasksets, 3000, replace=False))
    sub = b.select(sample)
    for policy in (0, 1):
        wc, sc = binding.rta_batch(ts, policy, w.timeslice_us, w.overhead_us)
        torch.cuda.synchronize()
        wc, sc = wc.cpu().numpy().reshape(-1, 80), sc.cpu().numpy()
        w_ref, s_ref, _ = rta.analyse(sub, policy, w.timeslice_us, w.overhead_us)
        assert (sc[sample] == s_ref).all()
        assert (wc[sample].reshape(-1) == w_ref).all()
        # any size: flags are 0/1; schedulable <=> no sentinel; at most one MISS per taskset
        assert sc.max() <= 1
        has_neg = (wc < 0).any(axis=1)
        assert ((sc == 1) == ~has_neg).all()
        assert ((wc == binding.WCRT_MISS).sum(axis=1) <= 1).all()
        D = b.deadline.reshape(-1, 80)
        ok = wc >= 0
        assert (wc[ok] <= D[ok]).all()


def _sampled_parity(batch, ts, policy, L, ovh, rng, n_sample, what):
    """Runs the library on the whole device batch and the oracle on a random sample of tasksets."""
    wc, sc = binding.rta_batch(ts, policy, L, ovh)
    torch.cuda.synchronize()
    wc, sc = wc.cpu().numpy(), sc.cpu().numpy()
    sample = np.sort(rng.choice(batch.n_tasksets, min(n_sample, batch.n_tasksets), replace=False))
    sub = batch.select(sample)
    w_ref, s_ref, _ = rta.analyse(sub, policy, L, ovh)
    assert (sc[sample] == s_ref).all(), what
    pos = np.concatenate([np.arange(batch.task_off[t], batch.task_off[t + 1]) for t in sample])
    assert (wc[pos] == w_ref).all(), what
    # properties that hold at any size
    assert sc.max() <= 1, what
    first = batch.task_off[:-1]
    nonempty = np.diff(batch.task_off) > 0
    has_neg = np.zeros(batch.n_tasksets, bool)
    has_neg[nonempty] = np.minimum.reduceat(wc, first[nonempty]) < 0
    assert ((sc == 1) == ~has_neg).all(), what
    ok = wc >= 0
    assert (wc[ok] <= batch.deadline[ok]).all(), what
    return sc


def test_full_size_schedulability_sweep_sampled():
    """All nine points of the utilisation sweep at 100,000 tasksets each, both policies."""
    w = taskgen.WORKLOADS["sweep"]
    rng = np.random.default_rng(17)
    ratio = {0: [], 1: []}
    for stream in range(len(w.streams)):
        b = w.generate(0, w.n_tasksets, stream=stream)
        ts = binding.DeviceTasksets.from_host(b)
        for policy in (0, 1):
            sc = _sampled_parity(b, ts, policy, w.timeslice_us, w.overhead_us, rng, 700,
                                 "sweep point %d policy %d" % (stream, policy))
            ratio[policy].append(float((sc == 1).mean()))
    # schedulability falls as the utilisation per core rises, and GCAPS stays above round robin
    for policy in (0, 1):
        assert ratio[policy][0] >= ratio[policy][-1]
    assert ratio[0][0] > 0.9 and ratio[0][0] > ratio[1][0]


def test_full_size_rr_driver_model_sweep_sampled():
    """200,000 tasksets under round robin for all 25 (time slice, context switch) pairs."""
    w = taskgen.WORKLOADS["rr_model"]
    rng = np.random.default_rng(18)
    b = w.generate(0, w.n_tasksets)
    ts = binding.DeviceTasksets.from_host(b)
    for L in w.timeslices:
        for theta in w.overheads:
            _sampled_parity(b, ts, 1, L, theta, rng, 300, "rr model L=%d theta=%d" % (L, theta))


def test_full_size_divergence_stress_sampled():
    """The 10,000,000-taskset divergence workload in chunks of 1,000,000, both policies."""
    w = taskgen.WORKLOADS["divergence"]
    rng = np.random.default_rng(19)
    chunk = 1_000_000
    for first in range(0, w.n_tasksets, chunk):
        b = w.generate(first, chunk)
        ts = binding.DeviceTasksets.from_host(b)
        for policy in (0, 1):
            _sampled_parity(b, ts, policy, w.timeslice_us, w.overhead_us, rng, 400,
                            "divergence chunk %d policy %d" % (first // chunk, policy))
        del ts
        torch.cuda.empty_cache()
