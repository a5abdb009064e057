"""The integer-only taskset generator (csrc/igen.h, host build) against its oracle
(oracle/igen_oracle.py, plain Python integers), and the oracle against what fixes it: the exact
value of 2^y and what the generation procedure of the paper's Sec. 7.1 / Table 3 states (ranges,
sums, rate-monotonic priorities, worst-fit-decreasing allocation).  The generator holds none of
the analysis arithmetic."""
import ctypes
import math

import numpy as np
import pytest

from paper_2406_05221_b200 import taskgen

from oracle.igen_oracle import exp2_q32, reference_taskset


STREAMS = [("pr1", 0), ("sweep", 0), ("sweep", 6), ("large", 0), ("rr_model", 0), ("divergence", 0)]


@pytest.mark.parametrize("name,stream", STREAMS)
def test_host_build_against_the_python_restatement(name, stream):
    w = taskgen.WORKLOADS[name]
    first, count = 12345, 40 if name in ("large", "divergence") else 150
    got = w.generate(first, count, stream=stream, integer=True)
    p = w.streams[stream].int_params()
    want = taskgen.TasksetBatch.from_tasksets([reference_taskset(p, first + t) for t in range(count)])
    for f in taskgen.ARRAY_FIELDS:
        assert np.array_equal(getattr(got, f), getattr(want, f)), f


def test_exp2_is_the_rounded_power_of_two():
    lib = taskgen._load()
    rng = np.random.default_rng(3)
    ys = [0, 1, (1 << 32) - 1, 1 << 32, (23 << 32) + 12345, 29 << 32] + [int(x) for x in rng.integers(0, 30 << 32, 3000)]
    for y in ys:
        got = int(lib.ig_exp2(y))
        assert got == exp2_q32(y)
        # the fraction is cut to 24 bits and the product of roots is truncated: the result stays
        # within one part in 2^23 (and within one unit) of the real power
        real = 2.0 ** (y / 4294967296.0)
        assert abs(got - real) <= 0.5 + real * 2.0 ** -23 + 1e-9 * real, (y, got, real)
    assert int(lib.ig_exp2(10 << 32)) == 1024 and int(lib.ig_exp2(q := (10 << 32) + (1 << 31))) == round(1024 * math.sqrt(2))


@pytest.mark.parametrize("name,stream", STREAMS)
def test_what_the_generation_procedure_fixes(name, stream):
    w = taskgen.WORKLOADS[name]
    g = w.streams[stream]
    b = w.generate(0, 4000, stream=stream, integer=True)
    n = np.diff(b.task_off)
    assert n.min() >= g.cores[0] * g.tasks_per_core[0] and n.max() <= g.cores[1] * g.tasks_per_core[1]
    assert b.period.min() >= g.period_us[0] and b.period.max() <= g.period_us[1]
    assert np.array_equal(b.deadline, b.period)
    eta = np.diff(b.gseg_off)
    assert np.array_equal(np.diff(b.cseg_off), eta + 1)           # eta + 1 CPU segments
    assert eta.max() <= g.gpu_segments[1]
    assert b.cseg_wcet.min() >= 1 and (b.gseg_misc + b.gseg_exec).min() >= 1
    assert np.array_equal(b.gseg_misc, (b.gseg_misc + b.gseg_exec) // 5)  # 20 % / 80 %
    # demand per task and utilisation per taskset
    C = np.add.reduceat(b.cseg_wcet, b.cseg_off[:-1])
    G = np.zeros_like(C)
    has = eta > 0
    G[has] = np.add.reduceat(b.gseg_misc + b.gseg_exec, b.gseg_off[:-1][has])
    assert ((C + G) <= b.period).all()
    u = (C + G) / b.period
    per_set = np.add.reduceat(u, b.task_off[:-1])
    cores_mid = 0.5 * (g.cores[0] + g.cores[1])
    want = cores_mid * 0.5 * (g.util_per_core[0] + g.util_per_core[1])
    assert abs(per_set.mean() - want) < 0.03 * want + 0.02
    if g.gpu_mode == 0:
        # exactly round(share * n) tasks are picked; one whose demand is below 3 us cannot hold a
        # GPU segment between two CPU segments and stays CPU-only
        picked = np.add.reduceat(has.astype(np.int64), b.task_off[:-1])
        want_gpu = np.floor(g.gpu_frac * n + 0.5).astype(np.int64)
        assert (picked <= want_gpu).all() and picked.sum() > 0.98 * want_gpu.sum()
        ratio = (G[has] / (C + G)[has])
        assert g.gpu_ratio[0] - 0.05 < ratio.mean() < g.gpu_ratio[1] + 0.05
    # log-uniform periods: the mean of log2 T sits in the middle of the range (non-harmonic sets)
    if g.harmonic_frac == 0:
        mid = 0.5 * (math.log2(g.period_us[0]) + math.log2(g.period_us[1]))
        assert abs(np.log2(b.period).mean() - mid) < 0.05
        edges = np.linspace(math.log2(g.period_us[0]), math.log2(g.period_us[1]), 9)
        hist, _ = np.histogram(np.log2(b.period), edges)
        assert hist.min() > 0.85 * hist.mean() and hist.max() < 1.15 * hist.mean()
    # rate-monotonic, unique priorities 1..n inside every taskset
    for t in range(0, 200):
        a, e = b.task_off[t], b.task_off[t + 1]
        pr, T = b.priority[a:e], b.period[a:e]
        assert sorted(pr.tolist()) == list(range(1, e - a + 1))
        order = np.argsort(-pr, kind="stable")
        assert (np.diff(T[order]) >= 0).all()
        if g.wfd:   # worst fit decreasing keeps the cores' loads close together
            load = np.bincount(b.core[a:e], weights=u[a:e], minlength=g.cores[1])
            assert load.max() - load.min() <= u[a:e].max() + 1e-9


def test_uniform_spacings_give_exchangeable_shares():
    """The split of a CPU's utilisation is uniform on the simplex (what UUniFast draws): every
    position has mean U/m, and the largest share of m = 4 has mean (1 + 1/2 + 1/3 + 1/4) / 4."""
    w = taskgen.WORKLOADS["pr1"]           # 2 cores x 4 tasks, U = 0.5 per core
    b = w.generate(0, 20000, integer=True)
    C = np.add.reduceat(b.cseg_wcet, b.cseg_off[:-1])
    G = np.zeros_like(C)
    has = np.diff(b.gseg_off) > 0
    G[has] = np.add.reduceat(b.gseg_misc + b.gseg_exec, b.gseg_off[:-1][has])
    share = ((C + G) / b.period).reshape(-1, 2, 4) / 0.5
    assert np.abs(share.mean(axis=(0, 1)) - 0.25).max() < 0.005
    assert abs(share.max(axis=2).mean() - (1 + 1 / 2 + 1 / 3 + 1 / 4) / 4) < 0.005


def test_any_slice_can_be_generated_alone():
    w = taskgen.WORKLOADS["divergence"]
    whole = w.generate(100, 300, integer=True)
    part = w.generate(250, 50, integer=True)
    sub = whole.select(range(150, 200))
    for f in taskgen.ARRAY_FIELDS:
        assert np.array_equal(getattr(part, f), getattr(sub, f)), f
    assert whole.checksum() != w.generate(100, 300).checksum()   # not the floating-point stream
