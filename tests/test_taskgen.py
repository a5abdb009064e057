"""The seeded input generator: determinism, slicing and the shape of the five workloads."""
import numpy as np
import pytest

from oracle import rta
from paper_2406_05221_b200 import taskgen as tg


def test_any_slice_can_be_generated_alone():
    w = tg.WORKLOADS["divergence"]
    full = w.generate(0, 300)
    part = w.generate(120, 50)
    assert full.slice(120, 170).checksum() == part.checksum()
    assert tg.TasksetBatch.concat([full.slice(0, 7), full.slice(7, 300)]).checksum() == full.checksum()
    assert w.generate(0, 300).checksum() == full.checksum()
    picked = full.select([5, 200, 17])
    assert picked.n_tasksets == 3
    assert np.array_equal(picked.slice(1, 2).period, w.generate(200, 1).period)


@pytest.mark.parametrize("name,n_tasks,cores", [("pr1", 8, 2), ("sweep", 20, 4), ("large", 80, 8),
                                                ("rr_model", 24, 4)])
def test_fixed_shape_workloads(name, n_tasks, cores):
    w = tg.WORKLOADS[name]
    b = w.generate(0, 200, stream=len(w.streams) - 1)
    assert b.n_tasksets == 200 and b.n_tasks == 200 * n_tasks
    assert (np.diff(b.task_off) == n_tasks).all()
    assert rta.validate(b).max() == 0
    assert b.core.min() == 0 and b.core.max() == cores - 1
    p = w.streams[0]
    assert b.period.min() >= p.period_us[0] and b.period.max() <= p.period_us[1]
    assert (b.deadline == b.period).all()
    # rate-monotonic, unique priorities 1..n
    pr = b.priority.reshape(200, n_tasks)
    T = b.period.reshape(200, n_tasks)
    assert (np.sort(pr, axis=1) == np.arange(1, n_tasks + 1)).all()
    for k in range(5):
        order = np.argsort(-pr[k])
        assert (np.diff(T[k][order]) >= 0).all()
    eta = np.diff(b.gseg_off)
    assert (np.diff(b.cseg_off) == eta + 1).all()
    want_gpu = round(p.gpu_frac * n_tasks)
    per_set = (eta.reshape(200, n_tasks) > 0).sum(axis=1)
    assert per_set.max() <= want_gpu and per_set.mean() > 0.7 * want_gpu
    assert eta.max() <= p.gpu_segments[1]
    assert (b.cseg_wcet >= 1).all() and (b.gseg_exec >= 1).all() and (b.gseg_misc >= 0).all()


def test_utilisation_matches_the_request():
    w = tg.WORKLOADS["sweep"]
    for stream in (0, 4, 8):
        b = w.generate(0, 500, stream=stream)
        C = np.add.reduceat(b.cseg_wcet, b.cseg_off[:-1])
        G = np.zeros(b.n_tasks, np.int64)
        has = np.diff(b.gseg_off) > 0
        G[has] = np.add.reduceat(b.gseg_misc + b.gseg_exec, b.gseg_off[:-1][has])
        util = ((C + G) / b.period).reshape(500, 20).sum(axis=1)
        want = 4 * 0.1 * (stream + 1)
        assert abs(util.mean() - want) < 0.02 * want + 0.005
        # worst-fit decreasing keeps the cores balanced
        per_core = np.zeros((500, 4))
        u = ((C + G) / b.period).reshape(500, 20)
        for c in range(4):
            per_core[:, c] = np.where(b.core.reshape(500, 20) == c, u, 0).sum(axis=1)
        assert (per_core.max(axis=1) - per_core.min(axis=1)).mean() < 0.35 * want / 4 + 0.02


def test_divergence_workload_is_ragged():
    b = tg.WORKLOADS["divergence"].generate(0, 2000)
    n = np.diff(b.task_off)
    assert n.min() >= 4 and n.max() <= 192 and n.min() < 12 and n.max() > 120
    assert rta.validate(b).max() == 0
    eta = np.diff(b.gseg_off)
    assert eta.min() == 0 and eta.max() == 8
    assert b.period.min() >= 100 and b.period.max() <= 10_000_000
