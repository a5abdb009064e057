"""Pins of the oracle's best-effort reading (tasks without a real-time priority, Sec. 7.1's last
experiment and Table 4): hand-derived vectors, the case-study rows of Table 5, and properties
that hold for any taskset."""
import copy

import numpy as np
import pytest

from oracle import rta
from tests.helpers import ALL_MODES, BEST_EFFORT, batch_of, parse_vectors, random_tasksets
from tests.test_oracle_golden import _table5


def test_hand_derived_vectors():
    tasks, cases = parse_vectors("table2_best_effort_vectors.txt")
    assert len(cases) == 6
    b = batch_of([tasks])
    for c in cases:
        wcrt, sched, _ = rta.analyse(b, c["policy"], c["L"], c["ovh"])
        assert wcrt.tolist() == c["expect"], c["name"]
        rt = [x for x in c["expect"] if x != rta.WCRT_BEST_EFFORT]
        assert sched[0] == (1 if min(rt) >= 0 else 0), c["name"]


def test_case_study_rows_with_the_two_best_effort_tasks_flagged():
    """Table 4 lists tasks 6 and 7 without a real-time priority.  Flagged as best-effort they get
    no bound, and the rows of tasks 1..5 are the ones the unflagged run gives when the two sit at
    the bottom of the priority order -- including task 1 under round robin, 11 + 1.224*5*8 =
    59.96 ms (the printed 60), where the 5 counts both best-effort tasks."""
    rows, paper = _table5()
    tasks = []
    for C, G, T, core, prio in rows:
        C, G, T = int(C * 1000), int(G * 1000), int(T * 1000)
        seg = dict(cseg=[C // 2, C - C // 2], gseg=[(G // 5, G - G // 5)]) if G else dict(cseg=[C])
        tasks.append(dict(T=T, prio=int(prio), core=int(core), **seg))
    b = batch_of([tasks])
    for pol, ovh in ((1, 200), (1 | 0x100, 200), (0, 1250), (0 | 0x100, 1250)):
        plain, _, _ = rta.analyse(b, pol, 1024, ovh)
        flagged, sched, _ = rta.analyse(b, pol | BEST_EFFORT, 1024, ovh)
        assert flagged[:5].tolist() == plain[:5].tolist()
        assert flagged[5:].tolist() == [rta.WCRT_BEST_EFFORT] * 2
        assert sched[0] == (1 if (flagged[:5] >= 0).all() else 0)
    assert rta.analyse(b, 1 | BEST_EFFORT, 1024, 200)[0][0] == 59960
    # the failing row of Table 5 (round robin, busy-waiting) still fails at task 5
    assert rta.analyse(b, 1 | 0x100 | BEST_EFFORT, 1024, 200)[0][4] == rta.WCRT_MISS
    # GCAPS accepts the real-time part of the case study, as Table 5 does
    assert rta.analyse(b, 0 | BEST_EFFORT, 1024, 1250)[1][0] == 1


def _demote(tasksets, rng):
    """Gives the lowest-priority tasks of every taskset (a random number of them) priorities
    0, -1, ... in their old order; returns the new tasksets and the best-effort masks."""
    out, masks = [], []
    for ts in tasksets:
        ts = copy.deepcopy(ts)
        order = sorted(range(len(ts)), key=lambda i: (-ts[i]["prio"], i))
        for i in ts:
            i["prio"] += 1000            # real-time priorities are positive
        k = int(rng.integers(0, len(ts) + 1))
        mask = [False] * len(ts)
        for r, i in enumerate(order[len(ts) - k:]):
            ts[i]["prio"] = -r
            mask[i] = True
        out.append(ts)
        masks.append(mask)
    return out, masks


@pytest.mark.parametrize("policy", ALL_MODES)
def test_real_time_tasks_see_best_effort_tasks_only_through_the_gpu_count(policy):
    rng = np.random.default_rng(40 + policy)
    sets, masks = _demote(random_tasksets(rng, 400, max_tasks=8, max_cores=3), rng)
    b = batch_of(sets)
    be = np.concatenate([np.array(m, bool) for m in masks if m]) if b.n_tasks else np.zeros(0, bool)
    for L, ovh in ((3, 0), (5, 2)):
        plain, _, _ = rta.analyse(b, policy, L, ovh)
        flagged, sched, _ = rta.analyse(b, policy | BEST_EFFORT, L, ovh)
        # best-effort tasks sit below every real-time task, so flagging them changes nothing above
        assert (flagged[~be] == plain[~be]).all()
        assert (flagged[be] == rta.WCRT_BEST_EFFORT).all()
        off = b.task_off
        for t in range(b.n_tasksets):
            rt = flagged[off[t]:off[t + 1]][~be[off[t]:off[t + 1]]]
            assert sched[t] == (1 if (rt >= 0).all() else 0)
        # deleting the best-effort tasks: no change under GCAPS; under round robin only their
        # share of the time-sliced GPU goes away, so no bound grows
        kept = [[x for x, m in zip(ts, mk) if not m] for ts, mk in zip(sets, masks)]
        alone, s_alone, _ = rta.analyse(batch_of(kept), policy, L, ovh)
        if (policy & 0xff) == 0:
            assert (alone == flagged[~be]).all()
        else:
            both = (alone >= 0) & (flagged[~be] >= 0)
            assert (alone[both] <= flagged[~be][both]).all()
            assert (s_alone >= sched).all()


def test_cpu_only_best_effort_tasks_change_nothing_and_gpu_ones_do_under_round_robin():
    rt = [dict(T=100, prio=5, core=0, cseg=[10], gseg=[(1, 8)]),
          dict(T=200, prio=4, core=0, cseg=[20], gseg=[(2, 6)])]
    be_cpu = dict(T=50, prio=0, core=0, cseg=[40])
    be_gpu = dict(T=50, prio=0, core=1, cseg=[1], gseg=[(1, 30)])
    for policy in (1, 1 | 0x100):
        base, _, _ = rta.analyse(batch_of([rt]), policy | BEST_EFFORT, 4, 1)
        with_cpu, _, _ = rta.analyse(batch_of([rt + [be_cpu]]), policy | BEST_EFFORT, 4, 1)
        with_gpu, _, _ = rta.analyse(batch_of([rt + [be_gpu]]), policy | BEST_EFFORT, 4, 1)
        assert with_cpu[:2].tolist() == base.tolist()
        # Lemma 1: (L + theta) * (N_g - 1) * slices grows from 5*1*2 to 5*2*2 for the first task
        assert with_gpu[0] - base[0] == 5 * 2
        assert with_gpu[1] > base[1]


def test_flag_is_rejected_nowhere_and_empty_real_time_part_is_schedulable():
    only_be = [dict(T=10, prio=0, core=0, cseg=[100], gseg=[(50, 50)])]   # would miss if analysed
    for policy in ALL_MODES:
        w, s, _ = rta.analyse(batch_of([only_be]), policy | BEST_EFFORT, 4, 0)
        assert w.tolist() == [rta.WCRT_BEST_EFFORT] and s.tolist() == [1]
