"""The oracle of the analysis with separate GPU-segment priorities (paper Sec. 5.3, 6.4)."""
import os

import numpy as np
import pytest

from oracle import rta, sim
from tests.helpers import BUSY, GOLDEN, batch_of, parse_vectors, random_tasksets

ASSIGN = rta.FLAG_ASSIGN


def gp_cases():
    out = []
    with open(os.path.join(GOLDEN, "table2_gpu_priority_vectors.txt")) as fh:
        for line in fh:
            tok = line.split("#", 1)[0].split()
            if not tok or tok[0] != "case":
                continue
            kv = dict(x.split("=", 1) for x in tok[2:])
            out.append(dict(name=tok[1], busy=kv["busy"] == "1", eps=int(kv["eps"]),
                            gpu=None if kv["gpu"] == "assign" else [int(x) for x in kv["gpu"].split(",")],
                            expect=[int(x) for x in kv["expect"].split(",")], sched=int(kv["sched"]),
                            levels=[int(x) for x in kv["levels"].split(",")] if "levels" in kv else None))
    return out


def test_table2_vectors_and_the_papers_assignment():
    tasks, _ = parse_vectors("table2_vectors.txt")
    b = batch_of([tasks])
    cases = gp_cases()
    assert len(cases) >= 7
    for c in cases:
        flags = (BUSY if c["busy"] else 0) | (ASSIGN if c["gpu"] is None else 0)
        w, s, gp = rta.analyse_gpu_priority(b, flags, c["eps"], gpu_priority=c["gpu"])
        assert w.tolist() == c["expect"] and s[0] == c["sched"], c["name"]
        if c["levels"]:
            assert gp.tolist() == c["levels"], c["name"]


def test_simulated_schedule_of_the_papers_assignment():
    """Fig. 5b: with GPU priority tau1 > tau2 > tau4 > tau3 every task meets its deadline in
    the drawn scenario (tau3 released at 70), and stays within the analytic bounds."""
    tasks, _ = parse_vectors("table2_vectors.txt")
    b = batch_of([tasks])
    w, s, _ = rta.analyse_gpu_priority(b, 0, 0, gpu_priority=[4, 3, 1, 2])
    resp, unf = sim.simulate(b, 0, [0, 0, 70, 0], 0, False, 4, 2000, gpu_priority=[4, 3, 1, 2])
    assert (unf <= w).all() and (resp <= w).all() and (resp <= b.deadline).all() and (resp > 0).all()


def _same_core_rule_holds(ts, gp):
    for i, ti in enumerate(ts):
        for q, tq in enumerate(ts):
            if ti["core"] == tq["core"] and tq["prio"] > ti["prio"] and gp[q] < gp[i]:
                return False
    return True


def test_assignment_invariants():
    """(a) D_h jitters can only raise a bound over the R_h jitters of Sec. 6.3; (b) whenever the
    CPU priorities pass as GPU priorities the search succeeds; (c) what the search returns keeps
    the same-core order, is a permutation of 1..n and reproduces its bounds when analysed as
    given; (d) it never does worse than the CPU priorities."""
    rng = np.random.default_rng(41)
    found_gain = 0
    for ts in random_tasksets(rng, 500, max_tasks=7, max_cores=3, wcet_hi=7):
        b = batch_of([ts])
        prio = [tk["prio"] for tk in ts]
        for busy in (0, BUSY):
            for eps in (0, 1):
                w0, s0, _ = rta.analyse(b, 0 | busy, 4, eps)
                wd, sd, _ = rta.analyse_gpu_priority(b, busy, eps, gpu_priority=prio)
                if s0[0] == 1:
                    assert all(x >= y for x, y in zip(wd, w0) if x >= 0)          # (a)
                wa, sa, gp = rta.analyse_gpu_priority(b, busy | ASSIGN, eps)
                if sd[0] == 1:
                    assert sa[0] == 1                                              # (b), (d)
                if sa[0] == 1:
                    assert sorted(gp.tolist()) == list(range(1, len(ts) + 1))
                    assert _same_core_rule_holds(ts, gp)
                    wr, sr, _ = rta.analyse_gpu_priority(b, busy, eps, gpu_priority=gp)
                    assert sr[0] == 1 and wr.tolist() == wa.tolist()               # (c)
                    found_gain += int(sd[0] == 0)
                else:
                    assert (wa == rta.WCRT_MISS).any() and (gp == 0).any()
    assert found_gain > 5   # the search rescues tasksets the CPU priorities fail


def test_rule_violation_and_lone_task():
    ts = [dict(T=100, prio=2, core=0, cseg=[5], gseg=[(1, 3)]), dict(T=100, prio=1, core=0, cseg=[5], gseg=[(1, 3)])]
    w, s, _ = rta.analyse_gpu_priority(batch_of([ts]), 0, 0, gpu_priority=[1, 2])
    assert s[0] == rta.SCHED_INVALID and (w == rta.WCRT_INVALID).all()
    lone = [dict(T=1000, prio=1, core=0, cseg=[5, 6], gseg=[(1, 3)])]
    for eps in (0, 7):
        w, s, gp = rta.analyse_gpu_priority(batch_of([lone]), ASSIGN, eps)
        assert w.tolist() == [15 + 4 * eps] and s[0] == 1 and gp.tolist() == [1]


def test_bounds_hold_in_simulation_with_assigned_priorities():
    rng = np.random.default_rng(43)
    checked = 0
    periods = [8, 10, 12, 15, 16, 20, 24, 30, 40]
    for _ in range(1200):
        n = int(rng.integers(2, 5))
        ts = []
        for _i in range(n):
            T = int(rng.choice(periods))
            ng = int(rng.integers(0, 3))
            cs = [int(rng.integers(0, 3)) for _ in range(ng + 1)]
            cs[0] = max(cs[0], 1)
            ts.append(dict(T=T, prio=0, core=int(rng.integers(0, 2)), cseg=cs,
                           gseg=[(int(rng.integers(0, 2)), int(rng.integers(1, 5))) for _ in range(ng)]))
        for r, i in enumerate(sorted(range(n), key=lambda i: (ts[i]["T"], i))):
            ts[i]["prio"] = n - r
        b = batch_of([ts])
        for busy in (False, True):
            w, s, gp = rta.analyse_gpu_priority(b, ASSIGN | (BUSY if busy else 0), 0)
            if s[0] != 1:
                continue
            checked += 1
            hyper = int(np.lcm.reduce(b.period))
            for trial in range(6):
                off = [0] * n if trial == 0 else [int(rng.integers(0, t["T"])) for t in ts]
                resp, unf = sim.simulate(b, 0, off, 0, busy, 1, 2 * hyper + max(off) + 1, gpu_priority=gp)
                assert (resp <= w).all() and (unf <= w).all(), (ts, gp, off, w, resp)
    assert checked > 300


def test_jitter_of_a_task_that_cannot_meet_its_own_deadline_is_zero():
    """Sec. 6.4 puts D_h where Sec. 6.3 has R_h, which presumes R_h <= D_h.  tau_h here needs
    C + G^m = 35 > D = 20: J^c_h is taken as 0, not -15.  By hand for the lower task (eps = 0):
    R = 6 + ceil(R/40)*35 + ceil((R+17)/40)*3 -> 6, 44, 82, 120, 123, 158, 161, 196, 199, 199."""
    sets = [[dict(T=40, D=20, prio=2, core=0, cseg=[30], gseg=[(5, 3)]),
             dict(T=400, D=400, prio=1, core=0, cseg=[3], gseg=[(1, 2)])]]
    b = batch_of(sets)
    wcrt, sched, _ = rta.analyse_gpu_priority(b, 0, 0, gpu_priority=np.array([2, 1]))
    assert wcrt.tolist() == [rta.WCRT_MISS, 199] and sched.tolist() == [0]
    # far below zero: still no negative term (base + 35 per job of tau_h at least)
    sets[0][0]["cseg"] = [3000]
    wcrt, _, _ = rta.analyse_gpu_priority(batch_of(sets), 0, 0, gpu_priority=np.array([2, 1]))
    assert wcrt.tolist() == [rta.WCRT_MISS, rta.WCRT_MISS]
