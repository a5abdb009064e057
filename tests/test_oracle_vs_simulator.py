"""Brute force: on tiny tasksets no simulated schedule may exceed the oracle's bounds.

Two sweeps: random release-offset vectors on many tasksets, and every offset vector on a grid
of one tick over two hyperperiods on three-task tasksets.  Overheads are zero here: with theta > 0 or eps > 0 the tick simulator does not model the
context-switch and runlist-update costs, so those cases are pinned by the closed forms, the
monotonicity tests and the hand-derived vectors instead.
"""
import numpy as np
import pytest

from oracle import rta, sim
from tests.helpers import BUSY, batch_of

PERIODS = [8, 10, 12, 15, 16, 20, 24, 30, 40]


def tiny_taskset(rng):
    n = int(rng.integers(2, 5))
    cores = int(rng.integers(1, 3))
    ts = []
    for _ in range(n):
        T = int(rng.choice(PERIODS))
        ng = int(rng.integers(0, 3))
        cs = [int(rng.integers(0, 3)) for _ in range(ng + 1)]
        if sum(cs) == 0:
            cs[0] = 1
        gs = [(int(rng.integers(0, 2)), int(rng.integers(1, 5))) for _ in range(ng)]
        ts.append(dict(T=T, prio=0, core=int(rng.integers(0, cores)), cseg=cs, gseg=gs))
    order = sorted(range(n), key=lambda i: (ts[i]["T"], i))
    for r, i in enumerate(order):
        ts[i]["prio"] = n - r
    return ts


@pytest.mark.parametrize("policy,busy", [(0, False), (0, True), (1, False), (1, True)])
def test_observed_response_never_exceeds_bound(policy, busy):
    rng = np.random.default_rng(100 + policy * 2 + int(busy))
    checked = tight = 0
    for _ in range(1500):
        ts = tiny_taskset(rng)
        b = batch_of([ts])
        n = len(ts)
        L = int(rng.integers(1, 4))
        wcrt, sched, _ = rta.analyse(b, policy | (BUSY if busy else 0), L, 0)
        if sched[0] != rta.SCHED_YES:
            continue
        checked += 1
        hyper = int(np.lcm.reduce(b.period))
        worst = np.zeros(n, np.int64)
        for trial in range(10):
            off = [0] * n if trial == 0 else [int(rng.integers(0, t["T"])) for t in ts]
            resp, unfinished = sim.simulate(b, 0, off, policy, busy, L, 2 * hyper + max(off) + 1)
            assert (resp <= wcrt).all() and (unfinished <= wcrt).all(), (ts, off, L, wcrt, resp)
            worst = np.maximum(worst, resp)
        tight += int((worst == wcrt).sum())
    assert checked > 300
    assert tight > checked  # the bounds are reached exactly for many tasks: the check has teeth


def chain_taskset(rng):
    """tau_x alone on core 1 (highest priority, one long pure-GPU part, long period) delays the
    GPU part of tau_h; tau_i runs below tau_h on tau_h's core and is CPU-only in half the cases.
    A late GPU part of one job of tau_h followed by an undelayed next job puts more than one
    job's worth of tau_h's CPU demand into a window shorter than T_h: the situation the
    self-suspension jitters J^c_h, J^g_h of Sec. 6.2.2 / 6.3 account for."""
    Th = int(rng.choice([8, 10, 12, 15]))
    Tx, Ti = int(rng.choice([20, 24, 30])), int(rng.choice([20, 24, 30]))
    x = dict(T=Tx, prio=3, core=1, cseg=[int(rng.integers(0, 2))], gseg=[(0, int(rng.integers(2, 8)))])
    h = dict(T=Th, prio=2, core=0, cseg=[int(rng.integers(0, 3)), int(rng.integers(1, 4))],
             gseg=[(int(rng.integers(0, 2)), int(rng.integers(1, 4)))])
    if rng.integers(0, 2):
        i = dict(T=Ti, prio=1, core=0, cseg=[int(rng.integers(1, 5))], gseg=[])
    else:
        i = dict(T=Ti, prio=1, core=0, cseg=[int(rng.integers(0, 3)), int(rng.integers(0, 3))],
                 gseg=[(int(rng.integers(0, 2)), int(rng.integers(1, 4)))])
    return [x, h, i]


def classic_bound(C, hp, limit):
    """Textbook fixed-priority response time C + sum ceil(R/T_h) * C_h (no jitter)."""
    R = C
    while R <= limit:
        nxt = C + sum(-(-R // T) * Ch for T, Ch in hp)
        if nxt == R:
            return R
        R = nxt
    return None


@pytest.mark.parametrize("policy,busy", [(0, False), (0, True), (1, False), (1, True)])
def test_every_release_offset_over_two_hyperperiods(policy, busy):
    """Brute force in full: EVERY vector of release offsets (grid of one tick, below the periods)
    over two hyperperiods, on tasksets of three tasks.  No observed response may exceed a bound.
    In the self-suspension modes the sweep also has to find schedules in which a CPU-only tau_i
    is delayed longer than the jitter-free textbook bound over tau_h allows, i.e. schedules that
    only the jitter J^c_h covers: a bound that lost that jitter would be exceeded here."""
    rng = np.random.default_rng(900 + policy * 2 + int(busy))
    checked = runs = tight = beyond_classic = 0
    families = [chain_taskset] * 200 + [tiny_taskset] * 120
    for make in families:
        ts = make(rng)[:3]
        b = batch_of([ts])
        if int(np.lcm.reduce(b.period)) > 240:
            continue
        L = int(rng.integers(1, 4))
        wcrt, sched, _ = rta.analyse(b, policy | (BUSY if busy else 0), L, 0)
        if sched[0] != rta.SCHED_YES:
            continue
        checked += 1
        worst, r = sim.sweep_offsets(b, 0, policy, busy, L, step=1)
        runs += r
        assert (worst <= wcrt).all(), (ts, L, wcrt, worst)
        tight += int((worst == wcrt).sum())
        if make is chain_taskset and not busy and not ts[2]["gseg"]:
            h = ts[1]
            free = classic_bound(sum(ts[2]["cseg"]), [(h["T"], sum(h["cseg"]) + h["gseg"][0][0])],
                                 ts[2]["T"])
            if free is not None and worst[2] > free:
                beyond_classic += 1
    assert checked > 60 and runs > 200000
    assert tight > checked
    if not busy:
        assert beyond_classic >= 3, beyond_classic


def test_simulator_basics():
    """One task alone: response = sum of its segments; two CPU-only tasks on one core: the
    classic critical instant."""
    b = batch_of([[dict(T=50, prio=1, core=0, cseg=[2, 3], gseg=[(1, 4)])]])
    for pol in (0, 1):
        for busy in (False, True):
            resp, unf = sim.simulate(b, 0, [3], pol, busy, 2, 200)
            assert resp.tolist() == [10] and unf.tolist() == [0]
    b = batch_of([[dict(T=5, prio=2, core=0, cseg=[2]), dict(T=20, prio=1, core=0, cseg=[5])]])
    resp, _ = sim.simulate(b, 0, [0, 0], 0, False, 2, 200)
    assert resp.tolist() == [2, 9]
    # round robin with slice 2: two equal 4-tick GPU parts interleave 2+2+2+2
    b = batch_of([[dict(T=50, prio=2, core=0, cseg=[1], gseg=[(0, 4)]),
                   dict(T=50, prio=1, core=1, cseg=[1], gseg=[(0, 4)])]])
    resp, _ = sim.simulate(b, 0, [0, 0], 1, False, 2, 200)
    assert resp.tolist() == [1 + 6, 1 + 8]
    resp, _ = sim.simulate(b, 0, [0, 0], 0, False, 2, 200)   # GCAPS: strict priority
    assert resp.tolist() == [1 + 4, 1 + 8]
