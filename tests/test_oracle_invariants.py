"""The oracle against closed forms, special cases and invariants of the analysis."""
import copy

import numpy as np
import pytest

from oracle import rta
from tests.helpers import ALL_MODES, BUSY, LITERAL, batch_of, random_tasksets


def run(tasksets, policy, L=3, ovh=0, **kw):
    return rta.analyse(batch_of(tasksets), policy, L, ovh, **kw)


def sums(tk):
    C = sum(tk.get("cseg", []))
    Gm = sum(m for m, _ in tk.get("gseg", []))
    Ge = sum(e for _, e in tk.get("gseg", []))
    return C, Gm, Ge, len(tk.get("gseg", []))


def classic_rta(tasks, own_extra=0):
    """Textbook fixed-priority response-time analysis (Joseph & Pandya / Audsley et al.) of
    CPU-only tasks on partitioned cores: R = C + sum_{hp, same core} ceil(R/T_h) C_h.
    ``own_extra`` is added to the cost of the task under analysis only."""
    n = len(tasks)
    order = sorted(range(n), key=lambda i: (-tasks[i]["prio"], i))
    out = [None] * n
    for pos, i in enumerate(order):
        Ci = sum(tasks[i]["cseg"]) + own_extra
        hp = [h for h in order[:pos] if tasks[h]["core"] == tasks[i]["core"]]
        R = Ci
        while True:
            nxt = Ci + sum(-(-R // tasks[h]["T"]) * sum(tasks[h]["cseg"]) for h in hp)
            if nxt == R or R > tasks[i]["D"]:
                break
            R = nxt
        out[i] = R if R <= tasks[i]["D"] else None
    return out


def test_lone_task_closed_forms():
    """A lone task: RR gives C+G for any L, theta (Lemma 1 with an empty interleaving set);
    GCAPS gives C + G + 2*eps*eta + (eta+1)*eps (Sec. 6.3 G*, Lemma 8)."""
    rng = np.random.default_rng(1)
    for ts in random_tasksets(rng, 200, max_tasks=1):
        tk = ts[0]
        tk["D"] = tk["T"] = 10_000
        C, Gm, Ge, eta = sums(tk)
        for pol in ALL_MODES:
            for ovh in (0, 1, 7):
                w, s, _ = run([ts], pol, L=int(rng.integers(1, 9)), ovh=ovh)
                want = C + Gm + Ge + ((3 * eta + 1) * ovh if pol & 1 == 0 else 0)
                assert w[0] == want and s[0] == 1


def _expect_in_order(ts, want):
    order = sorted(range(len(ts)), key=lambda i: (-ts[i]["prio"], i))
    out, missed = [None] * len(ts), False
    for i in order:
        if missed:
            out[i] = rta.WCRT_SKIPPED
        elif want[i] is None:
            out[i], missed = rta.WCRT_MISS, True
        else:
            out[i] = want[i]
    return out


def test_cpu_only_reduces_to_classic_rta():
    """No GPU segments, zero overhead: every analysis is the classic RTA (the printed Lemma 7
    is the exception: it keeps a jitter R_h - C_h for CPU-only tasks, so it can only be larger).
    GCAPS with eps > 0 adds Lemma 8's single eps to the cost of the task under analysis."""
    rng = np.random.default_rng(2)
    misses = 0
    for ts in random_tasksets(rng, 400, max_gseg=0, wcet_hi=9):
        want = _expect_in_order(ts, classic_rta(ts))
        misses += rta.WCRT_MISS in want
        for pol in ALL_MODES:
            w, s, _ = run([ts], pol, ovh=0)
            if pol == (1 | LITERAL):
                assert all(a >= b for a, b in zip(w.tolist(), want) if a >= 0 and b >= 0)
            else:
                assert w.tolist() == want
        want5 = _expect_in_order(ts, classic_rta(ts, own_extra=5))
        for pol in (0, BUSY, LITERAL, BUSY | LITERAL):
            w, s, _ = run([ts], pol, ovh=5)
            assert w.tolist() == want5
    assert misses > 20


def test_highest_priority_task_and_bounds():
    """The top-priority task has no interferer: R = base.  Every converged R_i lies in
    [C_i + G_i, D_i]."""
    rng = np.random.default_rng(3)
    for ts in random_tasksets(rng, 300):
        for pol in ALL_MODES:
            L, ovh = int(rng.integers(1, 6)), int(rng.integers(0, 4))
            w, s, _ = run([ts], pol, L, ovh)
            top = min(range(len(ts)), key=lambda i: (-ts[i]["prio"], i))
            C, Gm, Ge, eta = sums(ts[top])
            n_gpu = sum(1 for tk in ts if tk.get("gseg"))
            if pol & 1 == 0:
                base = C + Gm + Ge + (3 * eta + 1) * ovh
            else:
                slices = sum(-(-e // L) for _, e in ts[top].get("gseg", []))
                base = C + Gm + Ge + (L + ovh) * (n_gpu - 1) * slices * (1 if eta else 0)
            assert w[top] == (base if base <= ts[top]["D"] else rta.WCRT_MISS)
            for i, tk in enumerate(ts):
                if w[i] >= 0:
                    C, Gm, Ge, _ = sums(tk)
                    assert C + Gm + Ge <= w[i] <= tk["D"]
            assert s[0] == (1 if (w >= 0).all() else 0)


def test_sentinel_convention():
    """Exactly one MISS (or none); everything after it in priority order is SKIPPED and
    everything before it converged."""
    rng = np.random.default_rng(4)
    seen_miss = 0
    for ts in random_tasksets(rng, 400, wcet_hi=12):
        for pol in ALL_MODES:
            w, s, _ = run([ts], pol, 2, 1)
            order = sorted(range(len(ts)), key=lambda i: (-ts[i]["prio"], i))
            vals = [w[i] for i in order]
            if s[0] == 1:
                assert min(vals) >= 0
                continue
            k = vals.index(rta.WCRT_MISS)
            seen_miss += 1
            assert all(v >= 0 for v in vals[:k]) and all(v == rta.WCRT_SKIPPED for v in vals[k + 1:])
    assert seen_miss > 100


def test_monotone_in_wcet_overhead_and_added_tasks():
    """Raising a WCET, eps/theta, or adding a task never lowers a converged bound and never
    turns an unschedulable taskset schedulable (all terms are non-decreasing)."""
    rng = np.random.default_rng(5)

    def dominated(w_small, s_small, w_big, s_big, idx):
        # compare in priority order up to the first non-converged task of the bigger system
        if s_big == 1:
            assert s_small == 1
        for i in idx:
            if w_big[i] >= 0:
                assert 0 <= w_small[i] <= w_big[i]

    for ts in random_tasksets(rng, 250, max_tasks=5):
        n = len(ts)
        for pol in ALL_MODES:
            L = int(rng.integers(1, 5))
            w, s, _ = run([ts], pol, L, 1)
            more = copy.deepcopy(ts)
            tk = more[int(rng.integers(0, n))]
            if tk.get("gseg") and rng.random() < 0.5:
                j = int(rng.integers(0, len(tk["gseg"])))
                m, e = tk["gseg"][j]
                tk["gseg"][j] = (m + 1, e) if rng.random() < 0.5 else (m, e + 1)
            else:
                tk["cseg"][0] += 1
            w2, s2, _ = run([more], pol, L, 1)
            dominated(w, s[0], w2, s2[0], range(n))
            w3, s3, _ = run([ts], pol, L, 2)
            dominated(w, s[0], w3, s3[0], range(n))
            extra = copy.deepcopy(ts)
            extra.append(dict(T=25, D=25, prio=100, core=0, cseg=[1], gseg=[(0, 1)]))
            w4, s4, _ = run([extra], pol, L, 1)
            dominated(w, s[0], w4[:n], s4[0], range(n))


def test_permutation_and_scaling():
    """Outputs follow a permutation of the tasks; multiplying every time (and L, eps/theta) by k
    multiplies every bound by k."""
    rng = np.random.default_rng(6)
    for ts in random_tasksets(rng, 200):
        n = len(ts)
        perm = rng.permutation(n)
        shuffled = [ts[j] for j in perm]
        for pol in ALL_MODES:
            w, s, _ = run([ts], pol, 3, 1)
            wp, sp, _ = run([shuffled], pol, 3, 1)
            assert s[0] == sp[0] and [w[j] for j in perm] == wp.tolist()
            k = 7
            scaled = copy.deepcopy(ts)
            for tk in scaled:
                tk["T"] *= k
                tk["D"] *= k
                tk["cseg"] = [x * k for x in tk["cseg"]]
                tk["gseg"] = [(m * k, e * k) for m, e in tk["gseg"]]
            wk, sk, _ = run([scaled], pol, 3 * k, 1 * k)
            assert sk[0] == s[0]
            assert wk.tolist() == [x * k if x >= 0 else x for x in w.tolist()]


def test_priority_ties_go_to_the_earlier_task():
    ts = [dict(T=100, prio=5, core=0, cseg=[10]), dict(T=100, prio=5, core=0, cseg=[20])]
    w, _, _ = run([ts], 0)
    assert w.tolist() == [10, 30]
    w, _, _ = run([ts[::-1]], 0)
    assert w.tolist() == [20, 30]


def test_zero_terms_of_the_lemmas():
    """Lemmas 2, 3, 6, 9, 14 as structure: RR ignores tasks' priorities across cores and the CPU
    demand of other cores; GCAPS ignores L; self-suspension charges a CPU-only task nothing for
    GPU work on other cores."""
    rng = np.random.default_rng(7)
    for ts in random_tasksets(rng, 200, max_cores=2):
        for busy in (0, BUSY):
            a, _, _ = run([ts], 0 | busy, 2, 1)
            b, _, _ = run([ts], 0 | busy, 9, 1)
            assert a.tolist() == b.tolist()          # Lemma 9: no interleaving under GCAPS
        # RR: inflate the CPU segments of core-1 tasks; core-0 results must not move as long as
        # the GPU-using set is unchanged (Lemmas 2, 5, 7 only look at hpp)
        other = copy.deepcopy(ts)
        for tk in other:
            if tk["core"] == 1:
                tk["cseg"] = [x + 3 for x in tk["cseg"]]
        for pol in (1, 1 | BUSY):
            w, s, _ = run([ts], pol, 2, 1)
            w2, s2, _ = run([other], pol, 2, 1)
            if s[0] == 1 and s2[0] == 1:
                for i, tk in enumerate(ts):
                    if tk["core"] == 0:
                        assert w[i] == w2[i]
        # GCAPS suspend: a CPU-only task is unaffected by GPU work on other cores (Lemmas 13, 14)
        heavier = copy.deepcopy(ts)
        for tk in heavier:
            if tk["core"] == 1 and tk["gseg"]:
                tk["gseg"] = [(m, e + 2) for m, e in tk["gseg"]]
        w, s, _ = run([ts], 0, 2, 1)
        w2, s2, _ = run([heavier], 0, 2, 1)
        if s[0] == 1 and s2[0] == 1:
            for i, tk in enumerate(ts):
                if tk["core"] == 0 and not tk["gseg"] and not any(
                        t2["core"] == 0 and t2["gseg"] for t2 in ts):
                    assert w[i] == w2[i]


def test_literal_flag_only_changes_the_two_repaired_forms():
    rng = np.random.default_rng(8)
    differs = {0: 0, BUSY: 0, 1: 0, 1 | BUSY: 0}
    for ts in random_tasksets(rng, 400):
        for pol in differs:
            w, _, _ = run([ts], pol, 2, 1)
            wl, _, _ = run([ts], pol | LITERAL, 2, 1)
            if w.tolist() != wl.tolist():
                differs[pol] += 1
                if pol == BUSY:   # repaired form charges more: literal bounds are never larger
                    assert all(a <= b for a, b in zip(wl, w) if a >= 0 and b >= 0)
                if pol == 1:      # literal adds jitter for CPU-only tasks: never smaller
                    assert all(a >= b for a, b in zip(wl, w) if a >= 0 and b >= 0)
    assert differs[0] == 0 and differs[1 | BUSY] == 0
    assert differs[BUSY] > 0 and differs[1] > 0


def test_iteration_cap_and_slow_convergence():
    """tau_h with T=2, C=2 makes tau_i's iterate grow by 2 per sweep: 1, 3, 5, ...  With a
    deadline beyond 2*cap the cap is what stops it."""
    ts = [dict(T=2, prio=2, core=0, cseg=[2]), dict(T=1 << 23, prio=1, core=0, cseg=[1])]
    w, s, c = run([ts], 0, iter_cap=1000)
    assert w.tolist() == [2, rta.WCRT_ITER_LIMIT] and s[0] == 0 and c.sweeps == 1001
    ts[1]["T"] = 1001
    w, s, c = run([ts], 0, iter_cap=1000)
    assert w.tolist() == [2, rta.WCRT_MISS]      # 1003 > 1001 after 501 sweeps
    assert c.sweeps == 1 + 501


def test_invalid_tasksets_and_arguments():
    good = [dict(T=10, prio=1, core=0, cseg=[1])]
    bad_deadline = [dict(T=10, D=11, prio=1, core=0, cseg=[1]), dict(T=10, prio=0, core=0, cseg=[1])]
    bad_wcet = [dict(T=10, prio=1, core=0, cseg=[-1])]
    bad_core = [dict(T=10, prio=1, core=-1, cseg=[1])]
    bad_period = [dict(T=0, D=0, prio=1, core=0, cseg=[1])]
    b = batch_of([good, bad_deadline, bad_wcet, [], bad_core, bad_period, good])
    w, s, _ = rta.analyse(b, 0, 4, 0)
    assert s.tolist() == [1, 2, 2, 1, 2, 2, 1]
    assert w.tolist() == [1, -4, -4, -4, -4, -4, 1]
    assert rta.validate(b).tolist() == [0, 8, 32, 0, 16, 4 | 8, 0]
    b.task_off[2] = 99
    assert rta.validate(b).tolist()[1:3] == [1, 1]
    for kw in (dict(policy=2), dict(policy=0x400), dict(policy=1, timeslice_us=0),
               dict(policy=0, overhead_us=-1), dict(policy=0, overhead_us=(1 << 40) + 1)):
        with pytest.raises(ValueError):
            rta.analyse(batch_of([good]), **kw)


def test_extreme_values_do_not_overflow():
    """Times at the top of the domain (2^40).  GCAPS suspend, eps = 0, B = 2^40:
    R_1 = B/4;  R_2 = (B/8+1) + 1*(3B/16) + 1*(B/16) = 3B/8+1;
    R_3 = (B/2+1) + 1*(B/16) + 1*(B/16) = 5B/8+1 (one job of each in the window)."""
    B = 1 << 40
    ts = [dict(T=B, prio=3, core=0, cseg=[B // 8], gseg=[(B // 16, B // 16)]),
          dict(T=B, prio=2, core=0, cseg=[B // 16], gseg=[(1, B // 16)]),
          dict(T=B, prio=1, core=1, cseg=[B // 2], gseg=[(0, 1)])]
    w, s, _ = run([ts], 0, 1, 0)
    assert w.tolist() == [B // 4, 3 * B // 8 + 1, 5 * B // 8 + 1] and s[0] == 1
    # RR busy with L = 1, theta = 2^40: (L+theta)*nu*slices ~ 2^40 * 2 * 2^36 must read as a miss
    w, s, _ = run([ts], 1 | BUSY, 1, B)
    assert w[0] == rta.WCRT_MISS and s[0] == 0
    # many large segments: sums stay exact
    ts = [dict(T=B, prio=1, core=0, cseg=[B >> 10] * 512, gseg=[(B >> 12, B >> 12)] * 512)]
    w, s, _ = run([ts], 1, B, 0)
    assert w.tolist() == [B // 2 + B // 4]
