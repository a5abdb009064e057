"""Shared helpers of the test-suite (fixture parsing, small random tasksets)."""
from __future__ import annotations

import os

import numpy as np

from paper_2406_05221_b200.taskgen import TasksetBatch

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

POLICY = {"gcaps": 0, "rr": 1}
BUSY, LITERAL, BEST_EFFORT = 0x100, 0x200, 0x800
ALL_MODES = [0, BUSY, LITERAL, BUSY | LITERAL, 1, 1 | BUSY, 1 | LITERAL, 1 | BUSY | LITERAL]


def parse_vector_sets(name):
    """Reads a fixture of `taskset <name>` / `task ...` / `case ...` lines; returns a list of
    (taskset name, list of task dicts, list of cases), one entry per taskset of the file (a file
    without `taskset` lines holds one unnamed taskset)."""
    sets = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            tok = line.split()
            if tok[0] == "taskset":
                sets.append((tok[1], [], []))
                continue
            if not sets:
                sets.append(("", [], []))
            _, tasks, cases = sets[-1]
            kv = dict(x.split("=", 1) for x in tok[2:])
            if tok[0] == "task":
                cseg = [int(x) for x in kv["cseg"].split(",") if x]
                gseg = [tuple(int(y) for y in x.split(":")) for x in kv["gseg"].split(",") if x]
                tasks.append(dict(T=int(kv["T"]), prio=int(kv["prio"]), core=int(kv["core"]),
                                  cseg=cseg, gseg=gseg))
            elif tok[0] == "case":
                flags = POLICY[kv["policy"]] | (BUSY if kv["busy"] == "1" else 0) | (
                    LITERAL if kv["literal"] == "1" else 0) | (
                    BEST_EFFORT if kv.get("be", "0") == "1" else 0)
                cases.append(dict(name=tok[1], policy=flags, L=int(kv["L"]), ovh=int(kv["ovh"]),
                                  expect=[int(x) for x in kv["expect"].split(",")]))
    return sets


def parse_vectors(name):
    """Reads a one-taskset fixture; returns (list of task dicts, list of cases)."""
    sets = parse_vector_sets(name)
    assert len(sets) == 1, name
    return sets[0][1], sets[0][2]


def random_tasksets(rng, count, max_tasks=6, max_cores=3, periods=(20, 30, 40, 60, 80, 120, 200),
                    max_gseg=3, wcet_hi=6, unique_prio=True):
    """Small random tasksets as lists of task dicts (rate-monotonic priorities)."""
    out = []
    for _ in range(count):
        n = int(rng.integers(1, max_tasks + 1))
        cores = int(rng.integers(1, max_cores + 1))
        ts = []
        for _i in range(n):
            T = int(rng.choice(periods))
            ng = int(rng.integers(0, max_gseg + 1))
            cs = [int(rng.integers(0, wcet_hi)) for _ in range(int(rng.integers(1, ng + 3)))]
            gs = [(int(rng.integers(0, 3)), int(rng.integers(0, wcet_hi))) for _ in range(ng)]
            ts.append(dict(T=T, D=int(rng.integers(max(1, T // 2), T + 1)), prio=0,
                           core=int(rng.integers(0, cores)), cseg=cs, gseg=gs))
        order = sorted(range(n), key=lambda i: (ts[i]["T"], i))
        for r, i in enumerate(order):
            ts[i]["prio"] = (n - r) if unique_prio else (n - r) // 2
        out.append(ts)
    return out


def batch_of(tasksets):
    return TasksetBatch.from_tasksets(tasksets)
