"""ctypes wrapper of ``des_sim.c`` -- TEST INFRASTRUCTURE ONLY (see the package docstring)."""
from __future__ import annotations

import ctypes
from typing import Sequence, Tuple

import numpy as np

from . import build as _build

_p64 = ctypes.POINTER(ctypes.c_int64)
_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build("des_sim"))
        lib.des_simulate_gp.argtypes = [ctypes.c_int] + [_p64] * 10 + [
            ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int64, _p64, _p64]
        lib.des_simulate_gp.restype = ctypes.c_int
        lib.des_sweep_offsets.argtypes = [ctypes.c_int] + [_p64] * 9 + [
            ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, _p64, _p64]
        lib.des_sweep_offsets.restype = ctypes.c_int
        _lib = lib
    return _lib


def simulate(batch, t: int, offsets: Sequence[int], policy: int, busy: bool, timeslice: int,
             horizon: int, gpu_priority=None) -> Tuple[np.ndarray, np.ndarray]:
    """Simulates taskset ``t`` of ``batch`` for ``horizon`` ticks.

    Returns ``(max_resp, unfinished)`` per task: the largest response time of a completed job and
    the age of a job still in progress at the horizon (0 if none).  ``gpu_priority`` (per task of
    the taskset) arbitrates the GPU under GCAPS instead of the CPU priorities.
    """
    lib = _load()
    a, b = int(batch.task_off[t]), int(batch.task_off[t + 1])
    n = b - a
    c = lambda x: np.ascontiguousarray(x, dtype=np.int64)
    T, prio, core = c(batch.period[a:b]), c(batch.priority[a:b]), c(batch.core[a:b])
    gprio = prio if gpu_priority is None else c(gpu_priority)  # GPU-segment priorities (GCAPS)
    assert gprio.shape[0] == n
    off = c(offsets)
    assert off.shape[0] == n
    c_off = c(batch.cseg_off[a:b + 1] - batch.cseg_off[a])
    g_off = c(batch.gseg_off[a:b + 1] - batch.gseg_off[a])
    cs = c(batch.cseg_wcet[batch.cseg_off[a]:batch.cseg_off[b]])
    gm = c(batch.gseg_misc[batch.gseg_off[a]:batch.gseg_off[b]])
    ge = c(batch.gseg_exec[batch.gseg_off[a]:batch.gseg_off[b]])
    max_resp = np.zeros(n, np.int64)
    unfinished = np.zeros(n, np.int64)
    p = lambda x: x.ctypes.data_as(_p64)
    rc = lib.des_simulate_gp(n, p(T), p(prio), p(gprio), p(core), p(off), p(c_off), p(cs), p(g_off), p(gm),
                          p(ge), policy, 1 if busy else 0, timeslice, horizon, p(max_resp),
                          p(unfinished))
    if rc != 0:
        raise ValueError("taskset does not fit the simulator's limits")
    return max_resp, unfinished


def sweep_offsets(batch, t: int, policy: int, busy: bool, timeslice: int, step: int = 1,
                  gpu_priority=None) -> Tuple[np.ndarray, int]:
    """Simulates taskset ``t`` of ``batch`` once for every vector of release offsets on a grid of
    ``step`` ticks below the tasks' periods, each run over two hyperperiods.

    Returns ``(worst, runs)``: per task the largest response time observed in any run (a job
    still running at a horizon counts with its age) and the number of offset vectors tried.
    """
    lib = _load()
    a, b = int(batch.task_off[t]), int(batch.task_off[t + 1])
    n = b - a
    c = lambda x: np.ascontiguousarray(x, dtype=np.int64)
    T, prio, core = c(batch.period[a:b]), c(batch.priority[a:b]), c(batch.core[a:b])
    gprio = prio if gpu_priority is None else c(gpu_priority)
    c_off = c(batch.cseg_off[a:b + 1] - batch.cseg_off[a])
    g_off = c(batch.gseg_off[a:b + 1] - batch.gseg_off[a])
    cs = c(batch.cseg_wcet[batch.cseg_off[a]:batch.cseg_off[b]])
    gm = c(batch.gseg_misc[batch.gseg_off[a]:batch.gseg_off[b]])
    ge = c(batch.gseg_exec[batch.gseg_off[a]:batch.gseg_off[b]])
    worst = np.zeros(n, np.int64)
    runs = np.zeros(1, np.int64)
    p = lambda x: x.ctypes.data_as(_p64)
    hyper = int(np.lcm.reduce(T))
    rc = lib.des_sweep_offsets(n, p(T), p(prio), p(gprio), p(core), p(c_off), p(cs), p(g_off),
                               p(gm), p(ge), policy, 1 if busy else 0, timeslice, step, hyper,
                               p(worst), p(runs))
    if rc != 0:
        raise ValueError("taskset does not fit the simulator's limits")
    return worst, int(runs[0])
