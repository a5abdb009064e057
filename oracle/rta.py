"""ctypes wrapper of ``rta_oracle.c`` -- TEST INFRASTRUCTURE ONLY (see the package docstring).

``analyse(batch, policy, ...)`` runs the single-threaded CPU oracle over a batch of tasksets
(any object with the ten int64 numpy arrays of the CSR layout as attributes) and returns
``(wcrt, sched, counts)``.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Tuple

import numpy as np

from . import build as _build

POLICY_GCAPS = 0
POLICY_RR = 1
FLAG_BUSY = 0x100
FLAG_LITERAL = 0x200
FLAG_ASSIGN = 0x400
FLAG_BEST_EFFORT = 0x800

SCHED_NO, SCHED_YES, SCHED_INVALID = 0, 1, 2
WCRT_MISS, WCRT_SKIPPED, WCRT_ITER_LIMIT, WCRT_INVALID, WCRT_BEST_EFFORT = -1, -2, -3, -4, -5
ITER_CAP = 1 << 20

_FIELDS = ("task_off", "period", "deadline", "priority", "core",
           "cseg_off", "cseg_wcet", "gseg_off", "gseg_misc", "gseg_exec")
_p64 = ctypes.POINTER(ctypes.c_int64)


class _Tasksets(ctypes.Structure):
    _fields_ = [("n_tasks", ctypes.c_int64), ("n_csegs", ctypes.c_int64),
                ("n_gsegs", ctypes.c_int64)] + [(f, _p64) for f in _FIELDS]


class Counts(ctypes.Structure):
    """Work counters of one oracle run (they define the algorithmic work of the analysis)."""
    _fields_ = [("sweeps", ctypes.c_int64), ("terms", ctypes.c_int64), ("tasks", ctypes.c_int64)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build("rta_oracle"))
        lib.oracle_rta_range.argtypes = [
            ctypes.POINTER(_Tasksets), ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, _p64,
            ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(Counts)]
        lib.oracle_rta_range.restype = ctypes.c_int
        lib.oracle_validate_range.argtypes = [
            ctypes.POINTER(_Tasksets), ctypes.c_int64, ctypes.c_int64,
            ctypes.POINTER(ctypes.c_int32)]
        lib.oracle_validate_range.restype = None
        _lib = lib
    return _lib


def _pack(batch):
    keep = []
    s = _Tasksets()
    for f in _FIELDS:
        a = np.ascontiguousarray(getattr(batch, f), dtype=np.int64)
        keep.append(a)
        setattr(s, f, a.ctypes.data_as(_p64))
    s.n_tasks = keep[1].shape[0]
    s.n_csegs = keep[6].shape[0]
    s.n_gsegs = keep[8].shape[0]
    return s, keep


def analyse(batch, policy: int, timeslice_us: int = 1024, overhead_us: int = 0,
            first: int = 0, count: Optional[int] = None, iter_cap: int = ITER_CAP,
            out: Optional[Tuple[np.ndarray, np.ndarray]] = None):
    """Runs the oracle on tasksets ``first .. first+count-1`` of ``batch``.

    Returns ``(wcrt, sched, counts)``: ``wcrt`` int64 per task (indexed like the per-task input
    arrays; untouched slots hold ``WCRT_INVALID``), ``sched`` uint8 per taskset, ``counts`` the
    work counters.  Raises ValueError on analysis constants outside the domain.
    """
    lib = _load()
    s, keep = _pack(batch)
    n_tasksets = keep[0].shape[0] - 1
    if count is None:
        count = n_tasksets - first
    if out is None:
        wcrt = np.full(s.n_tasks, WCRT_INVALID, np.int64)
        sched = np.full(n_tasksets, SCHED_INVALID, np.uint8)
    else:
        wcrt, sched = out
    counts = Counts()
    rc = lib.oracle_rta_range(ctypes.byref(s), first, count, policy, timeslice_us, overhead_us,
                              iter_cap, wcrt.ctypes.data_as(_p64),
                              sched.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
                              ctypes.byref(counts))
    if rc != 0:
        raise ValueError("oracle: analysis constants outside the input domain")
    return wcrt, sched, counts


def analyse_sweep(batch, policy: int, timeslices_us, overheads_us, iter_cap: int = ITER_CAP):
    """The same batch under several ``(timeslice, overhead)`` pairs -- the paper's experiments
    re-run one set of tasksets while a parameter varies (Sec. 7.1).  By definition this is one
    independent ``analyse`` per pair, and that is all this function does.

    Returns ``(wcrt, sched)`` of shapes ``[n_params, n_tasks]`` and ``[n_params, n_tasksets]``.
    """
    assert len(timeslices_us) == len(overheads_us)
    n_tasksets = np.asarray(batch.task_off).shape[0] - 1
    n_tasks = np.asarray(batch.period).shape[0]
    wcrt = np.full((len(timeslices_us), n_tasks), WCRT_INVALID, np.int64)
    sched = np.full((len(timeslices_us), n_tasksets), SCHED_INVALID, np.uint8)
    for q, (L, ovh) in enumerate(zip(timeslices_us, overheads_us)):
        analyse(batch, policy, int(L), int(ovh), iter_cap=iter_cap, out=(wcrt[q], sched[q]))
    return wcrt, sched


def analyse_multi(batch, policies, timeslices_us, overheads_us, iter_cap: int = ITER_CAP):
    """Several analyses (``policies``: policy | flags words) of the same batch under several
    ``(timeslice, overhead)`` pairs: by definition one independent ``analyse`` per combination.
    Returns ``(wcrt, sched)`` of shapes ``[n_params, n_policies, n_tasks]`` and
    ``[n_params, n_policies, n_tasksets]``."""
    n_tasksets = np.asarray(batch.task_off).shape[0] - 1
    n_tasks = np.asarray(batch.period).shape[0]
    wcrt = np.full((len(overheads_us), len(policies), n_tasks), WCRT_INVALID, np.int64)
    sched = np.full((len(overheads_us), len(policies), n_tasksets), SCHED_INVALID, np.uint8)
    for q, (L, ovh) in enumerate(zip(timeslices_us, overheads_us)):
        for j, pol in enumerate(policies):
            analyse(batch, pol, int(L), int(ovh), iter_cap=iter_cap, out=(wcrt[q, j], sched[q, j]))
    return wcrt, sched


def validate(batch) -> np.ndarray:
    """Per-taskset domain check; 0 = valid, else a bit mask (1 task range, 2 segment range,
    4 period, 8 deadline, 16 core, 32 WCET)."""
    lib = _load()
    s, keep = _pack(batch)
    n_tasksets = keep[0].shape[0] - 1
    err = np.zeros(n_tasksets, np.int32)
    lib.oracle_validate_range(ctypes.byref(s), 0, n_tasksets,
                              err.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    return err


_gp_lib = None


def _load_gpu_prio():
    global _gp_lib
    if _gp_lib is None:
        lib = ctypes.CDLL(_build.build("gpu_prio_oracle"))
        lib.oracle_gpu_prio_range.argtypes = [
            ctypes.POINTER(_Tasksets), ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int64,
            ctypes.c_int64, _p64, _p64, _p64, ctypes.POINTER(ctypes.c_uint8)]
        lib.oracle_gpu_prio_range.restype = ctypes.c_int
        _gp_lib = lib
    return _gp_lib


def analyse_gpu_priority(batch, flags: int = 0, overhead_us: int = 0, gpu_priority=None,
                         iter_cap: int = ITER_CAP):
    """GCAPS analysis with separate GPU-segment priorities (paper Sec. 5.3 / 6.4).

    ``flags``: ``FLAG_BUSY``, ``FLAG_LITERAL``, ``FLAG_ASSIGN``.  With ``FLAG_ASSIGN`` the GPU
    priorities are searched (Audsley) and ``gpu_priority`` is ignored; otherwise ``gpu_priority``
    (int64 per task, larger = higher) is analysed as given.  Returns
    ``(wcrt, sched, gpu_priority_out)``.
    """
    lib = _load_gpu_prio()
    s, keep = _pack(batch)
    n_tasksets = keep[0].shape[0] - 1
    wcrt = np.full(s.n_tasks, WCRT_INVALID, np.int64)
    sched = np.full(n_tasksets, SCHED_INVALID, np.uint8)
    out_gp = np.zeros(s.n_tasks, np.int64)
    gp_in = None
    if gpu_priority is not None:
        gp_in = np.ascontiguousarray(gpu_priority, dtype=np.int64)
        assert gp_in.shape[0] == s.n_tasks
    rc = lib.oracle_gpu_prio_range(
        ctypes.byref(s), 0, n_tasksets, flags, overhead_us, iter_cap,
        gp_in.ctypes.data_as(_p64) if gp_in is not None else None, out_gp.ctypes.data_as(_p64),
        wcrt.ctypes.data_as(_p64), sched.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)))
    if rc != 0:
        raise ValueError("oracle: arguments outside the input domain")
    return wcrt, sched, out_gp
