"""Seeded synthetic tasksets in the CSR structure-of-arrays layout of ``include/gcaps_rta.h``.

This module only produces inputs (it holds none of the analysis arithmetic) and is the one piece
shared by the CUDA path's tests/bench and by the CPU oracle's tests.  The generator itself is C
(``csrc/taskgen.c``, OpenMP) and follows the paper's generation procedure (Sec. 7.1, Table 3):
tasks per CPU -> UUniFast utilisation per CPU -> period -> number of GPU segments -> segment
parameters -> rate-monotonic priorities -> optional worst-fit-decreasing re-allocation.

``WORKLOADS`` names the five benchmark workloads; every taskset is a pure function of
``(seed, stream, global index)`` so any slice of a workload can be generated alone.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
import threading
from typing import Dict, Iterable, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "taskgen.c")
_IGEN_H = os.path.join(_HERE, "csrc", "igen.h")
_LIB = os.path.join(_HERE, "_taskgen.so")
_lock = threading.Lock()
_lib = None

ARRAY_FIELDS = (
    "task_off", "period", "deadline", "priority", "core",
    "cseg_off", "cseg_wcet", "gseg_off", "gseg_misc", "gseg_exec",
)


def build_taskgen(force: bool = False) -> str:
    """Compiles csrc/taskgen.c into _taskgen.so beside this file (gcc, OpenMP)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(
                os.path.getmtime(_SRC), os.path.getmtime(_IGEN_H)):
            tmp = _LIB + ".%d.tmp" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [
        ("seed", ctypes.c_uint64), ("stream", ctypes.c_uint64),
        ("cores_lo", ctypes.c_int32), ("cores_hi", ctypes.c_int32),
        ("tpc_lo", ctypes.c_int32), ("tpc_hi", ctypes.c_int32),
        ("util_lo", ctypes.c_double), ("util_hi", ctypes.c_double),
        ("period_lo", ctypes.c_double), ("period_hi", ctypes.c_double),
        ("harmonic_frac", ctypes.c_double),
        ("gpu_mode", ctypes.c_int32),
        ("gpu_frac", ctypes.c_double),
        ("seg_lo", ctypes.c_int32), ("seg_hi", ctypes.c_int32),
        ("ratio_lo", ctypes.c_double), ("ratio_hi", ctypes.c_double),
        ("wfd", ctypes.c_int32), ("pad_", ctypes.c_int32),
    ]


class IntParams(ctypes.Structure):
    """Mirror of ``igen_params_t`` (csrc/igen.h) and of ``gcaps_gen_params_t`` (gcaps_rta.h)."""
    _fields_ = [
        ("seed", ctypes.c_uint64), ("stream", ctypes.c_uint64),
        ("cores_lo", ctypes.c_int32), ("cores_hi", ctypes.c_int32),
        ("tpc_lo", ctypes.c_int32), ("tpc_hi", ctypes.c_int32),
        ("util_lo", ctypes.c_uint64), ("util_hi", ctypes.c_uint64),
        ("log2_lo", ctypes.c_uint64), ("log2_hi", ctypes.c_uint64), ("log2_hi0", ctypes.c_uint64),
        ("period_lo", ctypes.c_int64), ("period_hi", ctypes.c_int64),
        ("harmonic", ctypes.c_uint64), ("gpu_frac", ctypes.c_uint64),
        ("ratio_lo", ctypes.c_uint64), ("ratio_hi", ctypes.c_uint64),
        ("gpu_mode", ctypes.c_int32), ("seg_lo", ctypes.c_int32), ("seg_hi", ctypes.c_int32),
        ("wfd", ctypes.c_int32),
    ]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_taskgen())
        p64 = ctypes.POINTER(ctypes.c_int64)
        lib.ig_sizes.argtypes = [ctypes.POINTER(IntParams), ctypes.c_int64, ctypes.c_int64, p64]
        lib.ig_sizes.restype = None
        lib.ig_fill.argtypes = [ctypes.POINTER(IntParams), ctypes.c_int64, ctypes.c_int64, p64] + [p64] * 10
        lib.ig_fill.restype = None
        lib.ig_params_size.restype = ctypes.c_size_t
        assert lib.ig_params_size() == ctypes.sizeof(IntParams)
        lib.ig_exp2.argtypes = [ctypes.c_uint64]
        lib.ig_exp2.restype = ctypes.c_uint64
        lib.tg_sizes.argtypes = [ctypes.POINTER(_Params), ctypes.c_int64, ctypes.c_int64, p64]
        lib.tg_sizes.restype = None
        lib.tg_fill.argtypes = [ctypes.POINTER(_Params), ctypes.c_int64, ctypes.c_int64, p64] + [p64] * 10
        lib.tg_fill.restype = None
        lib.tg_params_size.restype = ctypes.c_size_t
        assert lib.tg_params_size() == ctypes.sizeof(_Params)
        _lib = lib
    return _lib


@dataclasses.dataclass
class GenParams:
    """Ranges of one generator stream (see csrc/taskgen.c for the exact procedure)."""
    seed: int
    stream: int = 0
    cores: Sequence[int] = (4, 4)
    tasks_per_core: Sequence[int] = (3, 6)
    util_per_core: Sequence[float] = (0.4, 0.6)
    period_us: Sequence[float] = (30_000.0, 500_000.0)
    harmonic_frac: float = 0.0
    gpu_mode: int = 0            # 0: fixed fraction of GPU-using tasks; 1: eta^g drawn per task
    gpu_frac: float = 0.5
    gpu_segments: Sequence[int] = (1, 3)
    gpu_ratio: Sequence[float] = (0.1, 0.3)   # G_i / task WCET
    wfd: bool = False

    def _c(self) -> _Params:
        return _Params(
            self.seed, self.stream, self.cores[0], self.cores[1],
            self.tasks_per_core[0], self.tasks_per_core[1],
            self.util_per_core[0], self.util_per_core[1],
            self.period_us[0], self.period_us[1], self.harmonic_frac,
            self.gpu_mode, self.gpu_frac, self.gpu_segments[0], self.gpu_segments[1],
            self.gpu_ratio[0], self.gpu_ratio[1], 1 if self.wfd else 0, 0)

    def int_params(self) -> "IntParams":
        """The same ranges for the integer-only generator: fixed point with 32 fractional bits,
        period range as log2 (rounded here, once, on the host: both the host and the device
        generator receive these integers)."""
        import math
        lo, hi = float(self.period_us[0]), float(self.period_us[1])
        hi0 = min(lo * 100.0, hi)
        return IntParams(
            self.seed, self.stream, self.cores[0], self.cores[1],
            self.tasks_per_core[0], self.tasks_per_core[1],
            q32(self.util_per_core[0]), q32(self.util_per_core[1]),
            q32(math.log2(lo)), q32(math.log2(hi)), q32(math.log2(hi0)),
            int(lo), int(hi), q32(self.harmonic_frac), q32(self.gpu_frac),
            q32(self.gpu_ratio[0]), q32(self.gpu_ratio[1]),
            self.gpu_mode, self.gpu_segments[0], self.gpu_segments[1], 1 if self.wfd else 0)


@dataclasses.dataclass
class TasksetBatch:
    """A batch of tasksets; every array is a contiguous int64 numpy array (host memory)."""
    task_off: np.ndarray
    period: np.ndarray
    deadline: np.ndarray
    priority: np.ndarray
    core: np.ndarray
    cseg_off: np.ndarray
    cseg_wcet: np.ndarray
    gseg_off: np.ndarray
    gseg_misc: np.ndarray
    gseg_exec: np.ndarray

    @property
    def n_tasksets(self) -> int:
        return int(self.task_off.shape[0]) - 1

    @property
    def n_tasks(self) -> int:
        return int(self.period.shape[0])

    @property
    def n_csegs(self) -> int:
        return int(self.cseg_wcet.shape[0])

    @property
    def n_gsegs(self) -> int:
        return int(self.gseg_misc.shape[0])

    def input_bytes(self) -> int:
        """Bytes of all ten input arrays."""
        return int(sum(getattr(self, f).nbytes for f in ARRAY_FIELDS))

    def output_bytes(self) -> int:
        """Bytes of out_wcrt (int64 per task) + out_sched (one byte per taskset)."""
        return 8 * self.n_tasks + self.n_tasksets

    def arrays(self) -> Dict[str, np.ndarray]:
        return {f: getattr(self, f) for f in ARRAY_FIELDS}

    def select(self, idx: Iterable[int]) -> "TasksetBatch":
        """A new batch holding the given tasksets, in the given order."""
        idx = np.asarray(list(idx), dtype=np.int64)
        t0 = self.task_off[idx]
        t1 = self.task_off[idx + 1]
        n = t1 - t0
        task_off = np.zeros(idx.shape[0] + 1, np.int64)
        np.cumsum(n, out=task_off[1:])
        tsel = _ranges(t0, n)
        c0, c1 = self.cseg_off[tsel], self.cseg_off[tsel + 1]
        g0, g1 = self.gseg_off[tsel], self.gseg_off[tsel + 1]
        cseg_off = np.zeros(tsel.shape[0] + 1, np.int64)
        np.cumsum(c1 - c0, out=cseg_off[1:])
        gseg_off = np.zeros(tsel.shape[0] + 1, np.int64)
        np.cumsum(g1 - g0, out=gseg_off[1:])
        csel = _ranges(c0, c1 - c0)
        gsel = _ranges(g0, g1 - g0)
        return TasksetBatch(
            task_off, self.period[tsel].copy(), self.deadline[tsel].copy(),
            self.priority[tsel].copy(), self.core[tsel].copy(), cseg_off,
            self.cseg_wcet[csel].copy(), gseg_off, self.gseg_misc[gsel].copy(),
            self.gseg_exec[gsel].copy())

    def slice(self, start: int, stop: int) -> "TasksetBatch":
        return self.select(range(start, stop))

    @staticmethod
    def concat(batches: Sequence["TasksetBatch"]) -> "TasksetBatch":
        """Concatenates batches (offsets are rebased)."""
        if not batches:
            return TasksetBatch.from_tasksets([])
        def cat_off(name, sizes):
            parts, base = [np.zeros(1, np.int64)], 0
            for b, _ in zip(batches, sizes):
                parts.append(getattr(b, name)[1:] + base)
                base += int(getattr(b, name)[-1])
            return np.concatenate(parts)
        out = {}
        for f in ARRAY_FIELDS:
            if f.endswith("_off"):
                out[f] = cat_off(f, batches)
            else:
                out[f] = np.concatenate([getattr(b, f) for b in batches])
        return TasksetBatch(**out)

    @staticmethod
    def from_tasksets(tasksets: Sequence[Sequence[dict]]) -> "TasksetBatch":
        """Builds a batch from explicit tasks.

        Each task is a dict with keys ``T``, ``D`` (default ``T``), ``prio``, ``core``,
        ``cseg`` (list of CPU-segment WCETs) and ``gseg`` (list of ``(G^m, G^e)`` pairs).
        """
        task_off, cseg_off, gseg_off = [0], [0], [0]
        period, deadline, priority, core, cw, gm, ge = [], [], [], [], [], [], []
        for ts in tasksets:
            for tk in ts:
                period.append(int(tk["T"]))
                deadline.append(int(tk.get("D", tk["T"])))
                priority.append(int(tk["prio"]))
                core.append(int(tk["core"]))
                cw.extend(int(x) for x in tk.get("cseg", []))
                for m, e in tk.get("gseg", []):
                    gm.append(int(m))
                    ge.append(int(e))
                cseg_off.append(len(cw))
                gseg_off.append(len(gm))
            task_off.append(len(period))
        a = lambda x: np.asarray(x, dtype=np.int64)
        return TasksetBatch(a(task_off), a(period), a(deadline), a(priority), a(core),
                            a(cseg_off), a(cw), a(gseg_off), a(gm), a(ge))

    def checksum(self) -> str:
        """Hex digest (BLAKE2b-128) of all input arrays, in ARRAY_FIELDS order."""
        import hashlib
        h = hashlib.blake2b(digest_size=16)
        for f in ARRAY_FIELDS:
            a = np.ascontiguousarray(getattr(self, f))
            h.update(f.encode())
            h.update(a.shape[0].to_bytes(8, "little"))
            h.update(a.tobytes())
        return h.hexdigest()


def _ranges(start: np.ndarray, length: np.ndarray) -> np.ndarray:
    """Concatenation of arange(start[i], start[i]+length[i])."""
    total = int(length.sum())
    if total == 0:
        return np.zeros(0, np.int64)
    ends = np.cumsum(length)
    out = np.ones(total, np.int64)
    nz = length > 0
    firsts = (ends - length)[nz]
    s = start[nz]
    out[firsts] = s - np.concatenate([[0], (s + length[nz] - 1)[:-1]])
    out[0] = s[0]
    return np.cumsum(out)


def q32(x: float) -> int:
    """x as a fixed-point number with 32 fractional bits."""
    return int(round(x * 4294967296.0))


def generate(params: GenParams, first: int, count: int, threads: Optional[int] = None,
             alloc=None, integer: bool = False) -> TasksetBatch:
    """Tasksets ``first .. first+count-1`` of the stream described by ``params``.

    ``alloc(n)`` may supply the int64 output arrays (e.g. views of page-locked memory).
    ``integer=True`` uses the integer-only generator (csrc/igen.h), whose tasksets the CUDA
    library can also produce on the device, bit for bit; it is a different stream of tasksets
    with the same ranges and distributions."""
    lib = _load()
    if count <= 0:
        return TasksetBatch.from_tasksets([])
    if threads is not None:
        os.environ["OMP_NUM_THREADS"] = str(threads)
    cp = params.int_params() if integer else params._c()
    sizes_fn, fill_fn = (lib.ig_sizes, lib.ig_fill) if integer else (lib.tg_sizes, lib.tg_fill)
    counts = np.zeros((count, 3), np.int64)
    p64 = ctypes.POINTER(ctypes.c_int64)
    ptr = lambda a: a.ctypes.data_as(p64)
    sizes_fn(ctypes.byref(cp), first, count, ptr(counts))
    starts = np.zeros((count, 3), np.int64)
    np.cumsum(counts[:-1], axis=0, out=starts[1:])
    n_tasks, n_c, n_g = (int(x) for x in counts.sum(axis=0))
    if alloc is None:
        alloc = lambda n: np.empty(n, np.int64)
    sizes = {"task_off": count + 1, "period": n_tasks, "deadline": n_tasks, "priority": n_tasks,
             "core": n_tasks, "cseg_off": n_tasks + 1, "cseg_wcet": n_c, "gseg_off": n_tasks + 1,
             "gseg_misc": n_g, "gseg_exec": n_g}
    arr = {f: alloc(sizes[f]) for f in ARRAY_FIELDS}
    fill_fn(ctypes.byref(cp), first, count, ptr(starts), *[ptr(arr[f]) for f in ARRAY_FIELDS])
    return TasksetBatch(**arr)


@dataclasses.dataclass
class Workload:
    """One named benchmark workload: generator streams plus the analysis constants."""
    name: str
    n_tasksets: int                 # tasksets per stream
    streams: List[GenParams]        # one per sweep point
    timeslice_us: int = 1024        # L
    overhead_us: int = 50           # theta (RR) / epsilon (GCAPS)
    timeslices: Sequence[int] = ()  # RR driver-model sweep values of L
    overheads: Sequence[int] = ()   # RR driver-model sweep values of theta
    policies: Sequence[str] = ("gcaps", "rr")
    note: str = ""

    def generate(self, first: int = 0, count: Optional[int] = None, stream: int = 0,
                 alloc=None, integer: bool = False) -> TasksetBatch:
        if count is None:
            count = self.n_tasksets - first
        return generate(self.streams[stream], first, count, alloc=alloc, integer=integer)


def _workloads() -> Dict[str, Workload]:
    w: Dict[str, Workload] = {}
    w["pr1"] = Workload(
        "pr1", 1_000,
        [GenParams(seed=1, cores=(2, 2), tasks_per_core=(4, 4), util_per_core=(0.5, 0.5),
                   period_us=(1e4, 1e6), gpu_frac=0.5, gpu_segments=(1, 1), gpu_ratio=(0.1, 0.3))],
        note="1,000 tasksets, 2 cores x 4 tasks, U=0.5/core, 50% GPU tasks with 1 segment")
    w["sweep"] = Workload(
        "sweep", 100_000,
        [GenParams(seed=2, stream=k, cores=(4, 4), tasks_per_core=(5, 5),
                   util_per_core=(0.1 * (k + 1), 0.1 * (k + 1)), period_us=(1e4, 1e6),
                   gpu_frac=0.6, gpu_segments=(1, 3), gpu_ratio=(0.1, 0.5), wfd=True)
         for k in range(9)],
        note="9 points U/core=0.1..0.9, 100,000 tasksets each, 4 cores x 5 tasks, WFD")
    w["large"] = Workload(
        "large", 1_000_000,
        [GenParams(seed=3, cores=(8, 8), tasks_per_core=(10, 10), util_per_core=(0.3, 0.8),
                   period_us=(1e3, 1e6), gpu_frac=0.8, gpu_segments=(1, 5), gpu_ratio=(0.2, 0.6))],
        note="1,000,000 tasksets, 8 cores x 10 tasks (80 tasks), 80% GPU tasks, 1-5 segments")
    w["rr_model"] = Workload(
        "rr_model", 200_000,
        [GenParams(seed=4, cores=(4, 4), tasks_per_core=(6, 6), util_per_core=(0.6, 0.6),
                   period_us=(1e4, 1e6), gpu_frac=0.7, gpu_segments=(1, 3), gpu_ratio=(0.3, 0.3))],
        timeslices=(256, 512, 1024, 2048, 4096), overheads=(0, 25, 50, 100, 200),
        policies=("rr",),
        note="200,000 tasksets, 4 cores x 6 tasks, RR only, 5 timeslices x 5 overheads")
    w["divergence"] = Workload(
        "divergence", 10_000_000,
        [GenParams(seed=5, cores=(2, 16), tasks_per_core=(2, 12), util_per_core=(0.05, 0.95),
                   period_us=(1e2, 1e7), harmonic_frac=0.5, gpu_mode=1, gpu_segments=(0, 8),
                   gpu_ratio=(0.05, 0.9))],
        note="10,000,000 tasksets, 2-16 cores x 2-12 tasks, 0-8 segments, half harmonic periods")
    # a diagnostic beside the five benchmark workloads: the shape of `large` with so little load
    # and overhead that (under GCAPS) every taskset converges, so that the recurrence runs for all
    # 80 tasks of a taskset instead of stopping at an early deadline miss
    w["large_light"] = Workload(
        "large_light", 200_000,
        [GenParams(seed=6, cores=(8, 8), tasks_per_core=(10, 10), util_per_core=(0.05, 0.2),
                   period_us=(1e3, 1e6), gpu_frac=0.8, gpu_segments=(1, 5), gpu_ratio=(0.1, 0.3))],
        overhead_us=5,
        note="200,000 tasksets shaped like 'large' (8 cores x 10 tasks, 80% GPU tasks) with "
             "U/core 0.05-0.2, GPU share 10-30%, overhead 5 us: schedulable under GCAPS")
    return w


WORKLOADS: Dict[str, Workload] = _workloads()
