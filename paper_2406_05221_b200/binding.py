"""Thin ctypes binding of the C-ABI library ``libgcaps_rta.so`` (declared in include/gcaps_rta.h).

Argument marshalling only: every step of the analysis runs in the CUDA kernels of the library.
PyTorch is used for device memory and streams.  There is no CPU fallback: if the library is
missing or no B200 is present the calls raise.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
from typing import Dict, Optional, Tuple

import numpy as np

from . import build as _build
from .taskgen import ARRAY_FIELDS, GenParams, IntParams, TasksetBatch

POLICY_GCAPS = 0
POLICY_RR = 1
BUSY = 0x100
LITERAL = 0x200
ASSIGN = 0x400
BEST_EFFORT = 0x800

SCHED_NO, SCHED_YES, SCHED_INVALID = 0, 1, 2
WCRT_MISS, WCRT_SKIPPED, WCRT_ITER_LIMIT, WCRT_INVALID, WCRT_BEST_EFFORT = -1, -2, -3, -4, -5
MAX_TASKS = 256
MAX_TIME = 1 << 40

OK, ERR_INVALID_ARG, ERR_WORKSPACE, ERR_CUDA, ERR_NO_DEVICE, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5
STATIC_MAX_TASKSETS = 65536
MAX_SWEEP = 32
# analyses of rta_multi, in result order
GCAPS_SUSPEND, GCAPS_BUSY, RR_SUSPEND, RR_BUSY = 1, 2, 4, 8
ANALYSIS_POLICY = {GCAPS_SUSPEND: POLICY_GCAPS, GCAPS_BUSY: POLICY_GCAPS | BUSY,
                   RR_SUSPEND: POLICY_RR, RR_BUSY: POLICY_RR | BUSY}

EXPORTS = ("gcaps_rta_batch", "gcaps_rta_workspace_bytes", "gcaps_rta_batch_host",
           "gcaps_rta_release_host", "gcaps_rta_validate", "gcaps_rta_strerror",
           "gcaps_rta_last_cuda_error", "gcaps_rta_version", "gcaps_rta_batch_static",
           "gcaps_rta_batch_host_multi", "gcaps_rta_gpu_priority_batch", "gcaps_rta_sweep_batch", "gcaps_rta_multi_batch",
           "gcaps_gen_workspace_bytes", "gcaps_gen_count", "gcaps_gen_fill",
           "gcaps_rta_plan_batch", "gcaps_rta_int_issue_probe")

_p64 = ctypes.POINTER(ctypes.c_int64)


class CTasksets(ctypes.Structure):
    """Mirror of ``gcaps_tasksets_t``."""
    _fields_ = [("n_tasks", ctypes.c_int64), ("n_csegs", ctypes.c_int64),
                ("n_gsegs", ctypes.c_int64)] + [(f, ctypes.c_void_p) for f in ARRAY_FIELDS]


class GcapsError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__("gcaps_rta: %s (code %d)" % (text, code))
        self.code = code


_lib = None


def load_library(path: Optional[str] = None):
    """Loads libgcaps_rta.so (never builds it implicitly on a machine without the source
    being newer: a missing library is an error, not a reason to fall back)."""
    global _lib
    if _lib is None or path is not None:
        path = path or _build.CUDA_LIB
        if not os.path.exists(path):
            raise FileNotFoundError(
                "%s is missing: run `python -m paper_2406_05221_b200.build` (needs nvcc)" % path)
        lib = ctypes.CDLL(path)
        lib.gcaps_rta_batch.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        lib.gcaps_rta_batch.restype = ctypes.c_int
        lib.gcaps_rta_batch_static.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.gcaps_rta_batch_static.restype = ctypes.c_int
        lib.gcaps_rta_workspace_bytes.argtypes = [ctypes.c_int64]
        lib.gcaps_rta_workspace_bytes.restype = ctypes.c_size_t
        lib.gcaps_rta_batch_host.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p]
        lib.gcaps_rta_batch_host.restype = ctypes.c_int
        lib.gcaps_rta_batch_host_multi.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.POINTER(ctypes.c_int), ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.POINTER(ctypes.c_void_p),
            ctypes.POINTER(ctypes.c_void_p)]
        lib.gcaps_rta_batch_host_multi.restype = ctypes.c_int
        lib.gcaps_rta_gpu_priority_batch.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
            ctypes.c_void_p]
        lib.gcaps_rta_gpu_priority_batch.restype = ctypes.c_int
        lib.gcaps_rta_sweep_batch.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_int, ctypes.c_int, _p64, _p64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        lib.gcaps_rta_sweep_batch.restype = ctypes.c_int
        lib.gcaps_rta_multi_batch.argtypes = [
            ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, _p64, _p64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        lib.gcaps_rta_multi_batch.restype = ctypes.c_int
        lib.gcaps_gen_workspace_bytes.argtypes = [ctypes.POINTER(IntParams), ctypes.c_int64]
        lib.gcaps_gen_workspace_bytes.restype = ctypes.c_size_t
        lib.gcaps_gen_count.argtypes = [ctypes.POINTER(IntParams), ctypes.c_int64, ctypes.c_int64,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        lib.gcaps_gen_count.restype = ctypes.c_int
        lib.gcaps_gen_fill.argtypes = [ctypes.POINTER(IntParams), ctypes.c_int64, ctypes.c_int64,
                                       ctypes.POINTER(CTasksets), ctypes.c_void_p, ctypes.c_size_t,
                                       ctypes.c_void_p]
        lib.gcaps_gen_fill.restype = ctypes.c_int
        lib.gcaps_rta_plan_batch.argtypes = [ctypes.POINTER(CTasksets), ctypes.c_int64, ctypes.c_void_p,
                                             ctypes.c_size_t, ctypes.c_void_p]
        lib.gcaps_rta_plan_batch.restype = ctypes.c_int
        lib.gcaps_rta_int_issue_probe.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, _p64,
                                                  ctypes.c_void_p]
        lib.gcaps_rta_int_issue_probe.restype = ctypes.c_int
        lib.gcaps_rta_release_host.argtypes = []
        lib.gcaps_rta_release_host.restype = None
        lib.gcaps_rta_validate.argtypes = [ctypes.POINTER(CTasksets), ctypes.c_int64,
                                           ctypes.c_void_p, ctypes.c_void_p]
        lib.gcaps_rta_validate.restype = ctypes.c_int
        lib.gcaps_rta_strerror.argtypes = [ctypes.c_int]
        lib.gcaps_rta_strerror.restype = ctypes.c_char_p
        lib.gcaps_rta_last_cuda_error.restype = ctypes.c_int
        lib.gcaps_rta_version.restype = ctypes.c_int
        _lib = lib
    return _lib


@contextlib.contextmanager
def _device_and_stream(dev, stream):
    """Makes ``dev`` the current device and ``stream`` (default: torch's current one) the current
    stream.  Tensors the wrappers create inside (outputs, workspace) then belong to the stream the
    kernels run on, so torch's allocator cannot hand their memory to someone else while those
    kernels are still in flight."""
    import torch
    with torch.cuda.device(dev):
        st = stream if stream is not None else torch.cuda.current_stream(dev)
        with torch.cuda.stream(st):
            yield st


def _check(rc: int):
    if rc != OK:
        lib = load_library()
        text = lib.gcaps_rta_strerror(rc).decode()
        if rc == ERR_CUDA:
            text += " [cudaError %d]" % lib.gcaps_rta_last_cuda_error()
        raise GcapsError(rc, text)


def workspace_bytes(n_tasksets: int) -> int:
    return int(load_library().gcaps_rta_workspace_bytes(n_tasksets))


class DeviceTasksets:
    """The ten input arrays as int64 CUDA tensors plus the C struct that points at them."""

    def __init__(self, tensors: Dict[str, "torch.Tensor"]):
        self.t = tensors
        self.n_tasksets = int(tensors["task_off"].shape[0]) - 1
        self.n_tasks = int(tensors["period"].shape[0])
        self.n_csegs = int(tensors["cseg_wcet"].shape[0])
        self.n_gsegs = int(tensors["gseg_misc"].shape[0])
        self.c = CTasksets(self.n_tasks, self.n_csegs, self.n_gsegs,
                           *[tensors[f].data_ptr() for f in ARRAY_FIELDS])

    @staticmethod
    def from_host(batch: TasksetBatch, device="cuda:0") -> "DeviceTasksets":
        import torch
        return DeviceTasksets({f: torch.from_numpy(np.ascontiguousarray(getattr(batch, f))).to(device)
                               for f in ARRAY_FIELDS})

    def input_bytes(self) -> int:
        return sum(int(v.numel()) * 8 for v in self.t.values())


def rta_batch(ts: DeviceTasksets, policy: int, timeslice_us: int = 1024, overhead_us: int = 0,
              out_wcrt=None, out_sched=None, workspace=None, stream=None):
    """gcaps_rta_batch on device-resident inputs.  Returns ``(out_wcrt, out_sched)`` CUDA tensors
    (int64 per task, uint8 per taskset); asynchronous on ``stream`` (default: torch's current)."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    with _device_and_stream(dev, stream) as st:
        if out_wcrt is None:
            out_wcrt = torch.empty(ts.n_tasks, dtype=torch.int64, device=dev)
        if out_sched is None:
            out_sched = torch.empty(max(ts.n_tasksets, 0), dtype=torch.uint8, device=dev)
        need = workspace_bytes(ts.n_tasksets)
        if workspace is None:
            workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        rc = lib.gcaps_rta_batch(ctypes.byref(ts.c), ts.n_tasksets, policy, timeslice_us, overhead_us,
                                 out_wcrt.data_ptr(), out_sched.data_ptr(), workspace.data_ptr(),
                                 workspace.numel(), st.cuda_stream)
    _check(rc)
    return out_wcrt, out_sched


def rta_sweep(ts: DeviceTasksets, policy: int, timeslices_us, overheads_us, want_wcrt: bool = True,
              out_wcrt=None, out_sched=None, workspace=None, stream=None):
    """gcaps_rta_sweep_batch: the resident batch under every ``(timeslice, overhead)`` pair in one
    pass.  Returns ``(out_wcrt, out_sched)`` CUDA tensors of shapes ``[n_points, n_tasks]`` (None
    with ``want_wcrt=False``) and ``[n_points, n_tasksets]``."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    k = len(overheads_us)
    Ls = (ctypes.c_int64 * k)(*[int(x) for x in timeslices_us]) if timeslices_us is not None else None
    ov = (ctypes.c_int64 * k)(*[int(x) for x in overheads_us])
    with _device_and_stream(dev, stream) as st:
        if out_wcrt is None and want_wcrt:
            out_wcrt = torch.empty((k, ts.n_tasks), dtype=torch.int64, device=dev)
        if out_sched is None:
            out_sched = torch.empty((k, max(ts.n_tasksets, 0)), dtype=torch.uint8, device=dev)
        need = workspace_bytes(ts.n_tasksets)
        if workspace is None:
            workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
        rc = lib.gcaps_rta_sweep_batch(ctypes.byref(ts.c), ts.n_tasksets, policy, k, Ls, ov,
                                       out_wcrt.data_ptr() if out_wcrt is not None else None,
                                       out_sched.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                       st.cuda_stream)
    _check(rc)
    return out_wcrt, out_sched


def rta_multi(ts: DeviceTasksets, analyses: int, timeslices_us=(1024,), overheads_us=(0,), flags: int = 0,
              want_wcrt: bool = True, out_wcrt=None, out_sched=None, workspace=None, stream=None):
    """gcaps_rta_multi_batch: the analyses named in ``analyses`` (OR of ``GCAPS_SUSPEND``,
    ``GCAPS_BUSY``, ``RR_SUSPEND``, ``RR_BUSY``) for every ``(timeslice, overhead)`` pair, one pass
    over the resident batch.  Returns ``(out_wcrt, out_sched)`` CUDA tensors of shapes
    ``[n_points, k, n_tasks]`` (None with ``want_wcrt=False``) and ``[n_points, k, n_tasksets]``,
    ``k`` analyses in the order of the four constants."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    n_pts, k = len(overheads_us), bin(analyses & 15).count("1")
    Ls = (ctypes.c_int64 * n_pts)(*[int(x) for x in timeslices_us]) if timeslices_us is not None else None
    ov = (ctypes.c_int64 * n_pts)(*[int(x) for x in overheads_us])
    with _device_and_stream(dev, stream) as st:
        if out_wcrt is None and want_wcrt:
            out_wcrt = torch.empty((n_pts, k, ts.n_tasks), dtype=torch.int64, device=dev)
        if out_sched is None:
            out_sched = torch.empty((n_pts, k, max(ts.n_tasksets, 0)), dtype=torch.uint8, device=dev)
        if workspace is None:
            workspace = torch.empty(max(workspace_bytes(ts.n_tasksets), 256), dtype=torch.uint8, device=dev)
        rc = lib.gcaps_rta_multi_batch(ctypes.byref(ts.c), ts.n_tasksets, analyses, flags, n_pts, Ls, ov,
                                       out_wcrt.data_ptr() if out_wcrt is not None else None,
                                       out_sched.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                       st.cuda_stream)
    _check(rc)
    return out_wcrt, out_sched


def rta_batch_static(ts: DeviceTasksets, policy: int, timeslice_us: int = 1024, overhead_us: int = 0,
                     out_wcrt=None, out_sched=None, stream=None):
    """gcaps_rta_batch_static: the same analysis for callers that cannot allocate device memory.

    The library's built-in scratch array takes the place of the workspace, so the call itself
    allocates nothing; this wrapper only creates the two output tensors when the caller passes
    none.  At most ``STATIC_MAX_TASKSETS`` tasksets per call (``GcapsError`` with
    ``ERR_TOO_LARGE`` beyond).  Calls that could overlap on the GPU must be ordered by the caller:
    they share the one scratch array."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    with _device_and_stream(dev, stream) as st:
        if out_wcrt is None:
            out_wcrt = torch.empty(ts.n_tasks, dtype=torch.int64, device=dev)
        if out_sched is None:
            out_sched = torch.empty(max(ts.n_tasksets, 0), dtype=torch.uint8, device=dev)
        rc = lib.gcaps_rta_batch_static(ctypes.byref(ts.c), ts.n_tasksets, policy, timeslice_us,
                                        overhead_us, out_wcrt.data_ptr(), out_sched.data_ptr(),
                                        st.cuda_stream)
    _check(rc)
    return out_wcrt, out_sched


def rta_gpu_priority(ts: DeviceTasksets, flags: int = 0, overhead_us: int = 0, gpu_priority=None,
                     workspace=None, stream=None):
    """gcaps_rta_gpu_priority_batch: GCAPS with separate GPU-segment priorities.  ``gpu_priority``
    is an int64 CUDA tensor per task, or None together with ``ASSIGN`` in ``flags`` to search the
    priorities.  Returns ``(out_wcrt, out_sched, out_gpu_priority)`` CUDA tensors."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    with _device_and_stream(dev, stream) as st:
        out_wcrt = torch.full((ts.n_tasks,), WCRT_INVALID, dtype=torch.int64, device=dev)
        out_sched = torch.full((max(ts.n_tasksets, 0),), SCHED_INVALID, dtype=torch.uint8, device=dev)
        out_gp = torch.zeros(ts.n_tasks, dtype=torch.int64, device=dev)
        if workspace is None:
            workspace = torch.empty(max(workspace_bytes(ts.n_tasksets), 256), dtype=torch.uint8, device=dev)
        rc = lib.gcaps_rta_gpu_priority_batch(
            ctypes.byref(ts.c), ts.n_tasksets, flags, overhead_us,
            gpu_priority.data_ptr() if gpu_priority is not None else None, out_gp.data_ptr(),
            out_wcrt.data_ptr(), out_sched.data_ptr(), workspace.data_ptr(), workspace.numel(),
            st.cuda_stream)
    _check(rc)
    return out_wcrt, out_sched, out_gp


def generate_device(params: GenParams, first: int, count: int, device="cuda:0", stream=None,
                    timing=None) -> DeviceTasksets:
    """gcaps_gen_count + gcaps_gen_fill: tasksets ``first .. first+count-1`` of the stream, made
    on the device by the integer-only generator (the same tasksets as
    ``taskgen.generate(params, first, count, integer=True)``).  One 24-byte read-back of the array
    lengths sits between the two calls; nothing else crosses the host link.  ``timing``, if a
    dict, receives the device time of both calls in ms."""
    import torch
    lib = load_library()
    dev = torch.device(device)
    cp = params.int_params()
    with _device_and_stream(dev, stream) as st:
        ws = torch.empty(max(int(lib.gcaps_gen_workspace_bytes(ctypes.byref(cp), count)), 256), dtype=torch.uint8,
                         device=dev)
        totals = torch.zeros(3, dtype=torch.int64, device=dev)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if timing is not None else None
        if ev:
            ev[0].record(st)
        _check(lib.gcaps_gen_count(ctypes.byref(cp), first, count, totals.data_ptr(), ws.data_ptr(),
                                   ws.numel(), st.cuda_stream))
        if ev:
            ev[1].record(st)
        n_tasks, n_c, n_g = (int(x) for x in totals.cpu().tolist())
        sizes = {"task_off": max(count, 0) + 1, "period": n_tasks, "deadline": n_tasks,
                 "priority": n_tasks, "core": n_tasks, "cseg_off": n_tasks + 1, "cseg_wcet": n_c,
                 "gseg_off": n_tasks + 1, "gseg_misc": n_g, "gseg_exec": n_g}
        t = {f: torch.zeros(sizes[f], dtype=torch.int64, device=dev) for f in ARRAY_FIELDS}
        ts = DeviceTasksets(t)
        if ev:
            ev[2].record(st)
        _check(lib.gcaps_gen_fill(ctypes.byref(cp), first, count, ctypes.byref(ts.c), ws.data_ptr(),
                                  ws.numel(), st.cuda_stream))
        if ev:
            ev[3].record(st)
            torch.cuda.synchronize(dev)
            timing["count_ms"] = ev[0].elapsed_time(ev[1])
            timing["fill_ms"] = ev[2].elapsed_time(ev[3])
    return ts


def rta_plan(ts: DeviceTasksets, workspace, stream=None):
    """gcaps_rta_plan_batch: only the planning step of a call (for timing it apart)."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    with _device_and_stream(dev, stream) as st:
        rc = lib.gcaps_rta_plan_batch(ctypes.byref(ts.c), ts.n_tasksets, workspace.data_ptr(),
                                      workspace.numel(), st.cuda_stream)
    _check(rc)


def int_issue_rate(kind: int = 2, trips: int = 2048, repeats: int = 5, device="cuda:0") -> float:
    """Integer lane-operations per second of the device, measured with gcaps_rta_int_issue_probe
    (kind 0: multiply-add chains, 1: add chains, 2: both); best of ``repeats`` launches."""
    import torch
    lib = load_library()
    dev = torch.device(device)
    with torch.cuda.device(dev):
        scratch = torch.zeros(1, dtype=torch.int32, device=dev)
        st = torch.cuda.current_stream(dev)
        ops = ctypes.c_int64(0)
        best = None
        for k in range(repeats + 1):   # the first launch is a warm-up
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            _check(lib.gcaps_rta_int_issue_probe(kind, trips, scratch.data_ptr(), ctypes.byref(ops),
                                                 st.cuda_stream))
            e1.record(st)
            e1.synchronize()
            ms = e0.elapsed_time(e1)
            if k > 0 and (best is None or ms < best):
                best = ms
    return ops.value / (best * 1e-3)


def rta_validate(ts: DeviceTasksets, stream=None):
    """gcaps_rta_validate: int32 error mask per taskset (CUDA tensor)."""
    import torch
    lib = load_library()
    dev = ts.t["task_off"].device
    with _device_and_stream(dev, stream) as st:
        out = torch.empty(max(ts.n_tasksets, 0), dtype=torch.int32, device=dev)
        rc = lib.gcaps_rta_validate(ctypes.byref(ts.c), ts.n_tasksets, out.data_ptr(), st.cuda_stream)
    _check(rc)
    return out


def host_struct(arrays: Dict[str, np.ndarray]) -> Tuple[CTasksets, int]:
    """C struct over host arrays (numpy int64, contiguous); returns (struct, n_tasksets)."""
    for f in ARRAY_FIELDS:
        a = arrays[f]
        assert a.dtype == np.int64 and a.flags["C_CONTIGUOUS"], f
    c = CTasksets(arrays["period"].shape[0], arrays["cseg_wcet"].shape[0],
                  arrays["gseg_misc"].shape[0], *[arrays[f].ctypes.data for f in ARRAY_FIELDS])
    return c, int(arrays["task_off"].shape[0]) - 1


def rta_batch_host(arrays: Dict[str, np.ndarray], policy: int, timeslice_us: int = 1024,
                   overhead_us: int = 0, out_wcrt: Optional[np.ndarray] = None,
                   out_sched: Optional[np.ndarray] = None):
    """gcaps_rta_batch_host on host arrays (page-locked ones transfer fastest).  Synchronous.
    Returns ``(out_wcrt, out_sched)`` numpy arrays."""
    lib = load_library()
    c, n_tasksets = host_struct(arrays)
    if out_wcrt is None:
        out_wcrt = np.full(c.n_tasks, WCRT_INVALID, np.int64)
    if out_sched is None:
        out_sched = np.full(max(n_tasksets, 0), SCHED_INVALID, np.uint8)
    rc = lib.gcaps_rta_batch_host(ctypes.byref(c), n_tasksets, policy, timeslice_us, overhead_us,
                                  out_wcrt.ctypes.data, out_sched.ctypes.data)
    _check(rc)
    return out_wcrt, out_sched


def rta_batch_host_multi(arrays: Dict[str, np.ndarray], policies, timeslice_us: int = 1024,
                         overhead_us: int = 0, out_wcrt=None, out_sched=None):
    """gcaps_rta_batch_host_multi: one copy of the host arrays to the device, one analysis per
    entry of ``policies``.  Returns ``(list of out_wcrt, list of out_sched)`` numpy arrays."""
    lib = load_library()
    c, n_tasksets = host_struct(arrays)
    k = len(policies)
    if out_wcrt is None:
        out_wcrt = [np.full(c.n_tasks, WCRT_INVALID, np.int64) for _ in range(k)]
    if out_sched is None:
        out_sched = [np.full(max(n_tasksets, 0), SCHED_INVALID, np.uint8) for _ in range(k)]
    pol = (ctypes.c_int * k)(*policies)
    pw = (ctypes.c_void_p * k)(*[a.ctypes.data for a in out_wcrt])
    ps = (ctypes.c_void_p * k)(*[a.ctypes.data for a in out_sched])
    rc = lib.gcaps_rta_batch_host_multi(ctypes.byref(c), n_tasksets, pol, k, timeslice_us,
                                        overhead_us, pw, ps)
    _check(rc)
    return out_wcrt, out_sched


def release_host():
    load_library().gcaps_rta_release_host()
