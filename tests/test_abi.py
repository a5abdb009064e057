"""The C-ABI library loads and exports every symbol include/gcaps_rta.h declares (no GPU work)."""
import ctypes
import os
import re

import pytest

from paper_2406_05221_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gcaps_rta.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gcaps_(?:rta|gen)_[a-z_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    build.build_cuda()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert set(names) == set(binding.EXPORTS)
    for name in names:
        assert getattr(lib, name) is not None


def test_host_only_entry_points(lib):
    assert lib.gcaps_rta_version() == 100
    assert binding.workspace_bytes(0) == 0 and binding.workspace_bytes(-5) == 0
    small, big = binding.workspace_bytes(1), binding.workspace_bytes(1_000_000)
    assert small >= 4 and big >= 4 * 1_000_000 and big % 256 == 0
    from paper_2406_05221_b200 import taskgen
    gp = taskgen.WORKLOADS["large"].streams[0].int_params()
    assert lib.gcaps_gen_workspace_bytes(ctypes.byref(gp), 0) == 0
    big = lib.gcaps_gen_workspace_bytes(ctypes.byref(gp), 1000)
    assert big % 256 == 0 and big >= 1000 * (4 + 3 * 80) * 4
    for code in (0, -1, -2, -3, -4, -99):
        assert lib.gcaps_rta_strerror(code)


def test_header_constants_match_binding():
    text = open(os.path.join(ROOT, "include", "gcaps_rta.h")).read()
    def const(name):
        m = re.search(r"#define\s+%s\s+\(?(-?[0-9a-fx]+)\)?" % name, text)
        return int(m.group(1), 0)
    assert const("GCAPS_POLICY_GCAPS") == binding.POLICY_GCAPS
    assert const("GCAPS_POLICY_RR") == binding.POLICY_RR
    assert const("GCAPS_RTA_BUSY") == binding.BUSY and const("GCAPS_RTA_LITERAL") == binding.LITERAL
    assert const("GCAPS_WCRT_MISS") == binding.WCRT_MISS
    assert const("GCAPS_WCRT_SKIPPED") == binding.WCRT_SKIPPED
    assert const("GCAPS_WCRT_ITER_LIMIT") == binding.WCRT_ITER_LIMIT
    assert const("GCAPS_WCRT_INVALID") == binding.WCRT_INVALID
    assert const("GCAPS_RTA_MAX_TASKS") == binding.MAX_TASKS
    assert ctypes.sizeof(binding.CTasksets) == 13 * 8


def test_argument_errors_need_no_device(lib):
    """Argument checks come before any CUDA call, so they can be exercised without a GPU."""
    c = binding.CTasksets()
    bad = [dict(n=-1, policy=0, L=1, ovh=0), dict(n=1, policy=7, L=1, ovh=0),
           dict(n=1, policy=0x400, L=1, ovh=0), dict(n=1, policy=1, L=0, ovh=0),
           dict(n=1, policy=0, L=1, ovh=-1), dict(n=1, policy=0, L=1, ovh=(1 << 40) + 1),
           dict(n=1, policy=0, L=1, ovh=0)]  # last: null task_off
    for kw in bad:
        rc = lib.gcaps_rta_batch(ctypes.byref(c), kw["n"], kw["policy"], kw["L"], kw["ovh"],
                                 None, None, None, 0, None)
        assert rc == binding.ERR_INVALID_ARG, kw
        rc = lib.gcaps_rta_batch_host(ctypes.byref(c), kw["n"], kw["policy"], kw["L"], kw["ovh"],
                                      None, None)
        assert rc == binding.ERR_INVALID_ARG, kw
    assert lib.gcaps_rta_batch(None, 0, 0, 1, 0, None, None, None, 0, None) == binding.ERR_INVALID_ARG
    assert lib.gcaps_rta_batch(ctypes.byref(c), 0, 0, 1, 0, None, None, None, 0, None) == binding.OK


def test_host_only_calls_from_several_threads(lib):
    """The entry points may be called from several host threads at once; what can be checked
    without a device: argument errors and the pure host computations give the same answers."""
    import threading
    want = [binding.workspace_bytes(n) for n in range(0, 200_000, 997)]
    c = binding.CTasksets()
    wrong = []

    def run():
        for _ in range(20):
            if [binding.workspace_bytes(n) for n in range(0, 200_000, 997)] != want:
                wrong.append("workspace_bytes")
            for call in (lambda: lib.gcaps_rta_batch(ctypes.byref(c), 1, 7, 1, 0, None, None, None, 0, None),
                         lambda: lib.gcaps_rta_batch_host(ctypes.byref(c), 1, 0, 1, -1, None, None),
                         lambda: lib.gcaps_rta_batch_static(ctypes.byref(c), 1, 1, 0, 0, None, None, None)):
                if call() != binding.ERR_INVALID_ARG:
                    wrong.append("argument error")

    threads = [threading.Thread(target=run) for _ in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not wrong, wrong
