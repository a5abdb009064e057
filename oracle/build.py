"""Compiles the oracle's C sources (gcc) into shared objects beside them."""
from __future__ import annotations

import os
import subprocess
import threading

_HERE = os.path.dirname(os.path.abspath(__file__))
_lock = threading.Lock()


def build(name: str, force: bool = False) -> str:
    """Builds ``<name>.c`` into ``_<name>.so`` if missing or stale; returns the .so path."""
    src = os.path.join(_HERE, name + ".c")
    lib = os.path.join(_HERE, "_" + name + ".so")
    with _lock:
        if force or not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(src):
            tmp = lib + ".%d.tmp" % os.getpid()
            subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", tmp, src])
            os.replace(tmp, lib)
    return lib


def build_all(force: bool = False) -> None:
    for name in ("rta_oracle", "gpu_prio_oracle", "des_sim"):
        build(name, force)


if __name__ == "__main__":
    build_all(True)
