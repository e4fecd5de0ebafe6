"""TEST INFRASTRUCTURE: compiles the plain-C oracle into a shared library with gcc."""
from __future__ import annotations

import hashlib
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "zl_oracle.c")


def _host_tag() -> str:
    """The library is built with -march=native, so key it by the host's CPU flags and the
    source text: a copy built on another machine is never loaded by mistake."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(SRC, "rb") as f:
        src = f.read()
    return hashlib.sha1(flags.encode() + src).hexdigest()[:12]


def lib_path() -> str:
    return os.path.join(_HERE, f"libzl_oracle_{_host_tag()}.so")


def build(force: bool = False) -> str:
    lib = lib_path()
    if not force and os.path.exists(lib):
        return lib
    # No -ffast-math: summation order stays the order written in the source.
    tmp = f"{lib}.{os.getpid()}.tmp"
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-march=native",
           "-fno-fast-math", "-o", tmp, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True))
