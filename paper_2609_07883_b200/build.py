"""Build ``libsloweave.so`` from ``csrc/`` with nvcc for sm_100a (in-tree, next to this file).

``build_sanitized()`` links a second file, ``libsloweave_asan.so``, whose host-only sources (controller, telemetry,
error text) are compiled with ``-fsanitize=address,undefined``; the CPU tests are replayed against it (see
``tests/test_sanitizers.py``).  The device sources are the same objects in both files."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
INCLUDE = HERE.parent / "include"
LIB = HERE / "libsloweave.so"
LIB_SANITIZED = HERE / "libsloweave_asan.so"
HOST_SOURCES = ["sw_error.cpp", "sw_controller.cpp", "sw_telemetry.cpp"]
DEVICE_SOURCES = ["sw_api.cu", "sw_kernels.cu", "sw_static.cu"]
SOURCES = HOST_SOURCES + DEVICE_SOURCES
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
SANITIZE = ["-fsanitize=address,undefined", "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer", "-g", "-O1"]


def _nvcc() -> str:
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def _stale(lib: Path) -> bool:
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    deps = list(CSRC.iterdir()) + list(INCLUDE.iterdir()) + [Path(__file__)]
    return any(p.stat().st_mtime > t for p in deps)


def _objdir() -> Path:
    d = HERE / "build" / "default"
    d.mkdir(parents=True, exist_ok=True)
    return d


def _link(lib: Path, objs) -> Path:
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    subprocess.check_call([_nvcc(), "-shared", "-o", str(tmp)] + [str(o) for o in objs] + ARCH + ["-cudart", "static"])
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every source for sm_100a and link the shared library.  cudart is linked statically and the one
    driver function needed (tensor-map encode) is resolved at run time, so the library loads without a GPU."""
    if not force and not _stale(LIB):
        return LIB
    objdir = _objdir()
    common = [_nvcc(), "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I", str(INCLUDE), "-I", str(CSRC)] + ARCH
    if verbose:
        common += ["-Xptxas", "-v"]
    objs = []
    procs = []
    for src in SOURCES:
        obj = objdir / (src + ".o")
        objs.append(obj)
        cmd = common + (["-x", "cu"] if src.endswith(".cu") else []) + ["-c", str(CSRC / src), "-o", str(obj)]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, pr in procs:
        out, _ = pr.communicate()
        if pr.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src} ---\n{out}\n")
        failed = failed or pr.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    return _link(LIB, objs)


def build_sanitized(force: bool = False) -> Path:
    """The library with its host-only sources instrumented by AddressSanitizer and UndefinedBehaviorSanitizer (gcc).
    The sanitizer runtimes are not linked in: the process that loads this file has to start with them preloaded
    (``sanitizer_env()``)."""
    build(force=force)
    if not force and not _stale(LIB_SANITIZED) and LIB_SANITIZED.stat().st_mtime >= LIB.stat().st_mtime:
        return LIB_SANITIZED
    objdir = _objdir()
    objs = []
    for src in HOST_SOURCES:
        obj = objdir / (src + ".asan.o")
        subprocess.check_call(["g++", "-std=c++17", "-fPIC", "-I", str(INCLUDE), "-I", str(CSRC)] + SANITIZE +
                              ["-c", str(CSRC / src), "-o", str(obj)])
        objs.append(obj)
    objs += [objdir / (src + ".o") for src in DEVICE_SOURCES]
    return _link(LIB_SANITIZED, objs)


def sanitizer_env() -> dict:
    """Environment for a process that loads the instrumented libraries: the two runtimes preloaded, errors fatal, leak
    checking off (the interpreter itself never frees everything)."""
    runtimes = [subprocess.check_output(["gcc", f"-print-file-name={name}"], text=True).strip()
                for name in ("libasan.so", "libubsan.so")]
    env = dict(os.environ)
    env["LD_PRELOAD"] = ":".join(runtimes)
    env["ASAN_OPTIONS"] = "detect_leaks=0:abort_on_error=1"
    env["UBSAN_OPTIONS"] = "halt_on_error=1:print_stacktrace=1"
    return env


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
