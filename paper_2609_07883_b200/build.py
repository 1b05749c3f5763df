"""Build ``libsloweave.so`` from ``csrc/`` with nvcc for sm_100a (in-tree, next to this file)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
INCLUDE = HERE.parent / "include"
LIB = HERE / "libsloweave.so"
SOURCES = ["sw_error.cpp", "sw_controller.cpp", "sw_telemetry.cpp", "sw_api.cu", "sw_kernels.cu", "sw_static.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.iterdir()) + list(INCLUDE.iterdir()) + [Path(__file__)]
    return any(p.stat().st_mtime > t for p in deps)


def build(force: bool = False, verbose: bool = False, defines=(), out: Path | None = None) -> Path:
    """Compile every source for sm_100a and link the shared library.  cudart is linked statically and the one
    driver function needed (tensor-map encode) is resolved at run time, so the library loads without a GPU."""
    lib = Path(out) if out is not None else LIB
    if out is None and not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = HERE / "build" / (lib.stem if out is not None else "default")
    objdir.mkdir(parents=True, exist_ok=True)
    common = [nvcc, "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I", str(INCLUDE), "-I", str(CSRC)] + ARCH + [f"-D{d}" for d in defines]
    if verbose:
        common += ["-Xptxas", "-v"]
    objs = []
    procs = []
    for src in SOURCES:
        obj = objdir / (src + ".o")
        objs.append(str(obj))
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
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    subprocess.check_call([nvcc, "-shared", "-o", str(tmp)] + objs + ARCH + ["-cudart", "static"])
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
