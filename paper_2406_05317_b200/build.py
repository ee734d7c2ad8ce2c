"""Builds the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "liblococo.so"
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
NVCC_FLAGS = [*ARCH, "-lineinfo", "-O3", "-std=c++17", "--use_fast_math", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def sources():
    return sorted(CSRC.glob("*.cu"))


def stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*")) + list(INCLUDE.glob("*.h"))
    return any(p.stat().st_mtime > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every .cu under csrc/ into liblococo.so (object per source, then link)."""
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = PKG / "_build"
    objdir.mkdir(exist_ok=True)
    objs, procs = [], []
    for src in sources():
        obj = objdir / (src.stem + ".o")
        objs.append(obj)
        cmd = [nvcc, *NVCC_FLAGS, "-I", str(INCLUDE), "-I", str(CSRC), "-c", str(src), "-o", str(obj)]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    log = []
    failed = None
    for src, p in procs:
        out, _ = p.communicate()
        log.append(f"== {src.name}\n{out}")
        if p.returncode != 0 and failed is None:
            failed = src.name
    (objdir / "ptxas.log").write_text("\n".join(log))
    if failed:
        sys.stderr.write("\n".join(log))
        raise RuntimeError(f"nvcc failed on {failed}")
    if verbose:
        print("\n".join(log))
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    subprocess.check_call([nvcc, *ARCH, "-shared", "-o", str(tmp), *map(str, objs), "-lcuda"])
    os.replace(tmp, LIB)
    return LIB


PROBE_SRC = PKG.parent / "tests" / "cuda" / "wait_probe.cu"
PROBE_LIB = PKG.parent / "tests" / "cuda" / "libwait_probe.so"


def build_test_probe(force: bool = False) -> Path:
    """Compile the test-only library (a kernel whose bounded wait is made to run out) next to its source.
    It is not part of liblococo.so and exports nothing the header declares."""
    deps = [PROBE_SRC, CSRC / "tc_common.cuh"]
    if not force and PROBE_LIB.exists() and all(p.stat().st_mtime <= PROBE_LIB.stat().st_mtime for p in deps):
        return PROBE_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = PROBE_LIB.with_suffix(f".{os.getpid()}.tmp")
    subprocess.check_call([nvcc, *ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-shared", "-I", str(CSRC),
                           "-o", str(tmp), str(PROBE_SRC)])
    os.replace(tmp, PROBE_LIB)
    return PROBE_LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
    build_test_probe(force="--force" in sys.argv)
    print(LIB)
