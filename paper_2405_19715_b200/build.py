"""Builds libspecdec.so (sm_100a) in-tree with nvcc.  `python -m paper_2405_19715_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libspecdec.so"
SOURCES = ["api.cu", "verify.cu", "verify_stream.cu", "stop.cu", "head.cu", "verify_static.cu", "greedy.cu", "topk.cu", "verify_shard.cu", "verify_cluster.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not Path(nvcc).exists():
        raise RuntimeError("nvcc not found: libspecdec cannot be built")
    return nvcc


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) + [ROOT / "include" / "specdec.h"]
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False, stamps: bool = False) -> Path:
    """Regular build: libspecdec.so.  stamps=True: the diagnostic build libspecdec_stamps.so, compiled with
    -DSPECDEC_STAMPS (phase timestamps inside the verify/correct kernel); it is always rebuilt."""
    if stamps:
        return _compile(PKG / "libspecdec_stamps.so", PKG / "_build" / "stamps", ["-DSPECDEC_STAMPS"], verbose)
    if not force and not needs_build():
        return LIB
    return _compile(LIB, PKG / "_build", [], verbose)


def _compile(LIB: Path, obj_dir: Path, defines: list, verbose: bool) -> Path:
    obj_dir.mkdir(parents=True, exist_ok=True)
    nvcc = _nvcc()
    inc = ["-I", str(ROOT / "include"), "-I", str(CSRC)]
    extra = (["-Xptxas", "-v"] if verbose else []) + defines
    procs = []
    for src in SOURCES:
        cmd = [nvcc, *NVCC_FLAGS, *extra, *inc, "-c", str(CSRC / src), "-o", str(obj_dir / (src + ".o"))]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {src}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed building libspecdec")
    tmp = LIB.with_suffix(".so.tmp%d" % os.getpid())
    cmd = [nvcc, "-shared", "-Wno-deprecated-gpu-targets", "-o", str(tmp), *[str(obj_dir / (s + ".o")) for s in SOURCES], "-lcudart"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, stamps="--stamps" in sys.argv))
