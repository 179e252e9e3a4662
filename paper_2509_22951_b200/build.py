"""Builds libtq.so (host C++ + CUDA sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libtq.so"
SOURCES = [CSRC / "tq_device.cu", CSRC / "tq_gemm.cu", CSRC / "tq_gemm_ws.cu", CSRC / "tq_tiles.cu", CSRC / "tq_wide.cu", CSRC / "tq_encode.cu", CSRC / "tq_dict_device.cu", CSRC / "tq_host.cpp"]
HEADERS = [CSRC / "tq_internal.h", CSRC / "tq_sm100.cuh", CSRC / "tq_tiles_common.cuh", ROOT / "include" / "tq.h"]


def _nvcc() -> str | None:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    return cand if os.path.exists(cand) else None


def is_stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(p.stat().st_mtime > t for p in SOURCES + HEADERS if p.exists())


def build_library(force: bool = False, verbose: bool = False) -> Path:
    # a prebuilt library elsewhere (deployments without nvcc): TQ_LIBTQ=/path/to/libtq.so
    prebuilt = os.environ.get("TQ_LIBTQ")
    if prebuilt and not force:
        if not os.path.exists(prebuilt):
            raise RuntimeError(f"TQ_LIBTQ={prebuilt} does not exist")
        return Path(prebuilt)
    if not force and not is_stale():
        return LIB
    nvcc = _nvcc()
    if nvcc is None:
        raise RuntimeError("libtq.so is missing or stale and nvcc was not found; cannot build the CUDA library")
    tmp = LIB.with_name(f"libtq.tmp{os.getpid()}.so")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC,-O3,-pthread", "-shared", "-I", str(ROOT / "include"), "-I", str(CSRC),
           "-o", str(tmp)] + [str(s) for s in SOURCES] + ["-lpthread"]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv))
