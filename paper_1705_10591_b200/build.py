"""Builds libconv2d_b200.so (the C-ABI library) in-tree with nvcc for sm_100a.

Usage: python -m paper_1705_10591_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
CSRC = PKG / "csrc"
LIB = PKG / "libconv2d_b200.so"
SOURCES = ["conv2d_api.cu", "single_channel.cu", "general_ffma.cu", "general_ffma_r1.cu", "general_ffma_r2.cu",
           "general_ffma_r3.cu", "general_ffma_r4.cu", "general_ffma_r5.cu", "general_ffma_r7.cu", "general_tf32.cu",
           "pointwise_tma.cu"]


def _stale() -> bool:
    if not LIB.exists():
        return True
    built = LIB.stat().st_mtime
    deps = [CSRC / s for s in SOURCES] + list(CSRC.glob("*.cuh")) + [ROOT / "include" / "conv2d_b200.h"]
    return any(d.stat().st_mtime > built for d in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compiles every source to an object file (in parallel) and links the shared library."""
    if not force and not _stale():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    import tempfile

    common = [
        "nvcc", "-std=c++17", "-O3", "-lineinfo",
        "-gencode", "arch=compute_100a,code=sm_100a",
        "-Xcompiler", "-fPIC",
        "-I", str(ROOT / "include"), "-I", str(CSRC),
        "-DCONV2D_B200_BUILD",
    ]
    if verbose:
        common.insert(1, "-Xptxas=-v")
    if os.environ.get("CONV2D_B200_BUILD_DIAGNOSTICS"):
        # tuning build: the tensor-core kernel's MMA thread counts its cycles into status words 2-9
        common.append("-DCONV2D_B200_TC_DIAGNOSTICS")
    with tempfile.TemporaryDirectory(prefix="conv2d_b200_build_") as tmp:
        objs = [str(Path(tmp) / (Path(s).stem + ".o")) for s in SOURCES]

        def compile_one(job):
            src, obj = job
            return subprocess.run(common + ["-c", str(CSRC / src), "-o", obj], capture_output=True, text=True)

        with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
            results = list(pool.map(compile_one, zip(SOURCES, objs)))
        for res in results:
            if verbose:
                sys.stderr.write(res.stderr)
            if res.returncode != 0:
                raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
        link = ["nvcc", "-shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                "-o", str(LIB)] + objs
        res = subprocess.run(link, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc (link) failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
