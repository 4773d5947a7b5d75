"""ctypes front end of the C oracle (``conv2d_ref.c``) -- test infrastructure only.

The oracle is the definition of the operation written out as seven nested
loops with double accumulation (the paper's Fig. 3a problem statement with the
top-left anchored, un-flipped reading of Section 3.1 and Algorithm 2).  This
module only compiles the C file with gcc, marshals numpy arrays and returns
numpy arrays; it contains no arithmetic of its own.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "conv2d_ref.c"
_LIB = _HERE / "_build" / "libconv2d_oracle.so"
_lib = None

MODE_EXACT = 0      # fp32 operands as given
MODE_TF32_RNA = 1   # operands rounded to TF32, nearest / ties away
MODE_TF32_TRUNC = 2  # operands truncated to TF32


def build(force: bool = False) -> Path:
    """Compile the C oracle (gcc -O2 -fopenmp) if the library is missing or stale."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    _LIB.parent.mkdir(parents=True, exist_ok=True)
    tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
           "-ffp-contract=off", "-o", str(tmp), str(_SRC), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        i = ctypes.c_int
        lib.conv2d_oracle_range.argtypes = [fp, fp, dp, dp] + [i] * 7 + [i] * 6 + [i]
        lib.conv2d_oracle_range.restype = i
        lib.conv2d_oracle_threads.argtypes = []
        lib.conv2d_oracle_threads.restype = i
        _lib = lib
    return _lib


def oracle_threads() -> int:
    """Number of host threads the oracle's OpenMP loop uses."""
    return int(_load().conv2d_oracle_threads())


def conv2d_oracle_range(x, w, n_range=None, k_range=None, p_range=None, mode=MODE_EXACT):
    """Oracle outputs for a sub-range of images, maps and output rows.

    x: float32 [N,C,H,W]; w: float32 [K,C,R,S].  Returns ``(y64, yabs)`` as
    float64 arrays of shape [n,k,p,Q] restricted to the requested half-open
    ranges (full extent where a range is None).  ``yabs`` is the sum of the
    absolute values of the products, the scale of the parity tolerance.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    if x.ndim != 4 or w.ndim != 4 or x.shape[1] != w.shape[1]:
        raise ValueError("expected x[N,C,H,W] and w[K,C,R,S] with equal C")
    N, C, H, W = x.shape
    K, _, R, S = w.shape
    if R > H or S > W:
        raise ValueError("filter larger than image")
    P, Q = H - R + 1, W - S + 1
    n0, n1 = n_range if n_range is not None else (0, N)
    k0, k1 = k_range if k_range is not None else (0, K)
    p0, p1 = p_range if p_range is not None else (0, P)
    shape = (n1 - n0, k1 - k0, p1 - p0, Q)
    y64 = np.empty(shape, dtype=np.float64)
    yabs = np.empty(shape, dtype=np.float64)
    fp = ctypes.POINTER(ctypes.c_float)
    dp = ctypes.POINTER(ctypes.c_double)
    rc = _load().conv2d_oracle_range(
        x.ctypes.data_as(fp), w.ctypes.data_as(fp),
        y64.ctypes.data_as(dp), yabs.ctypes.data_as(dp),
        N, C, H, W, K, R, S, n0, n1, k0, k1, p0, p1, int(mode))
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (code {rc})")
    return y64, yabs


def conv2d_oracle(x, w, mode=MODE_EXACT):
    """Oracle outputs for the whole problem: ``(y64, yabs)``, each [N,K,P,Q] float64."""
    return conv2d_oracle_range(x, w, mode=mode)
