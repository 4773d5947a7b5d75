"""Counter-based seeded generators for the benchmark configurations.

Every element ``i`` of a tensor drawn under ``seed`` is a pure function of
``(seed, stream, i)`` through a 64-bit mixing function, so values do not depend
on generation order, chunking or thread count.  The paper publishes shapes
only (image size, filter size, channel and filter counts of its Fig. 7 and
Fig. 9 sweeps); the value distributions below are the ones the benchmark
configurations name.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on an array of uint64 counters."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
        return z ^ (z >> _U64(31))


def _bits(seed: int, stream: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        base = _mix64(np.array([seed], dtype=_U64) * _GOLDEN + _U64(stream))
        ctr = np.arange(count, dtype=_U64) * _GOLDEN + base
    return _mix64(ctr)


def _unit(seed: int, stream: int, count: int) -> np.ndarray:
    """float64 in [0,1) with 24 random bits (exactly representable in fp32)."""
    return (_bits(seed, stream, count) >> _U64(40)).astype(np.float64) * (2.0 ** -24)


def uniform(shape, seed: int, lo: float = -1.0, hi: float = 1.0) -> np.ndarray:
    n = int(np.prod(shape))
    u = _unit(seed, 0, n)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(shape, seed: int, std: float = 1.0) -> np.ndarray:
    """N(0, std^2) by Box-Muller in float64, rounded once to fp32."""
    n = int(np.prod(shape))
    u1 = ((_bits(seed, 1, n) >> _U64(40)).astype(np.float64) + 1.0) * (2.0 ** -24)  # (0,1]
    u2 = _unit(seed, 2, n)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (std * z).astype(np.float32).reshape(shape)


def relu_normal(shape, seed: int) -> np.ndarray:
    """max(N(0,1), 0): about half the entries are exact zeros."""
    return np.maximum(normal(shape, seed, 1.0), np.float32(0.0))


def small_integers(shape, seed: int, bound: int = 4) -> np.ndarray:
    """Integers in [-bound, bound] as fp32: exact in fp32 and in TF32."""
    n = int(np.prod(shape))
    v = (_bits(seed, 3, n) >> _U64(33)) % _U64(2 * bound + 1)
    return (v.astype(np.int64) - bound).astype(np.float32).reshape(shape)


@dataclass(frozen=True)
class ConvShape:
    name: str
    N: int
    C: int
    H: int
    W: int
    K: int
    R: int
    S: int
    x_dist: str      # "uniform_pm1" | "uniform_01" | "relu_normal"
    w_std: float     # 0 => uniform in [-1,1)
    seed: int

    @property
    def P(self) -> int:
        return self.H - self.R + 1

    @property
    def Q(self) -> int:
        return self.W - self.S + 1

    @property
    def flops(self) -> int:
        return 2 * self.N * self.K * self.C * self.R * self.S * self.P * self.Q

    @property
    def compulsory_bytes(self) -> int:
        """Each input, weight and output element moved once, 4 bytes each."""
        return 4 * (self.N * self.C * self.H * self.W + self.K * self.C * self.R * self.S
                    + self.N * self.K * self.P * self.Q)

    def as_dict(self) -> dict:
        return dict(N=self.N, C=self.C, H=self.H, W=self.W, K=self.K, R=self.R, S=self.S)


def _cfg5(r: int) -> ConvShape:
    return ConvShape(f"cfg5_r{r}", 64, 128, 32, 32, 128, r, r, "uniform_01",
                     (1.0 / (128 * r * r)) ** 0.5, 5 + 10 * r)


# The five benchmark configurations (cfg5 is a sweep over the filter size).
CONFIGS = {
    "cfg1": ConvShape("cfg1", 1, 1, 64, 64, 8, 3, 3, "uniform_pm1", 0.0, 1),
    "cfg2": ConvShape("cfg2", 1, 1, 4096, 4096, 32, 5, 5, "uniform_pm1", 0.2, 2),
    "cfg3": ConvShape("cfg3", 32, 64, 56, 56, 64, 3, 3, "relu_normal", (2.0 / (64 * 9)) ** 0.5, 3),
    "cfg4": ConvShape("cfg4", 32, 256, 14, 14, 256, 3, 3, "relu_normal", (2.0 / (256 * 9)) ** 0.5, 4),
    # profiling-size stand-in for cfg2 (same kernel instance, output 536 MB: still far beyond L2)
    "cfg2_half": ConvShape("cfg2_half", 1, 1, 2048, 2048, 32, 5, 5, "uniform_pm1", 0.2, 2),
    "cfg5_r1": _cfg5(1),
    "cfg5_r3": _cfg5(3),
    "cfg5_r5": _cfg5(5),
    "cfg5_r7": _cfg5(7),
}


def make_inputs(cfg: ConvShape, batch: int | None = None):
    """(x[N,C,H,W], w[K,C,R,S]) float32 numpy arrays for a configuration.

    ``batch`` overrides N (a smaller batch of the same per-image distribution).
    """
    n = cfg.N if batch is None else batch
    xs = (n, cfg.C, cfg.H, cfg.W)
    ws = (cfg.K, cfg.C, cfg.R, cfg.S)
    if cfg.x_dist == "uniform_pm1":
        x = uniform(xs, 1000 + cfg.seed)
    elif cfg.x_dist == "uniform_01":
        x = uniform(xs, 1000 + cfg.seed, 0.0, 1.0)
    elif cfg.x_dist == "relu_normal":
        x = relu_normal(xs, 1000 + cfg.seed)
    else:
        raise ValueError(cfg.x_dist)
    w = uniform(ws, 2000 + cfg.seed) if cfg.w_std == 0.0 else normal(ws, 2000 + cfg.seed, cfg.w_std)
    return x, w
