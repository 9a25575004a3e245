"""Counter-based seeded number streams (no op arithmetic lives here)."""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on an array of uint64 words (wrap-around arithmetic)."""
    z = np.asarray(z, dtype=np.uint64).copy()
    with np.errstate(over="ignore"):
        z ^= z >> np.uint64(30)
        z *= _M1
        z ^= z >> np.uint64(27)
        z *= _M2
        z ^= z >> np.uint64(31)
    return z


def _words(seed: int, stream: int, count: int, lane: int = 0) -> np.ndarray:
    """`count` 64-bit words for (seed, stream); `lane` selects an independent sub-stream."""
    with np.errstate(over="ignore"):
        key = mix64(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)]))[0]
        key = mix64(np.array([key ^ np.uint64((stream * 2 + lane + 1) & 0xFFFFFFFFFFFFFFFF)]))[0]
        idx = np.arange(1, count + 1, dtype=np.uint64)
        return mix64(key + idx * _GOLDEN)


def uniform(seed: int, stream: int, shape, lo: float, hi: float) -> np.ndarray:
    """fp32 tensor of i.i.d. uniform[lo, hi) values (24-bit fraction, half-open)."""
    count = int(np.prod(shape)) if len(shape) else 1
    frac = (_words(seed, stream, count) >> np.uint64(40)).astype(np.float64) * (1.0 / (1 << 24))
    out = (lo + (hi - lo) * frac).astype(np.float32)
    # the fp32 cast may round the largest fractions up to `hi`; keep the interval half-open
    top = np.nextafter(np.float32(hi), np.float32(lo))
    np.minimum(out, top, out=out)
    return out.reshape(shape)


def normal(seed: int, stream: int, shape, mean: float, std: float) -> np.ndarray:
    """fp32 tensor of i.i.d. N(mean, std^2) values (Box-Muller in float64, untruncated)."""
    count = int(np.prod(shape)) if len(shape) else 1
    w1 = _words(seed, stream, count, lane=0)
    w2 = _words(seed, stream, count, lane=1)
    u1 = ((w1 >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / (1 << 53))  # (0, 1]
    u2 = (w2 >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))  # [0, 1)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)


def small_integers(seed: int, stream: int, shape, lo: int, hi: int) -> np.ndarray:
    """fp32 tensor of integers drawn uniformly from {lo, ..., hi} (inclusive)."""
    count = int(np.prod(shape)) if len(shape) else 1
    span = np.uint64(hi - lo + 1)
    vals = (_words(seed, stream, count) >> np.uint64(20)) % span
    return (vals.astype(np.int64) + lo).astype(np.float32).reshape(shape)
