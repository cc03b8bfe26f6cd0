"""Seeded synthetic inputs for the DAB-Net inference hot path.

This module only *draws numbers*.  It holds none of the method's arithmetic (no
sorting, thresholds, masks, popcounts or rescales), so the CPU checker and the
CUDA library can both be fed from it without sharing any code of the method.

Every array is a pure function of (seed, stream id, element index) through a
counter-based generator (splitmix64 finaliser over a 64-bit counter), so any
sub-range can be regenerated independently and the order in which tensors are
requested does not matter.

The paper trains on free-hand sketch datasets (TU-Berlin, Sketchy), which it
describes as sparse and binary (Section 5).  Those datasets are replaced here by
synthetic tensors of the same shapes and sparsity: post-ReLU activations are
half-normal with 60 % exact zeros, stroke images are a zero background with
~5 % of the pixels set to one along random polylines.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

DEFAULT_SEED = 180402941

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 18


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function (Steele, Lea, Flood 2014), elementwise on uint64, in place."""
    t = z >> np.uint64(30)
    z ^= t
    z *= _M1
    np.right_shift(z, np.uint64(27), out=t)
    z ^= t
    z *= _M2
    np.right_shift(z, np.uint64(31), out=t)
    z ^= t
    return z


def _stream_key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)], dtype=np.uint64))
        k = _mix(k + np.uint64(stream & 0xFFFFFFFFFFFFFFFF) * _GOLDEN + np.uint64(1))
    return k[0]


def raw_u64(seed: int, stream: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """64 random bits for counters start..start+count-1 of (seed, stream, lane)."""
    key = _stream_key(seed, stream * 8 + lane)
    with np.errstate(over="ignore"):
        ctr = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        ctr *= _GOLDEN
        ctr += key
        return _mix(ctr)


def uniform01(seed: int, stream: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """float64 uniform in the open interval (0, 1): (top 53 bits + 0.5) / 2^53."""
    u = raw_u64(seed, stream, start, count, lane)
    u >>= np.uint64(11)
    f = u.astype(np.float64)
    f += 0.5
    f *= 1.0 / 9007199254740992.0
    return f


def _normal_block(seed, stream, start, count):
    u1 = uniform01(seed, stream, start, count, lane=0)
    u2 = uniform01(seed, stream, start, count, lane=1)
    np.log(u1, out=u1)
    u1 *= -2.0
    np.sqrt(u1, out=u1)
    u2 *= 2.0 * np.pi
    np.cos(u2, out=u2)
    u1 *= u2
    return u1


def _fill(shape, fn) -> np.ndarray:
    """Evaluates fn(start, count) over chunks of the flattened array (chunks are independent: any order)."""
    total = int(np.prod(shape, dtype=np.int64)) if len(shape) else 1
    out = np.empty(total, dtype=np.float32)

    def one(s):
        c = min(_CHUNK, total - s)
        out[s:s + c] = fn(s, c)

    starts = range(0, total, _CHUNK)
    if len(starts) <= 1:
        for s in starts:
            one(s)
    else:
        with ThreadPoolExecutor(max_workers=min(len(starts), os.cpu_count() or 1, 16)) as ex:
            list(ex.map(one, starts))
    return out.reshape(shape)


def normal(shape, std: float, seed: int = DEFAULT_SEED, stream: int = 0, mean: float = 0.0) -> np.ndarray:
    """fp32 N(mean, std^2) (Box-Muller on two counter-based uniforms)."""
    return _fill(tuple(shape), lambda s, c: mean + std * _normal_block(seed, stream, s, c))


def laplace(shape, b: float, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
    """fp32 Laplace(0, b) by inverse CDF."""
    def blk(s, c):
        u = uniform01(seed, stream, s, c, lane=0) - 0.5
        return -b * np.sign(u) * np.log1p(-2.0 * np.abs(u))
    return _fill(tuple(shape), blk)


def relu_activations(shape, zero_frac: float = 0.6, seed: int = DEFAULT_SEED, stream: int = 0,
                     scale: float = 1.0) -> np.ndarray:
    """fp32 half-normal |N(0, scale^2)| with an independent Bernoulli(zero_frac) mask to exact 0.0."""
    def blk(s, c):
        v = np.abs(_normal_block(seed, stream, s, c)) * scale
        z = uniform01(seed, stream, s, c, lane=2) < zero_frac
        v[z] = 0.0
        return v
    return _fill(tuple(shape), blk)


def dense_activations(shape, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
    """fp32 N(0,1) without zeros (residual-style input: shows the cost without the sparsity lever)."""
    return normal(shape, 1.0, seed, stream)


def two_cluster_rows(rows: int, n: int, frac_hi: float = 0.35, mu_lo: float = -0.02, mu_hi: float = 0.06,
                     sigma: float = 0.01, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
    """Rows drawn from a two-component mixture: frac_hi of the entries around mu_hi, the rest around mu_lo.

    Stands in for trained filters, whose normalised K the paper reports to settle near 0.35 (Figure 4)."""
    base = normal((rows, n), sigma, seed, stream)
    pick = _fill((rows, n), lambda s, c: uniform01(seed, stream, s, c, lane=3)) < frac_hi
    return (base + np.where(pick, mu_hi, mu_lo)).astype(np.float32)


def small_integer_rows(rows: int, n: int, lo: int = -4, hi: int = 4, seed: int = DEFAULT_SEED,
                       stream: int = 0) -> np.ndarray:
    """Rows of small integers: every sum is exact, so ties in the objective are exact ties."""
    u = _fill((rows, n), lambda s, c: uniform01(seed, stream, s, c, lane=0))
    return np.floor(lo + u.astype(np.float64) * (hi - lo + 1)).clip(lo, hi).astype(np.float32)


def stroke_image(h: int, w: int, target_frac: float = 0.05, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
    """A sketch-like image: background 0, pixels on random polyline strokes set to 1 until ~target_frac is on."""
    img = np.zeros((h, w), dtype=np.float32)
    want = int(target_frac * h * w)
    u = uniform01(seed, stream, 0, 8192, lane=0)
    k = 0
    on = 0
    x, y = u[0] * (w - 1), u[1] * (h - 1)
    k = 2
    while on < want and k + 3 < u.size:
        if u[k] < 0.2:                       # pen up: start a new stroke elsewhere
            x, y = u[k + 1] * (w - 1), u[k + 2] * (h - 1)
            k += 3
            continue
        nx = min(max(x + (u[k + 1] - 0.5) * 0.5 * w, 0), w - 1)
        ny = min(max(y + (u[k + 2] - 0.5) * 0.5 * h, 0), h - 1)
        k += 3
        steps = int(max(abs(nx - x), abs(ny - y))) + 1
        xs = np.rint(np.linspace(x, nx, steps)).astype(np.int64)
        ys = np.rint(np.linspace(y, ny, steps)).astype(np.int64)
        for dy in (0, 1):                    # two-pixel pen width
            yy = np.clip(ys + dy, 0, h - 1)
            img[yy, xs] = 1.0
        on = int(img.sum())
        x, y = nx, ny
    return img


def stroke_batch(n: int, c: int, h: int, w: int, seed: int = DEFAULT_SEED, stream: int = 0) -> np.ndarray:
    """N stroke images replicated over C channels, NCHW fp32."""
    out = np.empty((n, c, h, w), dtype=np.float32)
    for i in range(n):
        out[i, :] = stroke_image(h, w, seed=seed, stream=stream * 4096 + i)[None]
    return out
