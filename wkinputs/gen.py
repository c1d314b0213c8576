"""Counter-based seeded generators (numpy side).

Every element is a pure function of (seed, stream, element index), so any slice of any
tensor can be produced on its own, on the host or on the device, with bit-identical
results.  The device side (``gen.cu`` in this folder) implements the same integer hash
and the same fp32 operations; no transcendental function is used anywhere, so the two
cannot drift.

Recipe
------
* ``hash64(seed, stream, idx)``: two rounds of the splitmix64 finaliser.
* ``normal_f32``: the sum of eight 16-bit uniform integers taken from two hashes, centred
  and scaled to unit variance (Irwin-Hall, n = 8: support +-4.9 sigma, excess kurtosis
  -0.15).  Integer sum -> fp32 (exact) -> one fp32 multiply.
* bf16: round-to-nearest-even on the fp32 bit pattern.
* Key-redundancy stream (the benchmark's "per-position base vector + per-frame noise,
  30 % of positions redrawn per frame"): for layer l, global latent frame g, position p,
  ``src(g, p)`` is the latest frame <= g at which position p was redrawn (frame 0 always
  is); ``K[g, p, :] = bf16( base[src, p, :] + sigma * eps[g, p, :] )`` with base and eps
  unit normals, the multiply and the add rounded separately in fp32.  The stream is
  continuous across chunks: chunk c holds frames 3c .. 3c+2.
"""
from __future__ import annotations

import numpy as np

# stream = kind * 2**20 + sub-stream (layer, or layer * 64 + step)
STREAM_K_BASE = 1 << 20
STREAM_K_NOISE = 2 << 20
STREAM_K_REDRAW = 3 << 20
STREAM_V = 4 << 20
STREAM_Q = 5 << 20
STREAM_MISC = 6 << 20

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
REDRAW_THRESHOLD = 5033165  # floor(0.3 * 2**24): a position is redrawn when the top 24 hash bits fall below this
_NORMAL_CENTRE = np.float32(262140.0)  # 8 * 65535 / 2
_NORMAL_SCALE = np.float32(1.0 / 53509.98)  # 1 / sqrt(8 * (65536**2 - 1) / 12)


def _mix64(x: np.ndarray) -> np.ndarray:
    x = x ^ (x >> np.uint64(30))
    x = x * _M1
    x = x ^ (x >> np.uint64(27))
    x = x * _M2
    x = x ^ (x >> np.uint64(31))
    return x


def hash64(seed: int, stream: int, idx) -> np.ndarray:
    """64-bit hash of (seed, stream, idx); ``idx`` is an array of non-negative integers."""
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        key = _mix64(np.uint64(seed) * _GOLD + np.uint64(stream))
        return _mix64((key + idx * _GOLD).astype(np.uint64))


def normal_f32(seed: int, stream: int, idx) -> np.ndarray:
    """Unit-variance, zero-mean fp32 variates, one per entry of ``idx``."""
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h0 = hash64(seed, stream, idx * np.uint64(2))
        h1 = hash64(seed, stream, idx * np.uint64(2) + np.uint64(1))
    m = np.uint64(0xFFFF)
    s = np.zeros(idx.shape, dtype=np.uint64)
    for h in (h0, h1):
        for sh in (0, 16, 32, 48):
            s += (h >> np.uint64(sh)) & m
    x = s.astype(np.float32)  # <= 524280, exact
    return ((x - _NORMAL_CENTRE) * _NORMAL_SCALE).astype(np.float32)


def f32_to_bf16_bits(x) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def normal_bf16(seed: int, stream: int, idx0: int, n: int) -> np.ndarray:
    """n consecutive unit normals starting at element idx0, as bf16 bit patterns."""
    idx = np.arange(idx0, idx0 + n, dtype=np.uint64)
    return f32_to_bf16_bits(normal_f32(seed, stream, idx))


def redraw_mask(seed: int, layer: int, g, T: int) -> np.ndarray:
    """Boolean [len(g), T]: was position p redrawn at global frame g?  Frame 0 always is."""
    g = np.asarray(g, dtype=np.uint64).reshape(-1, 1)
    p = np.arange(T, dtype=np.uint64).reshape(1, -1)
    h = hash64(seed, STREAM_K_REDRAW + layer, g * np.uint64(T) + p)
    return ((h >> np.uint64(40)) < np.uint64(REDRAW_THRESHOLD)) | (g == 0)


def _source_frames(seed: int, layer: int, g0: int, n_frames: int, T: int) -> np.ndarray:
    """src[f, p]: latest frame <= g0+f at which position p was redrawn."""
    src = np.empty((n_frames, T), dtype=np.int64)
    for f in range(n_frames):
        g = np.full(T, g0 + f, dtype=np.int64)
        pending = np.ones(T, dtype=bool)
        while pending.any():
            p = np.nonzero(pending)[0]
            h = hash64(seed, STREAM_K_REDRAW + layer,
                       g[p].astype(np.uint64) * np.uint64(T) + p.astype(np.uint64))
            hit = ((h >> np.uint64(40)) < np.uint64(REDRAW_THRESHOLD)) | (g[p] == 0)
            pending[p[hit]] = False
            g[p[~hit]] -= 1
        src[f] = g
    return src


def key_frames_bf16(seed: int, layer: int, g0: int, n_frames: int, T: int, D: int,
                    sigma: float, cols=None) -> np.ndarray:
    """Keys of frames g0 .. g0+n_frames-1 of one layer: uint16 [n_frames*T, D] (bf16 bits).
    ``cols`` (an index array) restricts the result to those columns of the D-wide rows."""
    src = _source_frames(seed, layer, g0, n_frames, T)  # [n_frames, T]
    cidx = np.arange(D, dtype=np.uint64) if cols is None else np.asarray(cols, dtype=np.uint64)
    c = cidx.reshape(1, 1, -1)
    p = np.arange(T, dtype=np.uint64).reshape(1, T, 1)
    g = (g0 + np.arange(n_frames, dtype=np.uint64)).reshape(n_frames, 1, 1)
    with np.errstate(over="ignore"):
        base_idx = (src.astype(np.uint64).reshape(n_frames, T, 1) * np.uint64(T) + p) * np.uint64(D) + c
        eps_idx = (g * np.uint64(T) + p) * np.uint64(D) + c
    base = normal_f32(seed, STREAM_K_BASE + layer, base_idx)
    eps = normal_f32(seed, STREAM_K_NOISE + layer, eps_idx)
    scaled = (np.float32(sigma) * eps).astype(np.float32)  # fp32 multiply, rounded
    k = (base + scaled).astype(np.float32)  # fp32 add, rounded
    return f32_to_bf16_bits(k).reshape(n_frames * T, len(cidx))


def key_chunk_bf16(seed: int, layer: int, chunk: int, T: int, D: int, sigma: float,
                   F: int = 3, cols=None) -> np.ndarray:
    """Keys of chunk ``chunk`` (frames F*chunk .. F*chunk+F-1): uint16 [F*T, D] (or [F*T, len(cols)])."""
    return key_frames_bf16(seed, layer, F * chunk, F, T, D, sigma, cols=cols)


def _normal_rows_bf16(seed: int, stream: int, idx0: int, rows: int, D: int, cols=None) -> np.ndarray:
    """Row-major [rows, D] block of unit normals starting at element idx0, optionally only some columns."""
    if cols is None:
        return normal_bf16(seed, stream, idx0, rows * D).reshape(rows, D)
    cidx = np.asarray(cols, dtype=np.uint64).reshape(1, -1)
    r = np.arange(rows, dtype=np.uint64).reshape(-1, 1)
    with np.errstate(over="ignore"):
        idx = np.uint64(idx0) + r * np.uint64(D) + cidx
    return f32_to_bf16_bits(normal_f32(seed, stream, idx))


def value_chunk_bf16(seed: int, layer: int, chunk: int, T: int, D: int, F: int = 3, cols=None) -> np.ndarray:
    """Values of one chunk, i.i.d. unit normals: uint16 [F*T, D] (or [F*T, len(cols)])."""
    return _normal_rows_bf16(seed, STREAM_V + layer, chunk * F * T * D, F * T, D, cols)


def query_bf16(seed: int, layer: int, step: int, chunk: int, Lq: int, D: int, cols=None) -> np.ndarray:
    """Queries of one (layer, denoising step, chunk), i.i.d. unit normals: uint16 [Lq, D] (or [Lq, len(cols)])."""
    return _normal_rows_bf16(seed, STREAM_Q + layer * 64 + step, chunk * Lq * D, Lq, D, cols)
