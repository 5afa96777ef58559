"""Seeded synthetic activation tensors shaped like ViT inter-stage activations.

This module only makes inputs.  It holds none of the quantization method's
arithmetic and is the one piece of code that both the CPU oracle's tests and the
CUDA library's tests / benchmark use, so that both sides see identical bytes.

Every value is a pure function of (seed, stream, index): a counter-based
generator built on the SplitMix64 finaliser, so any slice of any tensor can be
regenerated independently and in any chunking.

  u(seed, stream, i)  uniform in (0,1), 53 bits
  Laplace(0,1)        inverse CDF of u
  N(0,1)              Box-Muller on two streams

The ViT-shaped tensors use a per-channel location and scale (channel = last,
contiguous dimension):  x = mu_c + s_c * Laplace(0,1),  mu_c = 0.1 * N(0,1),
s_c = exp(0.5 * N(0,1)).  All arithmetic is fp64 with one final rounding to fp32.
They stand in for the activations of a ViT pipeline stage (the paper's workload,
Sec. 4), which need trained weights and a dataset to produce.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)

# stream identifiers (arbitrary, fixed)
STREAM_VALUE = 1      # the i.i.d. draw of element i
STREAM_VALUE2 = 2     # second uniform for Box-Muller of element i
STREAM_MU_A = 3       # per-channel location, Box-Muller pair
STREAM_MU_B = 4
STREAM_S_A = 5        # per-channel log-scale, Box-Muller pair
STREAM_S_B = 6
STREAM_OUTLIER = 7    # per-channel draw ranking the outlier channels
STREAM_BANDWIDTH = 8  # per-step bandwidth trace
STREAM_CODES = 9      # random integer codes for pack/unpack round trips

_CHUNK = 1 << 20
_WORKERS = max(1, min(16, os.cpu_count() or 1))


def _for_chunks(n: int, fill) -> None:
    """fill(start, count) for every chunk of [0, n); chunks are independent (every value is a pure
    function of its index), so they are filled by a few threads at once (numpy releases the
    interpreter lock inside its loops)."""
    starts = range(0, n, _CHUNK)
    if _WORKERS == 1 or n <= _CHUNK:
        for start in starts:
            fill(start, min(_CHUNK, n - start))
        return
    with ThreadPoolExecutor(_WORKERS) as ex:
        list(ex.map(lambda start: fill(start, min(_CHUNK, n - start)), starts))


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function applied to uint64 array z (wraps mod 2^64)."""
    z = z.copy()
    z ^= z >> np.uint64(30)
    z *= np.uint64(0xBF58476D1CE4E5B9)
    z ^= z >> np.uint64(27)
    z *= np.uint64(0x94D049BB133111EB)
    z ^= z >> np.uint64(31)
    return z


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([np.uint64(seed) * _GOLDEN + np.uint64(0x632BE59BD9B4E019)], dtype=np.uint64))
        k = _mix(k ^ (np.uint64(stream) * np.uint64(0xD6E8FEB86659FD93)))
    return k[0]


def raw_u64(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """64 hashed bits for indices start .. start+count-1."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64)
        return _mix(_key(seed, stream) + (idx + np.uint64(1)) * _GOLDEN)


def uniform01(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """u in (0,1): (top 53 bits + 0.5) / 2^53, fp64."""
    h = raw_u64(seed, stream, start, count) >> np.uint64(11)
    return (h.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def laplace01(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    u = uniform01(seed, stream, start, count)
    d = u - 0.5
    return -np.sign(d) * np.log1p(-2.0 * np.abs(d))


def normal01(seed: int, stream_a: int, stream_b: int, start: int, count: int) -> np.ndarray:
    u1 = uniform01(seed, stream_a, start, count)
    u2 = uniform01(seed, stream_b, start, count)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def channel_params(seed: int, channels: int, outlier_frac: float = 0.0, outlier_gain: float = 20.0):
    """Per-channel (mu_c, s_c) in fp64; optionally the round(frac*C) channels with the
    smallest outlier draw get their scale multiplied by outlier_gain."""
    mu = 0.1 * normal01(seed, STREAM_MU_A, STREAM_MU_B, 0, channels)
    s = np.exp(0.5 * normal01(seed, STREAM_S_A, STREAM_S_B, 0, channels))
    n_out = int(round(outlier_frac * channels))
    if n_out > 0:
        rank = uniform01(seed, STREAM_OUTLIER, 0, channels)
        chosen = np.argsort(rank, kind="stable")[:n_out]
        s[chosen] *= outlier_gain
    return mu, s


def vit_activation(shape, seed: int, outlier_frac: float = 0.0, out: np.ndarray | None = None) -> np.ndarray:
    """fp32 tensor of the given shape, last dimension = channels (contiguous)."""
    shape = tuple(int(d) for d in shape)
    channels = shape[-1]
    n = int(np.prod(shape))
    mu, s = channel_params(seed, channels, outlier_frac)
    flat = out.reshape(-1) if out is not None else np.empty(n, dtype=np.float32)
    assert flat.size == n and flat.dtype == np.float32

    def fill(start, cnt):
        c = (np.arange(start, start + cnt, dtype=np.int64) % channels)
        flat[start:start + cnt] = (mu[c] + s[c] * laplace01(seed, STREAM_VALUE, start, cnt)).astype(np.float32)

    _for_chunks(n, fill)
    return flat.reshape(shape)


def flat_iid(n: int, seed: int, dist: str = "laplace", out: np.ndarray | None = None) -> np.ndarray:
    """Flat fp32 tensor of n i.i.d. Laplace(0,1) or N(0,1) values."""
    flat = out if out is not None else np.empty(n, dtype=np.float32)
    assert flat.size == n and flat.dtype == np.float32
    if dist not in ("laplace", "normal"):
        raise ValueError(f"unknown dist {dist!r}")

    def fill(start, cnt):
        if dist == "laplace":
            v = laplace01(seed, STREAM_VALUE, start, cnt)
        else:
            v = normal01(seed, STREAM_VALUE, STREAM_VALUE2, start, cnt)
        flat[start:start + cnt] = v.astype(np.float32)

    _for_chunks(n, fill)
    return flat


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest, ties to even); returns the uint16 bit patterns.
    NaN stays NaN (quiet bit forced)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    nan = (b & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = (b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    r = np.where(nan, (b >> np.uint32(16)) | np.uint32(0x0040), r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to fp32."""
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bandwidth_trace(seed: int, steps: int, lo_bps: float = 5e6, hi_bps: float = 200e6) -> np.ndarray:
    """Per-step link bandwidth in bit/s, uniform in [lo_bps, hi_bps]."""
    return lo_bps + (hi_bps - lo_bps) * uniform01(seed, STREAM_BANDWIDTH, 0, steps)


def random_codes(n: int, bits: int, seed: int) -> np.ndarray:
    """n uniformly random integer codes in [0, 2^bits)."""
    h = raw_u64(seed, STREAM_CODES, 0, n)
    return (h >> np.uint64(64 - bits)).astype(np.uint32)


# The five benchmark configurations: shape, seed, outlier fraction, bit-widths.
CONFIGS = {
    "c1": dict(shape=(1, 197, 768), seed=0, outlier_frac=0.0, bits=(2, 8)),
    "c2": dict(shape=(64, 197, 768), seed=1, outlier_frac=0.0, bits=(2, 3, 4, 6, 8)),
    "c3": dict(shape=(64, 197, 1024), seed=2, outlier_frac=0.01, bits=(2, 4, 8)),
    "c4": dict(shape=(128, 197, 1280), seed=3, outlier_frac=0.0, bits=(1, 2, 3, 4, 6, 8, 16)),
}
C4_TRACE_STEPS = 100
C4_BUDGET_S = 2.0
C4_ALLOWED_BITS = (1, 2, 3, 4, 6, 8, 16)
C5_SEED = 4
C5_BITS = (1, 2, 3, 4, 6, 8, 16)
C5_LOG2_ELEMS = tuple(range(18, 29))


def config_tensor(name: str, out: np.ndarray | None = None) -> np.ndarray:
    c = CONFIGS[name]
    return vit_activation(c["shape"], c["seed"], c["outlier_frac"], out=out)
