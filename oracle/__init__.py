"""ctypes front end of the CPU oracle (oracle/quantpipe_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg.  It never imports the CUDA package, and the CUDA package never imports it.

The shared object is compiled with gcc on first use (and again when the C source is newer
than the object), so no prebuilt binary is needed.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "quantpipe_oracle.c")
_SO = os.path.join(_HERE, "libqp_oracle.so")
_CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-msse4.1", "-Wall", "-Wextra", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.run(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _SO)
    return _SO


class Stats(C.Structure):
    _fields_ = [("n", C.c_uint64), ("nonfinite", C.c_uint64), ("mean", C.c_double), ("mean_abs", C.c_double),
                ("mad", C.c_double), ("var", C.c_double), ("min", C.c_double), ("max", C.c_double)]


class QParams(C.Structure):
    _fields_ = [("lo", C.c_float), ("hi", C.c_float), ("scale", C.c_float), ("inv_scale", C.c_float),
                ("bits", C.c_int32), ("flags", C.c_int32)]

    def as_tuple(self):
        return (np.float32(self.lo).tobytes(), np.float32(self.hi).tobytes(), np.float32(self.scale).tobytes(),
                np.float32(self.inv_scale).tobytes(), self.bits, self.flags)


class DSResult(C.Structure):
    _fields_ = [("b_e", C.c_double), ("b_r", C.c_double), ("b_star", C.c_double), ("alpha_e", C.c_double),
                ("alpha_star", C.c_double), ("mse_e", C.c_double), ("mse_star", C.c_double),
                ("k_star", C.c_int32), ("steps", C.c_int32), ("hist_bins", C.c_int32), ("bits", C.c_int32)]


class Controller(C.Structure):
    _fields_ = [("window", C.c_int32), ("count", C.c_int32), ("bits", C.c_int32), ("mode", C.c_int32),
                ("s_images", C.c_double), ("r_images_per_s", C.c_double), ("n_elems", C.c_uint64),
                ("overhead_bytes", C.c_uint64), ("rel_change", C.c_double), ("sum_bytes", C.c_double),
                ("sum_seconds", C.c_double), ("ref_bw", C.c_double), ("n_allowed", C.c_int32),
                ("allowed", C.c_int32 * 8)]


OK, ERR_ARG, ERR_BITS, WARN_INFEASIBLE, WARN_DEGENERATE = 0, -1, -2, 1, 2

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp, u32p, u8p, u64p, dp = (C.POINTER(C.c_float), C.POINTER(C.c_uint32), C.POINTER(C.c_uint8),
                                   C.POINTER(C.c_uint64), C.POINTER(C.c_double))
        L.orc_stats.argtypes = [fp, C.c_uint64, C.POINTER(Stats)]
        L.orc_stats.restype = None
        L.orc_aciq_F_laplace.argtypes = [C.c_int]
        L.orc_aciq_F_laplace.restype = C.c_double
        L.orc_aciq_F_gauss.argtypes = [C.c_int]
        L.orc_aciq_F_gauss.restype = C.c_double
        L.orc_make_qparams.argtypes = [C.c_double, C.c_double, C.c_int, C.POINTER(QParams)]
        L.orc_make_qparams.restype = C.c_int
        L.orc_quantize.argtypes = [fp, C.c_uint64, C.POINTER(QParams), u32p]
        L.orc_quantize.restype = None
        L.orc_dequantize.argtypes = [u32p, C.c_uint64, C.POINTER(QParams), fp]
        L.orc_dequantize.restype = None
        L.orc_quant_mse.argtypes = [fp, C.c_uint64, C.POINTER(QParams)]
        L.orc_quant_mse.restype = C.c_double
        L.orc_packed_bytes.argtypes = [C.c_uint64, C.c_int]
        L.orc_packed_bytes.restype = C.c_uint64
        L.orc_pack.argtypes = [u32p, C.c_uint64, C.c_int, u8p]
        L.orc_pack.restype = None
        L.orc_unpack.argtypes = [u8p, C.c_uint64, C.c_int, u32p]
        L.orc_unpack.restype = None
        L.orc_aciq_alpha.argtypes = [C.POINTER(Stats), C.c_int, C.c_int, C.c_int, C.c_double, dp, C.POINTER(QParams)]
        L.orc_aciq_alpha.restype = C.c_int
        L.orc_clip_range.argtypes = [C.POINTER(Stats), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, dp, dp,
                                     C.POINTER(QParams)]
        L.orc_clip_range.restype = C.c_int
        L.orc_stats_channels.argtypes = [fp, C.c_uint64, C.c_uint64, C.POINTER(Stats)]
        L.orc_stats_channels.restype = C.c_int
        L.orc_clip_channels.argtypes = [C.POINTER(Stats), C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                        C.POINTER(QParams)]
        L.orc_clip_channels.restype = C.c_int
        L.orc_ds_search_channels.argtypes = [fp, C.c_uint64, C.c_uint64, C.POINTER(Stats), C.c_int, C.c_int, C.c_int,
                                             C.c_int, C.POINTER(DSResult), C.POINTER(QParams), C.POINTER(C.c_double)]
        L.orc_ds_search_channels.restype = C.c_int
        L.orc_quantize_channels.argtypes = [fp, C.c_uint64, C.c_uint64, C.POINTER(QParams), u32p]
        L.orc_quantize_channels.restype = None
        L.orc_dequantize_channels.argtypes = [u32p, C.c_uint64, C.c_uint64, C.POINTER(QParams), fp]
        L.orc_dequantize_channels.restype = None
        L.orc_stats_tokens.argtypes = [fp, C.c_uint64, C.c_uint64, C.POINTER(Stats)]
        L.orc_stats_tokens.restype = C.c_int
        L.orc_quantize_tokens.argtypes = [fp, C.c_uint64, C.c_uint64, C.POINTER(QParams), u32p]
        L.orc_quantize_tokens.restype = None
        L.orc_dequantize_tokens.argtypes = [u32p, C.c_uint64, C.c_uint64, C.POINTER(QParams), fp]
        L.orc_dequantize_tokens.restype = None
        L.orc_midrise_range.argtypes = [C.c_double, C.c_double, C.c_int, dp, dp]
        L.orc_midrise_range.restype = None
        L.orc_hist_peak.argtypes = [fp, C.c_uint64, C.c_double, C.c_double, C.c_int, u64p]
        L.orc_hist_peak.restype = C.c_double
        L.orc_ds_search.argtypes = [fp, C.c_uint64, C.POINTER(Stats), C.c_int, C.c_int, C.c_int, C.c_int,
                                    C.POINTER(DSResult), C.POINTER(QParams), dp]
        L.orc_ds_search.restype = C.c_int
        L.orc_select_bits.argtypes = [C.c_double, C.c_double, C.c_uint64, C.c_uint64, C.POINTER(C.c_int32), C.c_int,
                                      C.POINTER(C.c_int32)]
        L.orc_select_bits.restype = C.c_int
        L.orc_select_bits_eq2.argtypes = [C.c_double, C.c_int, C.c_double, C.c_double, C.c_double, C.POINTER(C.c_int32)]
        L.orc_select_bits_eq2.restype = C.c_int
        L.orc_controller_init.argtypes = [C.POINTER(Controller), C.c_int, C.c_double, C.c_double, C.c_uint64,
                                          C.c_uint64, C.POINTER(C.c_int32), C.c_int, C.c_int, C.c_double, C.c_int]
        L.orc_controller_init.restype = None
        L.orc_controller_observe.argtypes = [C.POINTER(Controller), C.c_double, C.c_double, C.POINTER(C.c_int32)]
        L.orc_controller_observe.restype = C.c_int
        _lib = L
    return _lib


def _f32(x) -> np.ndarray:
    a = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    return a


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def widen_bf16(bits_u16) -> np.ndarray:
    """bfloat16 bit patterns -> the same values in fp32 (exact: the pattern shifted left 16)."""
    return (np.ascontiguousarray(bits_u16, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def stats(x) -> Stats:
    a = _f32(x)
    s = Stats()
    lib().orc_stats(_ptr(a, C.c_float), a.size, C.byref(s))
    return s


def aciq_F(bits: int, dist: int = 0) -> float:
    return lib().orc_aciq_F_gauss(bits) if dist == 1 else lib().orc_aciq_F_laplace(bits)


def make_qparams(lo: float, hi: float, bits: int):
    qp = QParams()
    rc = lib().orc_make_qparams(lo, hi, bits, C.byref(qp))
    return rc, qp


def aciq_alpha(st: Stats, bits: int, dist: int = 0, bmode: int = 0, b_override: float = 0.0):
    alpha = C.c_double()
    qp = QParams()
    rc = lib().orc_aciq_alpha(C.byref(st), bits, dist, bmode, b_override, C.byref(alpha), C.byref(qp))
    return rc, alpha.value, qp


CLIP_ACIQ, CLIP_MINMAX = 0, 2


B_MIDRISE = 0x10          # ds_search: bmode | B_MIDRISE scores every candidate on the mid-rise grid


def clip_range(st: Stats, bits: int, method: int = CLIP_ACIQ, intersect: bool = False, dist: int = 0, bmode: int = 0,
               midrise: bool = False):
    """(rc, lo, hi, quantizer) of the clip range by method: ACIQ, or naive PTQ's [min, max]."""
    lo, hi = C.c_double(), C.c_double()
    qp = QParams()
    rc = lib().orc_clip_range(C.byref(st), bits, method, (1 if intersect else 0) | (2 if midrise else 0), dist, bmode,
                              C.byref(lo), C.byref(hi), C.byref(qp))
    return rc, lo.value, hi.value, qp


def midrise_range(lo: float, hi: float, bits: int):
    a, b = C.c_double(), C.c_double()
    lib().orc_midrise_range(lo, hi, bits, C.byref(a), C.byref(b))
    return a.value, b.value


def quantize(x, qp: QParams) -> np.ndarray:
    a = _f32(x)
    codes = np.empty(a.size, dtype=np.uint32)
    lib().orc_quantize(_ptr(a, C.c_float), a.size, C.byref(qp), _ptr(codes, C.c_uint32))
    return codes


def dequantize(codes, qp: QParams) -> np.ndarray:
    c = np.ascontiguousarray(codes, dtype=np.uint32).reshape(-1)
    y = np.empty(c.size, dtype=np.float32)
    lib().orc_dequantize(_ptr(c, C.c_uint32), c.size, C.byref(qp), _ptr(y, C.c_float))
    return y


def quant_mse(x, qp: QParams) -> float:
    a = _f32(x)
    return lib().orc_quant_mse(_ptr(a, C.c_float), a.size, C.byref(qp))


def packed_bytes(n: int, bits: int) -> int:
    return int(lib().orc_packed_bytes(n, bits))


def pack(codes, bits: int) -> np.ndarray:
    c = np.ascontiguousarray(codes, dtype=np.uint32).reshape(-1)
    out = np.empty(packed_bytes(c.size, bits), dtype=np.uint8)
    lib().orc_pack(_ptr(c, C.c_uint32), c.size, bits, _ptr(out, C.c_uint8))
    return out


def unpack(packed, n: int, bits: int) -> np.ndarray:
    p = np.ascontiguousarray(packed, dtype=np.uint8).reshape(-1)
    assert p.size >= (n * bits + 7) // 8
    codes = np.empty(n, dtype=np.uint32)
    lib().orc_unpack(_ptr(p, C.c_uint8), n, bits, _ptr(codes, C.c_uint32))
    return codes


def stats_channels(x, channels: int):
    """Per-channel statistics of a [rows, channels] tensor: a ctypes array of `channels` Stats."""
    a = _f32(x)
    rows = a.size // channels
    assert rows * channels == a.size
    out = (Stats * channels)()
    rc = lib().orc_stats_channels(_ptr(a, C.c_float), rows, channels, out)
    assert rc == 0
    return out


def clip_channels(st, bits: int, method: int = CLIP_ACIQ, intersect: bool = False, dist: int = 0, bmode: int = 0,
                  midrise: bool = False):
    """(rc, ctypes array of per-channel QParams) from per-channel statistics."""
    channels = len(st)
    qp = (QParams * channels)()
    rc = lib().orc_clip_channels(st, channels, bits, method, (1 if intersect else 0) | (2 if midrise else 0), dist, bmode, qp)
    return rc, qp


def quantize_channels(x, channels: int, qp) -> np.ndarray:
    a = _f32(x)
    codes = np.empty(a.size, dtype=np.uint32)
    lib().orc_quantize_channels(_ptr(a, C.c_float), a.size // channels, channels, qp, _ptr(codes, C.c_uint32))
    return codes


def dequantize_channels(codes, channels: int, qp) -> np.ndarray:
    c = np.ascontiguousarray(codes, dtype=np.uint32)
    y = np.empty(c.size, dtype=np.float32)
    lib().orc_dequantize_channels(_ptr(c, C.c_uint32), c.size // channels, channels, qp, _ptr(y, C.c_float))
    return y


def stats_tokens(x, channels: int):
    """Per-token statistics of a [tokens, channels] tensor: a ctypes array of `tokens` Stats."""
    a = _f32(x)
    tokens = a.size // channels
    assert tokens * channels == a.size
    out = (Stats * max(tokens, 1))()
    rc = lib().orc_stats_tokens(_ptr(a, C.c_float), tokens, channels, out)
    assert rc == 0
    return out


def clip_tokens(st, bits: int, method: int = CLIP_ACIQ, intersect: bool = False, dist: int = 0, bmode: int = 0,
                midrise: bool = False):
    """(rc, ctypes array of per-token QParams) from per-token statistics (the same map as clip_channels)."""
    return clip_channels(st, bits, method, intersect, dist, bmode, midrise)


def quantize_tokens(x, channels: int, qp) -> np.ndarray:
    a = _f32(x)
    codes = np.empty(a.size, dtype=np.uint32)
    lib().orc_quantize_tokens(_ptr(a, C.c_float), a.size // channels, channels, qp, _ptr(codes, C.c_uint32))
    return codes


def dequantize_tokens(codes, channels: int, qp) -> np.ndarray:
    c = np.ascontiguousarray(codes, dtype=np.uint32)
    y = np.empty(c.size, dtype=np.float32)
    lib().orc_dequantize_tokens(_ptr(c, C.c_uint32), c.size // channels, channels, qp, _ptr(y, C.c_float))
    return y


def quantize_pack(x, qp: QParams) -> np.ndarray:
    return pack(quantize(x, qp), qp.bits)


def unpack_dequantize(packed, n: int, qp: QParams) -> np.ndarray:
    return dequantize(unpack(packed, n, qp.bits), qp)


def hist_peak(x, mn: float, mx: float, nb: int):
    a = _f32(x)
    counts = np.zeros(nb, dtype=np.uint64)
    peak = lib().orc_hist_peak(_ptr(a, C.c_float), a.size, mn, mx, nb, _ptr(counts, C.c_uint64))
    return peak, counts


def ds_search(x, st: Stats, bits: int, bmode: int = 0, steps: int = 100, hist_bins: int = 100):
    a = _f32(x)
    res = DSResult()
    qp = QParams()
    curve = np.empty(steps + 1, dtype=np.float64)
    rc = lib().orc_ds_search(_ptr(a, C.c_float), a.size, C.byref(st), bits, bmode, steps, hist_bins,
                             C.byref(res), C.byref(qp), _ptr(curve, C.c_double))
    return rc, res, qp, curve


def ds_search_channels(x, channels: int, st, bits: int, bmode: int = 0, steps: int = 100, hist_bins: int = 100):
    """Directed search per channel of a [rows, channels] tensor: (rc, DSResult[channels], QParams[channels], curves)."""
    a = _f32(x)
    rows = a.size // channels
    assert rows * channels == a.size
    res = (DSResult * channels)()
    qp = (QParams * channels)()
    curves = np.empty((channels, steps + 1), dtype=np.float64)
    rc = lib().orc_ds_search_channels(_ptr(a, C.c_float), rows, channels, st, bits, bmode, steps, hist_bins, res, qp,
                                      _ptr(curves, C.c_double))
    return rc, res, qp, curves


def select_bits(bandwidth_bps: float, budget_s: float, n_elems: int, overhead_bytes: int = 0,
                allowed=(32, 16, 8, 6, 4, 2)):
    arr = (C.c_int32 * len(allowed))(*allowed)
    out = C.c_int32()
    rc = lib().orc_select_bits(bandwidth_bps, budget_s, n_elems, overhead_bytes, arr, len(allowed), C.byref(out))
    return rc, out.value


def select_bits_eq2(v_bytes: float, q_t: int, s_images: float, r_images_per_s: float, bandwidth_bps: float):
    out = C.c_int32()
    rc = lib().orc_select_bits_eq2(v_bytes, q_t, s_images, r_images_per_s, bandwidth_bps, C.byref(out))
    return rc, out.value


def controller_init(window, s_images, r_images_per_s, n_elems, overhead_bytes=0, allowed=(32, 16, 8, 6, 4, 2), mode=0,
                    rel_change=0.0, initial_bits=32) -> Controller:
    c = Controller()
    arr = (C.c_int32 * len(allowed))(*allowed)
    lib().orc_controller_init(C.byref(c), window, s_images, r_images_per_s, n_elems, overhead_bytes, arr, len(allowed),
                              mode, rel_change, initial_bits)
    return c


def controller_observe(c: Controller, bytes_sent: float, seconds: float):
    out = C.c_int32()
    decided = lib().orc_controller_observe(C.byref(c), bytes_sent, seconds, C.byref(out))
    return out.value, bool(decided)
