"""ctypes binding of libquantpipe.so: argument marshalling only.

Every step of the path runs in the CUDA library; this module turns torch tensors into
pointers and sizes, passes the current CUDA stream, and raises on error codes.  There is no
CPU fallback: if the library has not been built, loading fails with an error.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# QUANTPIPE_LIB selects another build of the library (the one with index checks, libquantpipe_check.so)
LIB_PATH = os.environ.get("QUANTPIPE_LIB") or os.path.join(_PKG, "libquantpipe.so")

QP_OK = 0
QP_ERR_INVALID_ARG, QP_ERR_UNSUPPORTED_BITS, QP_ERR_UNSUPPORTED_DTYPE = -1, -2, -3
QP_ERR_BUFFER_TOO_SMALL, QP_ERR_ALIGNMENT, QP_ERR_CUDA, QP_ERR_TIMEOUT = -4, -5, -6, -7
QP_ERR_TOO_LARGE = -8
QP_STATS_STATIC_MAX_N = 1 << 31
QP_WARN_INFEASIBLE, QP_WARN_DEGENERATE, QP_WARN_NONFINITE = 1, 2, 3
QP_F32, QP_BF16 = 0, 1
QP_DIST_LAPLACE, QP_DIST_GAUSS = 0, 1
QP_B_MAD, QP_B_MEAN_ABS = 0, 1
QP_DEV_BITS_MISMATCH, QP_DEV_DEGENERATE, QP_DEV_NONFINITE, QP_DEV_STREAM_TIMEOUT, QP_DEV_HIST_MISSING = 1, 2, 4, 8, 16
QP_DEV_INDEX_RANGE = 32
QP_DEFAULT_STEPS, QP_DEFAULT_HIST_BINS = 100, 100
QP_SEARCH_AUTO, QP_SEARCH_CANDIDATES, QP_SEARCH_INTERVALS, QP_SEARCH_INTERVALS_PLAIN = 0, 1, 2, 3
QP_SENDER_AUTO, QP_SENDER_CHAIN, QP_SENDER_FUSED = 0, 1, 2
QP_STATS_AUTO, QP_STATS_TWO_KERNELS, QP_STATS_FUSED = 0, 1, 2
QP_CLIP_ACIQ, QP_CLIP_DSACIQ, QP_CLIP_MINMAX, QP_CLIP_INTERSECT, QP_CLIP_MIDRISE = 0, 1, 2, 0x10, 0x20
QP_B_MIDRISE = 0x10
QP_B_GAUSS = 0x20
QP_B_HIST_IN_STATS = 0x40

EXPORTS = (
    "qp_create", "qp_destroy", "qp_get_status", "qp_last_error", "qp_status_string", "qp_packed_bytes",
    "qp_aciq_F", "qp_make_qparams", "qp_stats", "qp_aciq_alpha", "qp_aciq_qparams_device", "qp_dsaciq_search",
    "qp_dsaciq_curve", "qp_policy_use_ds", "qp_quantize_pack", "qp_unpack_dequantize", "qp_select_bits",
    "qp_select_bits_eq2", "qp_launch_count", "qp_sender_host", "qp_receiver_host", "qp_stats_static", "qp_set_search_path", "qp_stats_carries_histogram", "qp_controller_init", "qp_controller_observe",
    "qp_controller_payload_bytes", "qp_sender_device", "qp_set_graph_replay", "qp_graph_replays", "qp_set_sender_path",
    "qp_clip_range", "qp_clip_qparams_device", "qp_stats_channels", "qp_dsaciq_search_channels", "qp_dsaciq_curve_channels", "qp_clip_qparams_channels_device",
    "qp_quantize_pack_channels", "qp_unpack_dequantize_channels", "qp_midrise_range", "qp_sender_channels_device",
    "qp_stats_tokens", "qp_clip_qparams_tokens_device", "qp_quantize_pack_tokens", "qp_unpack_dequantize_tokens",
    "qp_sender_tokens_device",
    "qp_built_with_index_checks", "qp_set_stats_path", "qp_dsaciq_candidates", "qp_dsaciq_candidates_channels", "qp_set_wait_limit_for_testing",
)


class Stats(C.Structure):
    _fields_ = [("n", C.c_uint64), ("nonfinite", C.c_uint64), ("mean", C.c_double), ("mean_abs", C.c_double),
                ("mad", C.c_double), ("var", C.c_double), ("min", C.c_double), ("max", C.c_double),
                ("hist_peak", C.c_uint64), ("hist_bins", C.c_int32), ("reserved", C.c_int32)]


class QParams(C.Structure):
    _fields_ = [("lo", C.c_float), ("hi", C.c_float), ("scale", C.c_float), ("inv_scale", C.c_float),
                ("bits", C.c_int32), ("flags", C.c_int32)]


class DSResult(C.Structure):
    _fields_ = [("b_e", C.c_double), ("b_r", C.c_double), ("b_star", C.c_double), ("alpha_e", C.c_double),
                ("alpha_star", C.c_double), ("mse_e", C.c_double), ("mse_star", C.c_double),
                ("k_star", C.c_int32), ("steps", C.c_int32), ("hist_bins", C.c_int32), ("bits", C.c_int32)]


class Controller(C.Structure):
    _fields_ = [("window", C.c_int32), ("count", C.c_int32), ("bits", C.c_int32), ("mode", C.c_int32),
                ("s_images", C.c_double), ("r_images_per_s", C.c_double), ("n_elems", C.c_uint64),
                ("overhead_bytes", C.c_uint64), ("rel_change", C.c_double), ("sum_bytes", C.c_double),
                ("sum_seconds", C.c_double), ("ref_bandwidth_bps", C.c_double), ("n_allowed", C.c_int32),
                ("allowed", C.c_int32 * 8)]


QP_CTRL_FIT, QP_CTRL_EQ2 = 0, 1


class QuantPipeError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"quantpipe status {status}: {message}")
        self.status = status


_lib = None


def load() -> C.CDLL:
    """Loads libquantpipe.so; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2211_04515_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, u64, i32, dbl = C.c_void_p, C.c_uint64, C.c_int32, C.c_double
    L.qp_create.argtypes = [C.c_int, C.POINTER(vp)]
    L.qp_destroy.argtypes = [vp]
    L.qp_get_status.argtypes = [vp, vp]
    L.qp_last_error.argtypes = [vp]
    L.qp_last_error.restype = C.c_char_p
    L.qp_status_string.argtypes = [i32]
    L.qp_status_string.restype = C.c_char_p
    L.qp_packed_bytes.argtypes = [u64, C.c_int]
    L.qp_packed_bytes.restype = u64
    L.qp_aciq_F.argtypes = [C.c_int, C.c_int]
    L.qp_aciq_F.restype = dbl
    L.qp_make_qparams.argtypes = [dbl, dbl, C.c_int, C.POINTER(QParams)]
    L.qp_stats.argtypes = [vp, vp, C.c_int, u64, C.c_int, vp, vp]
    L.qp_aciq_alpha.argtypes = [C.POINTER(Stats), C.c_int, C.c_int, C.c_int, dbl, C.POINTER(dbl), C.POINTER(QParams)]
    L.qp_aciq_qparams_device.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, vp, vp]
    L.qp_clip_range.argtypes = [C.POINTER(Stats), C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(dbl), C.POINTER(dbl),
                                C.POINTER(QParams)]
    L.qp_clip_qparams_device.argtypes = [vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    L.qp_midrise_range.argtypes = [dbl, dbl, C.c_int, C.POINTER(dbl), C.POINTER(dbl)]
    L.qp_stats_channels.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, vp, vp]
    L.qp_dsaciq_search_channels.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp,
                                            vp]
    L.qp_dsaciq_curve_channels.argtypes = [vp, C.c_uint32, C.POINTER(dbl), C.c_int, vp]
    L.qp_clip_qparams_channels_device.argtypes = [vp, vp, C.c_uint32, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    L.qp_quantize_pack_channels.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, C.c_int, vp, vp, u64, vp]
    L.qp_unpack_dequantize_channels.argtypes = [vp, vp, u64, C.c_uint32, C.c_int, vp, vp, C.c_int, vp]
    L.qp_sender_channels_device.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, C.c_int, C.c_int, C.c_int, vp, u64, vp, vp, vp]
    L.qp_stats_tokens.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, vp, vp]
    L.qp_clip_qparams_tokens_device.argtypes = [vp, vp, u64, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp]
    L.qp_quantize_pack_tokens.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, C.c_int, vp, vp, u64, vp]
    L.qp_unpack_dequantize_tokens.argtypes = [vp, vp, u64, C.c_uint32, C.c_int, vp, vp, C.c_int, vp]
    L.qp_sender_tokens_device.argtypes = [vp, vp, C.c_int, u64, C.c_uint32, C.c_int, C.c_int, C.c_int, vp, u64, vp, vp, vp]
    L.qp_dsaciq_search.argtypes = [vp, vp, C.c_int, u64, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp]
    L.qp_dsaciq_curve.argtypes = [vp, C.POINTER(dbl), C.c_int, vp]
    L.qp_policy_use_ds.argtypes = [C.c_int]
    L.qp_quantize_pack.argtypes = [vp, vp, C.c_int, u64, C.c_int, vp, C.c_int, vp, u64, vp]
    L.qp_unpack_dequantize.argtypes = [vp, vp, u64, C.c_int, vp, C.c_int, vp, C.c_int, vp]
    L.qp_select_bits.argtypes = [dbl, dbl, u64, u64, C.POINTER(i32), C.c_int, C.POINTER(i32)]
    L.qp_select_bits_eq2.argtypes = [dbl, C.c_int, dbl, dbl, dbl, C.POINTER(i32)]
    L.qp_stats_static.argtypes = [vp, C.c_int, u64, vp, vp]
    L.qp_set_search_path.argtypes = [vp, C.c_int]
    L.qp_stats_carries_histogram.argtypes = [vp, C.c_int, u64, C.c_int]
    L.qp_stats_carries_histogram.restype = C.c_int
    L.qp_set_graph_replay.argtypes = [vp, C.c_int]
    L.qp_set_sender_path.argtypes = [vp, C.c_int]
    L.qp_set_stats_path.argtypes = [vp, C.c_int]
    L.qp_built_with_index_checks.argtypes = []
    L.qp_dsaciq_candidates.argtypes = [vp, C.POINTER(QParams), C.c_int, vp]
    L.qp_dsaciq_candidates_channels.argtypes = [vp, C.POINTER(QParams), u64, vp]
    L.qp_set_wait_limit_for_testing.argtypes = [vp, C.c_longlong, C.c_uint32, C.c_int]
    L.qp_graph_replays.argtypes = [vp]
    L.qp_graph_replays.restype = u64
    L.qp_controller_init.argtypes = [C.POINTER(Controller), C.c_int, dbl, dbl, u64, u64, C.POINTER(i32), C.c_int,
                                     C.c_int, dbl, C.c_int]
    L.qp_controller_observe.argtypes = [C.POINTER(Controller), dbl, dbl, C.POINTER(i32), C.POINTER(i32)]
    L.qp_controller_payload_bytes.argtypes = [C.POINTER(Controller), C.c_int]
    L.qp_controller_payload_bytes.restype = u64
    L.qp_launch_count.argtypes = [vp]
    L.qp_launch_count.restype = u64
    L.qp_sender_host.argtypes = [vp, vp, C.c_int, u64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp, u64,
                                 C.POINTER(QParams), vp]
    L.qp_sender_device.argtypes = [vp, vp, C.c_int, u64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, vp, u64, vp, vp, vp]
    L.qp_receiver_host.argtypes = [vp, vp, u64, C.c_int, C.POINTER(QParams), vp, vp, vp, C.c_int, vp]
    for name in EXPORTS:
        fn = getattr(L, name)
        if name not in ("qp_last_error", "qp_status_string", "qp_packed_bytes", "qp_aciq_F", "qp_launch_count",
                        "qp_controller_payload_bytes", "qp_graph_replays"):
            fn.restype = i32
    _lib = L
    return L


# ------------------------------------------------------------- host, pure

def qp_built_with_index_checks() -> bool:
    return bool(load().qp_built_with_index_checks())


def qp_packed_bytes(n: int, bits: int) -> int:
    return int(load().qp_packed_bytes(n, bits))


def qp_aciq_F(bits: int, dist: int = QP_DIST_LAPLACE) -> float:
    return float(load().qp_aciq_F(bits, dist))


def qp_status_string(status: int) -> str:
    return load().qp_status_string(status).decode()


def qp_make_qparams(lo: float, hi: float, bits: int):
    qp = QParams()
    return int(load().qp_make_qparams(lo, hi, bits, C.byref(qp))), qp


def qp_aciq_alpha(stats: Stats, bits: int, dist: int = QP_DIST_LAPLACE, bmode: int = QP_B_MAD,
                  b_override: float = 0.0):
    alpha, qp = C.c_double(), QParams()
    rc = load().qp_aciq_alpha(C.byref(stats), bits, dist, bmode, b_override, C.byref(alpha), C.byref(qp))
    return int(rc), alpha.value, qp


def qp_clip_range(stats: Stats, bits: int, method: int = QP_CLIP_ACIQ, dist: int = QP_DIST_LAPLACE,
                  bmode: int = QP_B_MAD):
    """(status, lo, hi, quantizer) of the closed-form clip range: ACIQ (optionally | QP_CLIP_INTERSECT)
    or QP_CLIP_MINMAX."""
    lo, hi, qp = C.c_double(), C.c_double(), QParams()
    rc = load().qp_clip_range(C.byref(stats), bits, method, dist, bmode, C.byref(lo), C.byref(hi), C.byref(qp))
    return int(rc), lo.value, hi.value, qp


def qp_midrise_range(lo: float, hi: float, bits: int):
    a, b = C.c_double(), C.c_double()
    rc = load().qp_midrise_range(lo, hi, bits, C.byref(a), C.byref(b))
    return int(rc), a.value, b.value


def qp_stats_carries_histogram(x: torch.Tensor, hist_bins: int) -> bool:
    return bool(load().qp_stats_carries_histogram(x.data_ptr(), _dtype_code(x), x.numel(), hist_bins))


def qp_policy_use_ds(bits: int) -> bool:
    return bool(load().qp_policy_use_ds(bits))


def qp_select_bits(bandwidth_bps: float, budget_s: float, n_elems: int, overhead_bytes: int = 0, allowed=None):
    out = C.c_int32()
    if allowed is None:
        rc = load().qp_select_bits(bandwidth_bps, budget_s, n_elems, overhead_bytes, None, 0, C.byref(out))
    else:
        arr = (C.c_int32 * len(allowed))(*allowed)
        rc = load().qp_select_bits(bandwidth_bps, budget_s, n_elems, overhead_bytes, arr, len(allowed), C.byref(out))
    return int(rc), out.value


def qp_select_bits_eq2(v_bytes: float, q_t: int, s_images: float, r_images_per_s: float, bandwidth_bps: float):
    out = C.c_int32()
    rc = load().qp_select_bits_eq2(v_bytes, q_t, s_images, r_images_per_s, bandwidth_bps, C.byref(out))
    return int(rc), out.value


def qp_controller_init(window: int, s_images: float, r_images_per_s: float, n_elems: int, overhead_bytes: int = 0,
                       allowed=None, mode: int = QP_CTRL_FIT, rel_change: float = 0.0, initial_bits: int = 32):
    c = Controller()
    if allowed is None:
        rc = load().qp_controller_init(C.byref(c), window, s_images, r_images_per_s, n_elems, overhead_bytes, None, 0,
                                       mode, rel_change, initial_bits)
    else:
        arr = (C.c_int32 * len(allowed))(*allowed)
        rc = load().qp_controller_init(C.byref(c), window, s_images, r_images_per_s, n_elems, overhead_bytes, arr,
                                       len(allowed), mode, rel_change, initial_bits)
    return int(rc), c


def qp_controller_observe(c: Controller, bytes_sent: float, seconds: float):
    bits, decided = C.c_int32(), C.c_int32()
    rc = load().qp_controller_observe(C.byref(c), bytes_sent, seconds, C.byref(bits), C.byref(decided))
    return int(rc), bits.value, bool(decided.value)


def qp_controller_payload_bytes(c: Controller, bits: int) -> int:
    return int(load().qp_controller_payload_bytes(C.byref(c), bits))


# ------------------------------------------------------------ device calls

def qp_stats_static(x: "torch.Tensor", out: "torch.Tensor", n: int | None = None) -> int:
    """Statistics of x into the device buffer `out` (sizeof(Stats) bytes), for callers that may not
    allocate: no context, no allocation here or in the library (the caller brings `out`).
    Runs on x's device, which must be the current one, on torch's current stream.
    Returns the status code; negative codes are errors (QP_ERR_TOO_LARGE above
    QP_STATS_STATIC_MAX_N elements)."""
    count = x.numel() if n is None else n
    return int(load().qp_stats_static(x.data_ptr(), _dtype_code(x), count, out.data_ptr(), _stream(x.device)))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return QP_F32
    if t.dtype == torch.bfloat16:
        return QP_BF16
    raise QuantPipeError(QP_ERR_UNSUPPORTED_DTYPE, f"unsupported dtype {t.dtype}")


def _stream(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _as_struct(t: torch.Tensor, cls):
    """Copies a device byte buffer holding one struct to the host (synchronises)."""
    raw = t.detach().cpu().contiguous().numpy().tobytes()
    return cls.from_buffer_copy(raw[:C.sizeof(cls)])


class Context:
    """One qp_ctx on one device.  Methods enqueue work on torch's current stream."""

    def __init__(self, device: int | torch.device = 0):
        dev = torch.device("cuda", device) if isinstance(device, int) else torch.device(device)
        if dev.type != "cuda":
            raise QuantPipeError(QP_ERR_INVALID_ARG, "a CUDA device is required")
        self.device = torch.device("cuda", dev.index if dev.index is not None else torch.cuda.current_device())
        self._lib = load()
        handle = C.c_void_p()
        rc = self._lib.qp_create(self.device.index, C.byref(handle))
        if rc != QP_OK:
            raise QuantPipeError(rc, "qp_create failed: " + qp_status_string(rc))
        self._h = handle

    def close(self):
        if getattr(self, "_h", None):
            self._lib.qp_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers
    def _check(self, rc: int) -> int:
        if rc < 0:
            raise QuantPipeError(rc, self._lib.qp_last_error(self._h).decode())
        return int(rc)

    def _bytes(self, nbytes: int) -> torch.Tensor:
        return torch.empty(nbytes, dtype=torch.uint8, device=self.device)

    def _qp_arg(self, qp):
        """(pointer, on_device, keepalive) for a host QParams struct or a device byte tensor."""
        if isinstance(qp, QParams):
            return C.cast(C.pointer(qp), C.c_void_p), 0, qp
        if isinstance(qp, torch.Tensor) and qp.is_cuda:
            return C.c_void_p(qp.data_ptr()), 1, qp
        raise QuantPipeError(QP_ERR_INVALID_ARG, "qp must be a QParams struct or a device tensor")

    # -- a1
    def qp_stats(self, x: torch.Tensor, out: torch.Tensor | None = None, hist_bins: int = 0) -> torch.Tensor:
        """Statistics of x into an 80-byte device buffer (returned); hist_bins > 0 also asks
        for the peak of the search's histogram."""
        assert x.is_cuda and x.is_contiguous()
        out = self._bytes(C.sizeof(Stats)) if out is None else out
        self._check(self._lib.qp_stats(self._h, x.data_ptr(), _dtype_code(x), x.numel(), hist_bins, out.data_ptr(),
                                       _stream(self.device)))
        return out

    # -- a3
    def qp_clip_qparams_device(self, d_stats: torch.Tensor, bits: int, method: int = QP_CLIP_ACIQ,
                               dist: int = QP_DIST_LAPLACE, bmode: int = QP_B_MAD,
                               out: torch.Tensor | None = None) -> torch.Tensor:
        out = self._bytes(C.sizeof(QParams)) if out is None else out
        self._check(self._lib.qp_clip_qparams_device(self._h, d_stats.data_ptr(), bits, method, dist, bmode,
                                                     out.data_ptr(), _stream(self.device)))
        return out

    def qp_aciq_qparams_device(self, d_stats: torch.Tensor, bits: int, dist: int = QP_DIST_LAPLACE,
                               bmode: int = QP_B_MAD, out: torch.Tensor | None = None) -> torch.Tensor:
        out = self._bytes(C.sizeof(QParams)) if out is None else out
        self._check(self._lib.qp_aciq_qparams_device(self._h, d_stats.data_ptr(), bits, dist, bmode, out.data_ptr(),
                                                     _stream(self.device)))
        return out

    # -- a2 + a4
    def qp_dsaciq_search(self, x: torch.Tensor, d_stats: torch.Tensor, bits: int, bmode: int = QP_B_MAD,
                         steps: int = QP_DEFAULT_STEPS, hist_bins: int = QP_DEFAULT_HIST_BINS,
                         out_result: torch.Tensor | None = None, out_qp: torch.Tensor | None = None):
        """Directed search; returns (device DSResult bytes, device QParams bytes)."""
        assert x.is_cuda and x.is_contiguous()
        out_result = self._bytes(C.sizeof(DSResult)) if out_result is None else out_result
        out_qp = self._bytes(C.sizeof(QParams)) if out_qp is None else out_qp
        self._check(self._lib.qp_dsaciq_search(self._h, x.data_ptr(), _dtype_code(x), x.numel(), d_stats.data_ptr(),
                                               bits, bmode, steps, hist_bins, out_result.data_ptr(), out_qp.data_ptr(),
                                               _stream(self.device)))
        return out_result, out_qp

    def qp_set_search_path(self, path: int):
        self._check(self._lib.qp_set_search_path(self._h, path))

    def qp_set_sender_path(self, path: int):
        self._check(self._lib.qp_set_sender_path(self._h, path))

    def qp_set_stats_path(self, path: int):
        self._check(self._lib.qp_set_stats_path(self._h, path))

    def qp_set_wait_limit_for_testing(self, tile_wait_cycles: int = -1, barrier_polls: int = 0,
                                      barrier_extra_arrivals: int = 0):
        self._check(self._lib.qp_set_wait_limit_for_testing(self._h, tile_wait_cycles, barrier_polls,
                                                            barrier_extra_arrivals))

    def qp_dsaciq_candidates(self, steps: int):
        """Host array of the steps + 1 candidate quantizers of the last search (synchronises)."""
        buf = (QParams * (steps + 1))()
        self._check(self._lib.qp_dsaciq_candidates(self._h, buf, steps + 1, _stream(self.device)))
        return buf

    def qp_dsaciq_candidates_channels(self, channels: int, steps: int):
        """Host array [channels * (steps + 1)] of the candidate quantizers of the last channel-wise search."""
        buf = (QParams * (channels * (steps + 1)))()
        self._check(self._lib.qp_dsaciq_candidates_channels(self._h, buf, channels * (steps + 1), _stream(self.device)))
        return buf

    def qp_set_graph_replay(self, on: bool):
        self._check(self._lib.qp_set_graph_replay(self._h, 1 if on else 0))

    def qp_graph_replays(self) -> int:
        return int(self._lib.qp_graph_replays(self._h))

    def qp_dsaciq_curve(self, steps: int):
        buf = (C.c_double * (steps + 1))()
        self._check(self._lib.qp_dsaciq_curve(self._h, buf, steps + 1, _stream(self.device)))
        return list(buf)

    # -- a5
    def qp_quantize_pack(self, x: torch.Tensor, bits: int, qp, out: torch.Tensor | None = None) -> torch.Tensor:
        assert x.is_cuda and x.is_contiguous()
        need = qp_packed_bytes(x.numel(), bits)
        if out is None:
            out = self._bytes(need)
        ptr, on_dev, _keep = self._qp_arg(qp)
        self._check(self._lib.qp_quantize_pack(self._h, x.data_ptr(), _dtype_code(x), x.numel(), bits, ptr, on_dev,
                                               out.data_ptr(), out.numel() * out.element_size(),
                                               _stream(self.device)))
        return out

    # -- a6
    def qp_unpack_dequantize(self, packed: torch.Tensor, n: int, bits: int, qp, out: torch.Tensor | None = None,
                             out_dtype: torch.dtype = torch.float32) -> torch.Tensor:
        assert packed.is_cuda and packed.is_contiguous()
        if out is None:
            out = torch.empty(n, dtype=out_dtype, device=self.device)
        assert out.numel() >= n and out.is_contiguous()
        need = qp_packed_bytes(n, bits)
        if packed.numel() * packed.element_size() < need:
            raise QuantPipeError(QP_ERR_BUFFER_TOO_SMALL, "packed buffer shorter than qp_packed_bytes(n, bits)")
        ptr, on_dev, _keep = self._qp_arg(qp)
        self._check(self._lib.qp_unpack_dequantize(self._h, packed.data_ptr(), n, bits, ptr, on_dev, out.data_ptr(),
                                                   _dtype_code(out), _stream(self.device)))
        return out

    # -- whole sender on device buffers
    def qp_sender_device(self, x: torch.Tensor, bits: int, use_ds: bool, out_packed: torch.Tensor | None = None,
                         out_qp: torch.Tensor | None = None, out_stats: torch.Tensor | None = None,
                         bmode: int = QP_B_MAD, steps: int = QP_DEFAULT_STEPS, hist_bins: int = QP_DEFAULT_HIST_BINS):
        """stats -> clip -> quantize+pack in one call; returns (packed, device QParams bytes).
        use_ds: False/True (ACIQ / directed search) or a QP_CLIP_* method."""
        assert x.is_cuda and x.is_contiguous()
        out_packed = self._bytes(qp_packed_bytes(x.numel(), bits)) if out_packed is None else out_packed
        out_qp = self._bytes(C.sizeof(QParams)) if out_qp is None else out_qp
        self._check(self._lib.qp_sender_device(self._h, x.data_ptr(), _dtype_code(x), x.numel(), bits,
                                               int(use_ds), bmode, steps, hist_bins, out_packed.data_ptr(),
                                               out_packed.numel() * out_packed.element_size(), out_qp.data_ptr(),
                                               out_stats.data_ptr() if out_stats is not None else None,
                                               _stream(self.device)))
        return out_packed, out_qp

    # -- channel-wise variant: x is [rows, channels], the last dimension contiguous
    def qp_stats_channels(self, x: torch.Tensor, channels: int, out: torch.Tensor | None = None) -> torch.Tensor:
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        out = self._bytes(C.sizeof(Stats) * channels) if out is None else out
        self._check(self._lib.qp_stats_channels(self._h, x.data_ptr(), _dtype_code(x), x.numel() // channels, channels,
                                                out.data_ptr(), _stream(self.device)))
        return out

    def qp_dsaciq_search_channels(self, x: torch.Tensor, channels: int, d_stats: torch.Tensor, bits: int,
                                  bmode: int = QP_B_MAD, steps: int = QP_DEFAULT_STEPS,
                                  hist_bins: int = QP_DEFAULT_HIST_BINS, out_result: torch.Tensor | None = None,
                                  out_qp: torch.Tensor | None = None):
        """Directed search per channel; returns (device DSResult[channels] bytes, device QParams[channels] bytes)."""
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        out_result = self._bytes(C.sizeof(DSResult) * channels) if out_result is None else out_result
        out_qp = self._bytes(C.sizeof(QParams) * channels) if out_qp is None else out_qp
        self._check(self._lib.qp_dsaciq_search_channels(self._h, x.data_ptr(), _dtype_code(x), x.numel() // channels,
                                                        channels, d_stats.data_ptr(), bits, bmode, steps, hist_bins,
                                                        out_result.data_ptr(), out_qp.data_ptr(), _stream(self.device)))
        return out_result, out_qp

    def qp_dsaciq_curve_channels(self, channel: int, steps: int):
        buf = (C.c_double * (steps + 1))()
        self._check(self._lib.qp_dsaciq_curve_channels(self._h, channel, buf, steps + 1, _stream(self.device)))
        return list(buf)

    def qp_clip_qparams_channels_device(self, d_stats: torch.Tensor, channels: int, bits: int, method: int = QP_CLIP_ACIQ,
                                        dist: int = QP_DIST_LAPLACE, bmode: int = QP_B_MAD,
                                        out: torch.Tensor | None = None) -> torch.Tensor:
        out = self._bytes(C.sizeof(QParams) * channels) if out is None else out
        self._check(self._lib.qp_clip_qparams_channels_device(self._h, d_stats.data_ptr(), channels, bits, method, dist,
                                                              bmode, out.data_ptr(), _stream(self.device)))
        return out

    def qp_quantize_pack_channels(self, x: torch.Tensor, channels: int, bits: int, d_qp: torch.Tensor,
                                  out: torch.Tensor | None = None) -> torch.Tensor:
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        out = self._bytes(qp_packed_bytes(x.numel(), bits)) if out is None else out
        self._check(self._lib.qp_quantize_pack_channels(self._h, x.data_ptr(), _dtype_code(x), x.numel() // channels,
                                                        channels, bits, d_qp.data_ptr(), out.data_ptr(),
                                                        out.numel() * out.element_size(), _stream(self.device)))
        return out

    def qp_unpack_dequantize_channels(self, packed: torch.Tensor, rows: int, channels: int, bits: int, d_qp: torch.Tensor,
                                      out: torch.Tensor | None = None, out_dtype=torch.float32) -> torch.Tensor:
        out = torch.empty(rows * channels, dtype=out_dtype, device=packed.device) if out is None else out
        self._check(self._lib.qp_unpack_dequantize_channels(self._h, packed.data_ptr(), rows, channels, bits,
                                                            d_qp.data_ptr(), out.data_ptr(), _dtype_code(out),
                                                            _stream(self.device)))
        return out

    def qp_sender_channels_device(self, x: torch.Tensor, channels: int, bits: int, method: int = QP_CLIP_ACIQ,
                                  bmode: int = QP_B_MAD, out_packed: torch.Tensor | None = None,
                                  out_qp: torch.Tensor | None = None, out_stats: torch.Tensor | None = None):
        """Channel-wise statistics -> clip -> quantize+pack in one call; returns (packed, device QParams[channels])."""
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        out_packed = self._bytes(qp_packed_bytes(x.numel(), bits)) if out_packed is None else out_packed
        out_qp = self._bytes(C.sizeof(QParams) * channels) if out_qp is None else out_qp
        self._check(self._lib.qp_sender_channels_device(
            self._h, x.data_ptr(), _dtype_code(x), x.numel() // channels, channels, bits, method, bmode,
            out_packed.data_ptr(), out_packed.numel() * out_packed.element_size(), out_qp.data_ptr(),
            out_stats.data_ptr() if out_stats is not None else None, _stream(self.device)))
        return out_packed, out_qp

    # -- token-wise variant: x is [tokens, channels], a token = a row of `channels` contiguous elements
    def qp_stats_tokens(self, x: torch.Tensor, channels: int, out: torch.Tensor | None = None) -> torch.Tensor:
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        tokens = x.numel() // channels
        out = self._bytes(C.sizeof(Stats) * tokens) if out is None else out
        self._check(self._lib.qp_stats_tokens(self._h, x.data_ptr(), _dtype_code(x), tokens, channels, out.data_ptr(),
                                              _stream(self.device)))
        return out

    def qp_clip_qparams_tokens_device(self, d_stats: torch.Tensor, tokens: int, bits: int, method: int = QP_CLIP_ACIQ,
                                      dist: int = QP_DIST_LAPLACE, bmode: int = QP_B_MAD,
                                      out: torch.Tensor | None = None) -> torch.Tensor:
        out = self._bytes(C.sizeof(QParams) * tokens) if out is None else out
        self._check(self._lib.qp_clip_qparams_tokens_device(self._h, d_stats.data_ptr(), tokens, bits, method, dist, bmode,
                                                            out.data_ptr(), _stream(self.device)))
        return out

    def qp_quantize_pack_tokens(self, x: torch.Tensor, channels: int, bits: int, d_qp: torch.Tensor,
                                out: torch.Tensor | None = None) -> torch.Tensor:
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        out = self._bytes(qp_packed_bytes(x.numel(), bits)) if out is None else out
        self._check(self._lib.qp_quantize_pack_tokens(self._h, x.data_ptr(), _dtype_code(x), x.numel() // channels, channels,
                                                      bits, d_qp.data_ptr(), out.data_ptr(),
                                                      out.numel() * out.element_size(), _stream(self.device)))
        return out

    def qp_unpack_dequantize_tokens(self, packed: torch.Tensor, tokens: int, channels: int, bits: int, d_qp: torch.Tensor,
                                    out: torch.Tensor | None = None, out_dtype=torch.float32) -> torch.Tensor:
        out = torch.empty(tokens * channels, dtype=out_dtype, device=packed.device) if out is None else out
        self._check(self._lib.qp_unpack_dequantize_tokens(self._h, packed.data_ptr(), tokens, channels, bits,
                                                          d_qp.data_ptr(), out.data_ptr(), _dtype_code(out),
                                                          _stream(self.device)))
        return out

    def qp_sender_tokens_device(self, x: torch.Tensor, channels: int, bits: int, method: int = QP_CLIP_ACIQ,
                                bmode: int = QP_B_MAD, out_packed: torch.Tensor | None = None,
                                out_qp: torch.Tensor | None = None, stats_work: torch.Tensor | None = None):
        """Token-wise statistics -> clip -> quantize+pack in one call; returns (packed, device QParams[tokens])."""
        assert x.is_cuda and x.is_contiguous() and x.numel() % channels == 0
        tokens = x.numel() // channels
        out_packed = self._bytes(qp_packed_bytes(x.numel(), bits)) if out_packed is None else out_packed
        out_qp = self._bytes(C.sizeof(QParams) * tokens) if out_qp is None else out_qp
        stats_work = self._bytes(C.sizeof(Stats) * tokens) if stats_work is None else stats_work
        self._check(self._lib.qp_sender_tokens_device(
            self._h, x.data_ptr(), _dtype_code(x), tokens, channels, bits, method, bmode, out_packed.data_ptr(),
            out_packed.numel() * out_packed.element_size(), out_qp.data_ptr(), stats_work.data_ptr(), _stream(self.device)))
        return out_packed, out_qp

    # -- host-buffer sender / receiver
    def qp_sender_host(self, h_x: torch.Tensor, bits: int, use_ds: bool, d_x_work: torch.Tensor,
                       d_packed_work: torch.Tensor, h_packed: torch.Tensor, h_qp_out: QParams,
                       bmode: int = QP_B_MAD, steps: int = QP_DEFAULT_STEPS, hist_bins: int = QP_DEFAULT_HIST_BINS):
        """Host tensor in, packed host bytes + quantizer out (valid after a stream synchronise)."""
        assert not h_x.is_cuda and h_x.is_contiguous() and not h_packed.is_cuda
        self._check(self._lib.qp_sender_host(self._h, h_x.data_ptr(), _dtype_code(h_x), h_x.numel(), bits,
                                             int(use_ds), bmode, steps, hist_bins, d_x_work.data_ptr(),
                                             d_packed_work.data_ptr(), h_packed.data_ptr(),
                                             h_packed.numel() * h_packed.element_size(), C.byref(h_qp_out),
                                             _stream(self.device)))

    def qp_receiver_host(self, h_packed: torch.Tensor, n: int, bits: int, h_qp: QParams, d_packed_work: torch.Tensor,
                         d_y_work: torch.Tensor, h_y: torch.Tensor):
        assert not h_packed.is_cuda and not h_y.is_cuda and h_y.is_contiguous() and h_y.numel() >= n
        self._check(self._lib.qp_receiver_host(self._h, h_packed.data_ptr(), n, bits, C.byref(h_qp),
                                               d_packed_work.data_ptr(), d_y_work.data_ptr(), h_y.data_ptr(),
                                               _dtype_code(h_y), _stream(self.device)))

    def qp_launch_count(self) -> int:
        return int(self._lib.qp_launch_count(self._h))

    # -- status / read-back
    def qp_get_status(self) -> int:
        return self._check(self._lib.qp_get_status(self._h, _stream(self.device)))

    def read_stats(self, d_stats: torch.Tensor) -> Stats:
        return _as_struct(d_stats, Stats)

    def read_qparams(self, d_qp: torch.Tensor) -> QParams:
        return _as_struct(d_qp, QParams)

    def read_ds_result(self, d_res: torch.Tensor) -> DSResult:
        return _as_struct(d_res, DSResult)
