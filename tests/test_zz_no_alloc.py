"""qp_stats_static: the statistics entry point for callers that may not allocate.

A host program whose memory pool is frozen (or already fully handed out) cannot let a
library call cudaMalloc behind its back.  qp_stats_static therefore keeps its scratch in a
fixed array inside the library and takes only the caller's input and output buffers.  This
test calls it through the C ABI twice in a row (the array is shared and keeps the previous
call's contents, so the second call proves the clean-up) and compares both results with
the ordinary, context-based qp_stats within the statistics tolerance of the parity tests
(1e-5 relative).  It is collected last so that a run stopping at the first failure has
already run every other test; it needs nothing from them and passes alone in a fresh
process as well.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2211_04515_b200 as qp
import synth_inputs as si

pytestmark = pytest.mark.gpu

STATS_BYTES = ctypes.sizeof(qp.Stats)


def _close(a, b):
    assert a.n == b.n and a.nonfinite == b.nonfinite
    assert a.min == b.min and a.max == b.max
    assert abs(a.mean - b.mean) <= 1e-5 * max(abs(b.mean), b.mad)
    for f in ("mean_abs", "mad", "var"):
        assert abs(getattr(a, f) - getattr(b, f)) <= 1e-5 * abs(getattr(b, f)), f


def test_static_stats_matches_context_stats_twice():
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    ctx = qp.Context(0)
    x1 = torch.from_numpy(si.vit_activation((16, 197, 768), 41).reshape(-1)).cuda()
    x2_h = si.vit_activation((3, 197, 1024), 42, outlier_frac=0.01).reshape(-1)
    x2_h[[7, 1000]] = [np.nan, np.inf]                      # the non-finite path: reported through `nonfinite` only
    x2 = torch.from_numpy(x2_h).cuda()[1:]                  # and a 4-byte-aligned, ragged view
    out = torch.empty(STATS_BYTES, dtype=torch.uint8, device="cuda")  # the caller's buffer; nothing else is needed
    for x in (x1, x2):                                       # two calls in a row on the shared scratch
        want = ctx.read_stats(ctx.qp_stats(x))
        out.fill_(0xEE)
        assert qp.qp_stats_static(x, out) == qp.QP_OK
        got = ctx.read_stats(out)
        _close(got, want)
    assert got.nonfinite == 2                                # (this entry point has no status word to read)
    # bf16 input and the empty tensor
    xb = x1[:100003].to(torch.bfloat16)
    want = ctx.read_stats(ctx.qp_stats(xb))
    assert qp.qp_stats_static(xb, out) == qp.QP_OK
    _close(ctx.read_stats(out), want)
    assert qp.qp_stats_static(x1[:0], out) == qp.QP_OK
    assert ctx.read_stats(out).n == 0
    ctx.qp_get_status()
    ctx.close()


def test_static_stats_rejects_bad_arguments():
    x = torch.zeros(1024, device="cuda")
    out = torch.empty(STATS_BYTES, dtype=torch.uint8, device="cuda")
    # beyond the stated maximum: refused before anything is enqueued or read
    assert qp.qp_stats_static(x, out, n=qp.QP_STATS_STATIC_MAX_N + 1) == qp.QP_ERR_TOO_LARGE
    assert "maximum" in qp.qp_status_string(qp.QP_ERR_TOO_LARGE)
    assert qp.qp_stats_static(x, out[1:]) == qp.QP_ERR_ALIGNMENT
    with pytest.raises(qp.QuantPipeError):
        qp.qp_stats_static(x.double(), out)
    torch.cuda.synchronize()
