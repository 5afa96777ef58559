"""CPU-side checks of the C-ABI library: it loads, exports everything the header declares,
and its host-only functions agree with the oracle.  No kernel is launched here."""
import os
import re

import numpy as np
import pytest

import oracle
import paper_2211_04515_b200 as qp
import synth_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ALL_BITS = [1, 2, 3, 4, 5, 6, 7, 8, 16]


@pytest.fixture(scope="module")
def lib():
    from paper_2211_04515_b200 import build
    build.build()
    return qp.load()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "quantpipe.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(qp_[a-z0-9_A-Z]+)\s*\(", header))
    assert declared == set(qp.binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_layouts():
    import ctypes as C
    assert C.sizeof(qp.Stats) == 80 and C.sizeof(qp.QParams) == 24 and C.sizeof(qp.DSResult) == 72
    assert C.sizeof(oracle.Stats) == 64 and C.sizeof(oracle.QParams) == 24 and C.sizeof(oracle.DSResult) == 72


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    import paper_2211_04515_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        b.load()


@pytest.mark.parametrize("bits", ALL_BITS)
def test_packed_bytes_and_F(lib, bits):
    for n in (0, 1, 5, 127, 128, 129, 151296, 2 ** 28, 2 ** 33 + 3):
        assert qp.qp_packed_bytes(n, bits) == oracle.packed_bytes(n, bits)
    assert qp.qp_aciq_F(bits, 0) == pytest.approx(oracle.aciq_F(bits, 0), rel=1e-14)
    assert qp.qp_aciq_F(bits, 1) == pytest.approx(oracle.aciq_F(bits, 1), rel=1e-12)


def test_unsupported_bits(lib):
    assert qp.qp_packed_bytes(10, 9) == 0 and qp.qp_packed_bytes(10, 0) == 0
    assert qp.qp_aciq_F(12, 0) == 0.0 and qp.qp_aciq_F(4, 2) == 0.0
    assert qp.qp_make_qparams(0.0, 1.0, 9)[0] == qp.QP_ERR_UNSUPPORTED_BITS
    assert qp.qp_make_qparams(float("nan"), 1.0, 4)[0] == qp.QP_ERR_INVALID_ARG
    assert qp.qp_make_qparams(0.0, float("inf"), 4)[0] == qp.QP_ERR_INVALID_ARG
    assert [qp.qp_policy_use_ds(b) for b in (1, 2, 4, 6, 8, 16)] == [True, True, True, False, False, False]
    assert "bit-width" in qp.qp_status_string(qp.QP_ERR_UNSUPPORTED_BITS)


def _same_qp(a, b):
    fa = np.array([a.lo, a.hi, a.scale, a.inv_scale], dtype=np.float32).tobytes()
    fb = np.array([b.lo, b.hi, b.scale, b.inv_scale], dtype=np.float32).tobytes()
    return fa == fb and a.bits == b.bits and a.flags == b.flags


@pytest.mark.parametrize("bits", ALL_BITS)
def test_make_qparams_bit_identical_to_oracle(lib, bits):
    rng = np.random.default_rng(bits)
    for _ in range(200):
        lo = float(rng.normal() * 10 ** rng.uniform(-3, 3))
        hi = lo + float(abs(rng.normal()) * 10 ** rng.uniform(-3, 3))
        rc, q = qp.qp_make_qparams(lo, hi, bits)
        rc_o, q_o = oracle.make_qparams(lo, hi, bits)
        assert rc == rc_o and _same_qp(q, q_o), (lo, hi)
    rc, q = qp.qp_make_qparams(2.0, 2.0, bits)
    assert rc == qp.QP_WARN_DEGENERATE and q.flags == 1 and q.scale == 0.0 and q.inv_scale == 0.0
    assert qp.qp_make_qparams(3.0, 2.0, bits)[0] == qp.QP_WARN_DEGENERATE


def test_aciq_alpha_matches_oracle(lib):
    x = si.config_tensor("c1")
    st_o = oracle.stats(x)
    st = qp.Stats(st_o.n, st_o.nonfinite, st_o.mean, st_o.mean_abs, st_o.mad, st_o.var, st_o.min, st_o.max, 0, 0, 0)
    for bits in ALL_BITS:
        for dist, bmode, ov in ((0, 0, 0.0), (0, 1, 0.0), (1, 0, 0.0), (0, 0, 0.83)):
            rc, alpha, q = qp.qp_aciq_alpha(st, bits, dist, bmode, ov)
            rc_o, alpha_o, q_o = oracle.aciq_alpha(st_o, bits, dist, bmode, ov)
            assert rc == rc_o == 0
            assert alpha == pytest.approx(alpha_o, rel=1e-12)
            assert _same_qp(q, q_o)
    assert qp.qp_aciq_alpha(st, 9)[0] == qp.QP_ERR_UNSUPPORTED_BITS
    assert qp.qp_aciq_alpha(st, 4, 3)[0] == qp.QP_ERR_INVALID_ARG


def test_clip_range_matches_oracle(lib):
    x = si.vit_activation((2, 197, 96), 21, outlier_frac=0.02)
    st_o = oracle.stats(x)
    st = qp.Stats(st_o.n, st_o.nonfinite, st_o.mean, st_o.mean_abs, st_o.mad, st_o.var, st_o.min, st_o.max, 0, 0, 0)
    for bits in ALL_BITS:
        for method, o_method, cut in ((qp.QP_CLIP_ACIQ, oracle.CLIP_ACIQ, False), (qp.QP_CLIP_MINMAX, oracle.CLIP_MINMAX, False),
                                      (qp.QP_CLIP_ACIQ | qp.QP_CLIP_INTERSECT, oracle.CLIP_ACIQ, True)):
            for dist, bmode in ((0, 0), (0, 1), (1, 0)):
                rc, lo, hi, q = qp.qp_clip_range(st, bits, method, dist, bmode)
                rc_o, lo_o, hi_o, q_o = oracle.clip_range(st_o, bits, o_method, cut, dist, bmode)
                assert rc == rc_o == 0
                assert lo == pytest.approx(lo_o, rel=1e-12, abs=1e-300) and hi == pytest.approx(hi_o, rel=1e-12, abs=1e-300)
                assert _same_qp(q, q_o)
    # mid-rise grid: the same ranges pulled in by half a bin
    for bits in (1, 4, 8, 16):
        for method, o_method, cut in ((qp.QP_CLIP_ACIQ, oracle.CLIP_ACIQ, False), (qp.QP_CLIP_MINMAX, oracle.CLIP_MINMAX, False),
                                      (qp.QP_CLIP_ACIQ | qp.QP_CLIP_INTERSECT, oracle.CLIP_ACIQ, True)):
            rc, lo, hi, q = qp.qp_clip_range(st, bits, method | qp.QP_CLIP_MIDRISE)
            rc_o, lo_o, hi_o, q_o = oracle.clip_range(st_o, bits, o_method, cut, midrise=True)
            assert rc == rc_o == 0 and lo == pytest.approx(lo_o, rel=1e-12) and hi == pytest.approx(hi_o, rel=1e-12)
            assert _same_qp(q, q_o)
    assert qp.qp_midrise_range(0.0, 4.0, 2) == (0, 0.5, 3.5) and oracle.midrise_range(0.0, 4.0, 2) == (0.5, 3.5)
    assert qp.qp_midrise_range(0.0, 4.0, 9)[0] == qp.QP_ERR_UNSUPPORTED_BITS
    assert qp.qp_clip_range(st, 4, qp.QP_CLIP_DSACIQ)[0] == qp.QP_ERR_INVALID_ARG      # needs the tensor, not a closed form
    assert qp.qp_clip_range(st, 4, qp.QP_CLIP_ACIQ | 0x40)[0] == qp.QP_ERR_INVALID_ARG
    assert qp.qp_clip_range(st, 4, qp.QP_CLIP_MINMAX | qp.QP_CLIP_INTERSECT)[0] == qp.QP_ERR_INVALID_ARG
    assert qp.qp_clip_range(st, 9)[0] == qp.QP_ERR_UNSUPPORTED_BITS
    const = qp.Stats(10, 0, 2.0, 2.0, 0.0, 0.0, 2.0, 2.0, 0, 0, 0)
    assert qp.qp_clip_range(const, 4, qp.QP_CLIP_MINMAX)[0] == qp.QP_WARN_DEGENERATE


def test_select_bits_matches_oracle(lib):
    n = 128 * 197 * 1280
    trace = si.bandwidth_trace(3, si.C4_TRACE_STEPS)
    seen = set()
    for bw in trace:
        for allowed in (si.C4_ALLOWED_BITS, (2, 4, 6, 8, 16, 32)):
            got = qp.qp_select_bits(float(bw), si.C4_BUDGET_S, n, 24, allowed)
            assert got == oracle.select_bits(float(bw), si.C4_BUDGET_S, n, 24, allowed)
            seen.add(got)
    assert {q for rc, q in seen} >= {1, 2, 3, 4, 6, 8}            # the trace exercises every width up to 8
    assert any(rc == qp.QP_WARN_INFEASIBLE for rc, q in seen)
    # default set = the bit-widths of the paper's Table 1
    for bw in (30e6, 70e6, 100e6, 200e6, 400e6, 1e9):
        assert qp.qp_select_bits(bw, 0.64, 64 * 197 * 768) == oracle.select_bits(bw, 0.64, 64 * 197 * 768)
    assert qp.qp_select_bits(1e6, 1.0, 10, 0, ())[0] == qp.QP_ERR_INVALID_ARG
    assert qp.qp_select_bits(1e6, 1.0, 10, 0, (0,))[0] == qp.QP_ERR_INVALID_ARG
    assert qp.qp_select_bits(-1.0, 1.0, 10)[0] == qp.QP_ERR_INVALID_ARG


def test_select_bits_eq2_matches_oracle_and_paper_phases(lib):
    n = 64 * 197 * 768
    for mbps, bits in ((400, 16), (50, 2), (200, 8)):              # Sec. 4.2 phases 1-3
        assert qp.qp_select_bits_eq2(n * 4.0, 32, 64, 100, mbps * 1e6) == (0, bits)
    assert qp.qp_select_bits_eq2(n * 4.0, 32, 64, 100, 1e12) == (0, 32)   # phase 4: link not limited
    rng = np.random.default_rng(0)
    for _ in range(500):
        q_t = int(rng.choice([1, 2, 4, 6, 8, 16, 32]))
        args = (float(rng.uniform(1e3, 1e9)), q_t, float(rng.integers(1, 128)), float(rng.uniform(1, 500)),
                float(10 ** rng.uniform(3, 11)))
        assert qp.qp_select_bits_eq2(*args) == oracle.select_bits_eq2(*args)
    assert qp.qp_select_bits_eq2(0.0, 32, 64, 100, 1e6)[0] == qp.QP_ERR_INVALID_ARG
    assert qp.qp_select_bits_eq2(1.0, 0, 64, 100, 1e6)[0] == qp.QP_ERR_INVALID_ARG
