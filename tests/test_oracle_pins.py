"""Pins for the CPU oracle: each check compares the oracle with something that is not the
oracle -- a closed form, SciPy / NumPy routines, exact rational arithmetic, brute force on
tiny inputs, hand-worked examples (tests/golden) and the bit-widths of the paper's
bandwidth-phase run (Sec. 4.2)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.optimize
import scipy.special
import scipy.stats

import oracle
import synth_inputs as si

ALL_BITS = [1, 2, 3, 4, 5, 6, 7, 8, 16]
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- ACIQ F(q)

@pytest.mark.parametrize("q", ALL_BITS)
def test_F_laplace_is_lambert_w(q):
    F = oracle.aciq_F(q, 0)
    ref = float(np.real(scipy.special.lambertw(3.0 * 4.0 ** q)))
    assert F == pytest.approx(ref, rel=1e-12)
    assert F * math.exp(F) == pytest.approx(3.0 * 4.0 ** q, rel=1e-12)


@pytest.mark.parametrize("q", [1, 2, 3, 4, 6, 8])
def test_F_laplace_minimises_error_model(q):
    # Laplace(0,1): clipping noise 2 exp(-a), rounding noise a^2 / (3 * 4^q)
    model = lambda a: 2.0 * math.exp(-a) + a * a / (3.0 * 4.0 ** q)
    r = scipy.optimize.minimize_scalar(model, bounds=(0.01, 60.0), method="bounded", options=dict(xatol=1e-10))
    assert oracle.aciq_F(q, 0) == pytest.approx(r.x, rel=1e-5)


@pytest.mark.parametrize("q", ALL_BITS)
def test_F_gauss_minimises_error_model(q):
    n = scipy.stats.norm
    model = lambda a: 2.0 * ((1 + a * a) * n.sf(a) - a * n.pdf(a)) + a * a / (3.0 * 4.0 ** q)
    r = scipy.optimize.minimize_scalar(model, bounds=(0.01, 12.0), method="bounded", options=dict(xatol=1e-11))
    assert oracle.aciq_F(q, 1) == pytest.approx(r.x, rel=2e-5)


def test_F_known_magnitudes():
    # the Laplace clipping multipliers grow roughly linearly in q; 2-bit value near 2.83
    assert oracle.aciq_F(2, 0) == pytest.approx(2.8307, abs=1e-4)
    assert oracle.aciq_F(4, 0) == pytest.approx(5.0286, abs=1e-4)
    assert oracle.aciq_F(2, 1) == pytest.approx(1.7106, abs=1e-4)
    Fs = [oracle.aciq_F(q, 0) for q in range(1, 9)]
    assert all(b > a for a, b in zip(Fs, Fs[1:]))


def test_laplace_error_model_matches_data():
    # On i.i.d. Laplace(0,1) data the measured MSE at the ACIQ clip follows the model the
    # constants come from: 2 exp(-a) + a^2 / (3 (L-1)^2) for this grid (L-1 intervals).
    x = si.flat_iid(1 << 22, 11, "laplace")
    st = oracle.stats(x)
    for q in (4, 6, 8):
        rc, alpha, qp = oracle.aciq_alpha(st, q)
        a = alpha / st.mad
        model = st.mad ** 2 * (2.0 * math.exp(-a) + a * a / (3.0 * (2 ** q - 1) ** 2))
        assert oracle.quant_mse(x, qp) == pytest.approx(model, rel=0.06)


def test_aciq_alpha_linear_and_centred():
    x = si.vit_activation((4, 197, 64), 5)
    st = oracle.stats(x)
    for q in (2, 4, 8, 16):
        rc, alpha, qp = oracle.aciq_alpha(st, q)
        assert rc == 0
        assert alpha == pytest.approx(oracle.aciq_F(q) * st.mad, rel=1e-14)
        assert qp.lo == np.float32(st.mean - alpha) and qp.hi == np.float32(st.mean + alpha)
        st3 = oracle.stats(3.0 * x.astype(np.float64))
        _, alpha3, _ = oracle.aciq_alpha(st3, q)
        assert alpha3 == pytest.approx(3.0 * alpha, rel=1e-6)
    _, a_lit, _ = oracle.aciq_alpha(st, 4, 0, 1)
    assert a_lit == pytest.approx(oracle.aciq_F(4) * st.mean_abs, rel=1e-14)
    _, a_g, _ = oracle.aciq_alpha(st, 4, 1, 0)
    assert a_g == pytest.approx(oracle.aciq_F(4, 1) * math.sqrt(st.var), rel=1e-14)
    _, a_o, _ = oracle.aciq_alpha(st, 4, 0, 0, 0.7)
    assert a_o == pytest.approx(oracle.aciq_F(4) * 0.7, rel=1e-14)
    assert oracle.aciq_alpha(st, 9)[0] == oracle.ERR_BITS


# ------------------------------------------------------------------- stats

def test_stats_against_numpy_and_fsum():
    x = si.vit_activation((3, 197, 96), 7)
    st = oracle.stats(x)
    xd = x.astype(np.float64).reshape(-1)
    mean = math.fsum(xd) / xd.size
    assert st.n == xd.size and st.nonfinite == 0
    assert st.mean == pytest.approx(mean, rel=1e-13, abs=1e-16)
    assert st.mean_abs == pytest.approx(math.fsum(np.abs(xd)) / xd.size, rel=1e-13)
    assert st.mad == pytest.approx(math.fsum(np.abs(xd - mean)) / xd.size, rel=1e-13)
    assert st.var == pytest.approx(math.fsum((xd - mean) ** 2) / xd.size, rel=1e-13)
    assert st.min == xd.min() and st.max == xd.max()
    assert st.var == pytest.approx(np.var(xd), rel=1e-10)


def test_stats_closed_form_and_nonfinite():
    x = np.arange(1, 1002, dtype=np.float32)          # 1..1001: mean 501, mad 250500/1001*... closed forms
    st = oracle.stats(x)
    assert st.mean == 501.0 and st.min == 1.0 and st.max == 1001.0
    assert st.mean_abs == 501.0
    assert st.mad == pytest.approx(2 * sum(range(1, 501)) / 1001.0, rel=1e-15)
    assert st.var == pytest.approx((1001 ** 2 - 1) / 12.0, rel=1e-15)
    y = np.concatenate([x, np.array([np.nan, np.inf, -np.inf], dtype=np.float32)])
    st2 = oracle.stats(y)
    assert st2.n == 1004 and st2.nonfinite == 3
    assert (st2.mean, st2.mad, st2.var, st2.min, st2.max) == (st.mean, st.mad, st.var, st.min, st.max)
    st0 = oracle.stats(np.zeros(0, dtype=np.float32))
    assert st0.n == 0 and st0.mean == 0.0 and st0.mad == 0.0
    # cancellation: large offset, small spread
    z = (np.float32(4096.0) + si.flat_iid(50000, 3, "normal")).astype(np.float32)
    stz = oracle.stats(z)
    zd = z.astype(np.float64)
    assert stz.var == pytest.approx(np.var(zd), rel=1e-9)


# --------------------------------------------------------------- quantizer

def test_hand_examples(hand_examples):
    assert len(hand_examples) == 5
    for ex in hand_examples:
        rc, qp = oracle.make_qparams(ex["lo"], ex["hi"], ex["bits"])
        assert rc == 0
        x = np.array(ex["x"], dtype=np.float32)
        codes = oracle.quantize(x, qp)
        assert codes.tolist() == ex["codes"], ex
        packed = oracle.pack(codes, ex["bits"])
        nb = len(ex["bytes"])
        assert packed[:nb].tobytes() == ex["bytes"], ex
        assert not packed[nb:].any()
        assert packed.size % 16 == 0
        assert oracle.unpack(packed, len(codes), ex["bits"]).tolist() == ex["codes"]


@pytest.mark.parametrize("q", ALL_BITS)
def test_make_qparams_definition(q):
    lo, hi = -1.2345678901, 3.9876543212
    rc, qp = oracle.make_qparams(lo, hi, q)
    assert rc == 0 and qp.bits == q and qp.flags == 0
    lo_f, hi_f = np.float32(lo), np.float32(hi)
    rng = Fraction(float(hi_f)) - Fraction(float(lo_f))
    L1 = 2 ** q - 1
    # correctly rounded from the exact quotient (np.float32 of a fp64 value that is within
    # 2^-53 relative of the exact one; ties at that level do not occur for these numbers)
    assert qp.lo == lo_f and qp.hi == hi_f
    assert qp.scale == np.float32(float(rng / L1))
    assert qp.inv_scale == np.float32(float(L1 / rng))


def test_make_qparams_degenerate_and_errors():
    rc, qp = oracle.make_qparams(1.0, 1.0, 4)
    assert rc == oracle.WARN_DEGENERATE and qp.flags == 1 and qp.scale == 0.0 and qp.inv_scale == 0.0
    assert not oracle.quantize(np.array([-5, 1, 7, np.nan], dtype=np.float32), qp).any()
    assert oracle.dequantize(np.array([0, 0], dtype=np.uint32), qp).tolist() == [1.0, 1.0]
    assert oracle.make_qparams(2.0, 1.0, 4)[0] == oracle.WARN_DEGENERATE
    assert oracle.make_qparams(0.0, 1.0, 0)[0] == oracle.ERR_BITS
    assert oracle.make_qparams(0.0, 1.0, 12)[0] == oracle.ERR_BITS
    assert oracle.make_qparams(float("nan"), 1.0, 4)[0] == oracle.ERR_ARG
    assert oracle.make_qparams(0.0, float("inf"), 4)[0] == oracle.ERR_ARG


@pytest.mark.parametrize("q", ALL_BITS)
def test_quantizer_is_textbook_affine(q):
    # naive PTQ: range = [min, max] (Sec. 3).  Compare with the affine quantizer written
    # in fp64 NumPy; codes may differ only where the fp64 position is within 1e-4 of a tie.
    x = si.vit_activation((2, 197, 48), 9).reshape(-1)
    st = oracle.stats(x)
    rc, qp = oracle.make_qparams(st.min, st.max, q)
    codes = oracle.quantize(x, qp).astype(np.int64)
    L1 = 2 ** q - 1
    pos = (np.clip(x.astype(np.float64), qp.lo, qp.hi) - qp.lo) * (L1 / (float(qp.hi) - float(qp.lo)))
    ref = np.rint(pos).astype(np.int64)
    diff = codes != ref
    assert np.all(np.abs(pos[diff] - np.floor(pos[diff]) - 0.5) < 1e-4 * max(1.0, L1 / 256))
    assert diff.mean() < 1e-3 * max(1.0, L1 / 4096)
    assert codes.min() == 0 and codes.max() == L1
    # error bound of rounding to the nearest level
    y = oracle.dequantize(codes.astype(np.uint32), qp).astype(np.float64)
    assert np.max(np.abs(y - x)) <= 0.5 * float(qp.scale) * (1 + 1e-5) + 1e-6 * np.abs(x).max()


def test_quantizer_special_values():
    rc, qp = oracle.make_qparams(-1.0, 1.0, 4)
    x = np.array([np.nan, np.inf, -np.inf, -1.0, 1.0, 0.0, -0.0, 1e30, -1e30], dtype=np.float32)
    assert oracle.quantize(x, qp).tolist() == [0, 15, 0, 0, 15, 8, 8, 15, 0]  # 7.5 -> 8 (even)


@pytest.mark.parametrize("q", ALL_BITS)
def test_dequantize_exact_rational(q):
    rc, qp = oracle.make_qparams(-0.7361, 2.4419, q)
    codes = np.unique(np.concatenate([si.random_codes(300, q, 1), np.array([0, 2 ** q - 1], dtype=np.uint32)]))
    y = oracle.dequantize(codes, qp)
    lo, sc = Fraction(float(qp.lo)), Fraction(float(qp.scale))
    for c, v in zip(codes.tolist(), y.tolist()):
        exact = lo + c * sc
        # the correctly rounded fp32 of the exact value: nearest of the two neighbours
        f = np.float32(float(exact))
        cands = [f, np.nextafter(f, np.float32(np.inf)), np.nextafter(f, np.float32(-np.inf))]
        best = min(cands, key=lambda t: abs(Fraction(float(t)) - exact))
        assert v == float(best)
    # quantizing a reconstruction level gives its code back
    assert np.array_equal(oracle.quantize(y, qp), codes)


# ------------------------------------------------------------------ packing

@pytest.mark.parametrize("q", ALL_BITS)
@pytest.mark.parametrize("n", [0, 1, 7, 31, 32, 33, 127, 128, 129, 1000])
def test_pack_is_little_endian_integer(q, n):
    codes = si.random_codes(n, q, 100 + q)
    packed = oracle.pack(codes, q)
    assert packed.size == oracle.packed_bytes(n, q) == (((n * q + 7) // 8 + 15) // 16) * 16
    big = 0
    for i, c in enumerate(codes.tolist()):
        big |= c << (i * q)
    assert packed.tobytes() == big.to_bytes(packed.size, "little")     # pad bits are zero
    # same layout through NumPy's bit packer
    bits = ((codes[:, None] >> np.arange(q, dtype=np.uint32)[None, :]) & 1).astype(np.uint8).reshape(-1)
    ref = np.packbits(bits, bitorder="little")
    assert np.array_equal(packed[:ref.size], ref)
    assert np.array_equal(oracle.unpack(packed, n, q), codes)


def test_eight_bit_is_four_times_smaller():
    # Sec. 3: 8-bit codes compress fp32 activations 4x
    n = 64 * 197 * 768
    assert oracle.packed_bytes(n, 8) * 4 == n * 4
    assert oracle.packed_bytes(n, 2) * 16 == n * 4
    assert oracle.packed_bytes(n, 16) == 2 * n
    assert oracle.packed_bytes(5, 3) == 16 and oracle.packed_bytes(0, 3) == 0


def test_quantize_pack_roundtrip_composition():
    x = si.vit_activation((1, 50, 77), 2).reshape(-1)
    st = oracle.stats(x)
    for q in ALL_BITS:
        _, _, qp = oracle.aciq_alpha(st, q)
        p = oracle.quantize_pack(x, qp)
        y = oracle.unpack_dequantize(p, x.size, qp)
        assert np.array_equal(y, oracle.dequantize(oracle.quantize(x, qp), qp))
        # idempotence: re-quantizing the reconstruction changes nothing
        assert np.array_equal(oracle.quantize_pack(y, qp), p)


# ---------------------------------------------------------------------- MSE

def test_mse_matches_numpy_and_is_monotone_in_bits():
    x = si.vit_activation((2, 197, 128), 4).reshape(-1)
    st = oracle.stats(x)
    prev = None
    for q in range(1, 9):
        _, _, qp = oracle.aciq_alpha(st, q)
        y = oracle.dequantize(oracle.quantize(x, qp), qp).astype(np.float64)
        ref = math.fsum((y - x.astype(np.float64)) ** 2) / x.size
        m = oracle.quant_mse(x, qp)
        assert m == pytest.approx(ref, rel=1e-12)
        if prev is not None:
            assert m <= prev
        prev = m
    xn = np.concatenate([x, np.array([np.nan, np.inf], dtype=np.float32)])
    assert oracle.quant_mse(xn, qp) == pytest.approx(m, rel=1e-12)      # non-finite skipped


def test_one_bit_grid_minimum_at_laplace_scale():
    # With two levels mu +- a, Laplace(0,b) data has MSE(a) = 2b^2 - 2ab + a^2: minimum b^2 at a = b.
    x = si.flat_iid(1 << 20, 21, "laplace")
    st = oracle.stats(x)
    b = st.mad
    alphas = np.linspace(0.5 * b, 1.5 * b, 201)
    mses = [oracle.quant_mse(x, oracle.make_qparams(st.mean - a, st.mean + a, 1)[1]) for a in alphas]
    k = int(np.argmin(mses))
    assert alphas[k] == pytest.approx(b, rel=0.01)
    assert mses[k] == pytest.approx(st.var - b * b, rel=1e-3)            # E x^2 - 2ab + a^2 at a=b
    for a, m in zip(alphas[::40], mses[::40]):
        assert m == pytest.approx(st.var - 2 * a * b + a * a, rel=2e-3)


def test_naive_range_is_worse_on_heavy_tails():
    # Sec. 3: the min/max range is set by rare extreme values; clipping fixes it at low bit-widths.
    x = si.vit_activation((8, 197, 256), 2).reshape(-1)
    st = oracle.stats(x)
    for q in (2, 4):
        naive = oracle.quant_mse(x, oracle.make_qparams(st.min, st.max, q)[1])
        aciq = oracle.quant_mse(x, oracle.aciq_alpha(st, q)[2])
        assert naive > 3.0 * aciq


# ---------------------------------------------------------------- histogram

@pytest.mark.parametrize("nb", [1, 7, 100, 256, 2048])
def test_histogram_counts(nb):
    x = si.vit_activation((2, 197, 64), 6).reshape(-1)
    x = np.concatenate([x, np.array([np.nan, np.inf], dtype=np.float32)])
    st = oracle.stats(x)
    peak, counts = oracle.hist_peak(x, st.min, st.max, nb)
    fin = x[np.isfinite(x)]
    assert counts.sum() == fin.size
    ref, edges = np.histogram(fin.astype(np.float64), bins=nb, range=(st.min, st.max))
    # fp32 bin positions may move elements that sit on an edge; nothing else differs
    assert np.abs(counts.astype(np.int64) - ref).sum() <= max(2, fin.size // 2000)
    w = (st.max - st.min) / nb
    assert peak == pytest.approx(counts.max() / (fin.size * w), rel=1e-14)


def test_histogram_exact_on_bin_centres_and_sorted_count():
    nb = 16
    centres = (np.arange(nb) + 0.5) / nb * 8.0                 # range [0, 8], exactly representable
    reps = np.arange(1, nb + 1)
    x = np.concatenate([np.repeat(centres, reps), [0.0, 8.0]]).astype(np.float32)
    peak, counts = oracle.hist_peak(x, 0.0, 8.0, nb)
    expect = reps.copy()
    expect[0] += 1
    expect[-1] += 1                                            # max lands in the last (closed) bin
    assert counts.tolist() == expect.tolist()
    assert peak == pytest.approx((nb + 1) / (x.size * 0.5), rel=1e-15)
    assert oracle.hist_peak(x, 3.0, 3.0, nb)[0] == 0.0         # empty range


def test_histogram_peak_of_laplace_density():
    x = si.flat_iid(1 << 21, 8, "laplace")
    st = oracle.stats(x)
    peak, _ = oracle.hist_peak(x, st.min, st.max, 512)
    assert peak == pytest.approx(0.5, rel=0.05)                # Laplace(0,1) density at 0 is 1/2


# ----------------------------------------------------------- directed search

def _numpy_candidate_mse(x, mean, alpha, q):
    """Independent fp32 NumPy evaluation of one candidate (same single-precision steps)."""
    lo, hi = np.float32(mean - alpha), np.float32(mean + alpha)
    L1 = 2 ** q - 1
    rng = float(hi) - float(lo)
    scale, inv = np.float32(rng / L1), np.float32(L1 / rng)
    t = np.minimum(np.maximum(x, lo), hi)
    v = ((t - lo).astype(np.float32) * inv).astype(np.float32)
    code = np.clip(np.rint(v), 0, L1)
    dq = (np.float64(lo) + code.astype(np.float64) * np.float64(scale)).astype(np.float32)
    return float(np.mean((dq.astype(np.float64) - x.astype(np.float64)) ** 2))


@pytest.mark.parametrize("q,seed,nb", [(2, 1, 100), (4, 2, 100), (3, 3, 64), (8, 4, 100), (2, 5, 2048), (1, 6, 100)])
def test_ds_search_equals_brute_force(q, seed, nb):
    x = si.vit_activation((1, 16, 256), seed, outlier_frac=0.02 if seed % 2 else 0.0).reshape(-1)
    st = oracle.stats(x)
    rc, res, qp, curve = oracle.ds_search(x, st, q, 0, 100, nb)
    assert rc == 0
    fin = x.astype(np.float64)
    counts, _ = np.histogram(fin, bins=nb, range=(st.min, st.max))
    w = (st.max - st.min) / nb
    peak_ref = counts.max() / (x.size * w)
    assert res.b_e == st.mad
    assert res.b_r == pytest.approx(1.0 / (2.0 * peak_ref), rel=0.02)   # edge elements may move one count
    F = float(np.real(scipy.special.lambertw(3.0 * 4.0 ** q)))
    mses = np.array([_numpy_candidate_mse(x, st.mean, F * (res.b_e + k * (res.b_r - res.b_e) / 100), q)
                     for k in range(101)])
    assert np.allclose(curve, mses, rtol=1e-9)
    k_ref = int(np.argmin(mses))                       # first index of the minimum
    assert res.k_star == k_ref or abs(mses[res.k_star] - mses[k_ref]) <= 1e-12 * mses[k_ref]
    assert res.mse_star <= res.mse_e and res.mse_e == pytest.approx(mses[0], rel=1e-9)
    assert res.b_star == pytest.approx(res.b_e + res.k_star * (res.b_r - res.b_e) / 100, rel=1e-15)
    assert res.alpha_star == pytest.approx(F * res.b_star, rel=1e-12)
    assert res.alpha_e == pytest.approx(F * res.b_e, rel=1e-12)
    assert qp.lo == np.float32(st.mean - res.alpha_star) and qp.hi == np.float32(st.mean + res.alpha_star)
    assert oracle.quant_mse(x, qp) == res.mse_star
    # never worse than plain ACIQ, never better than a fine exhaustive scan of the same interval
    lo_b, hi_b = min(res.b_e, res.b_r), max(res.b_e, res.b_r)
    fine = min(_numpy_candidate_mse(x, st.mean, F * b, q) for b in np.linspace(lo_b, hi_b, 2001))
    assert fine <= res.mse_star * (1 + 1e-9)
    assert res.mse_star <= fine * 1.05 or res.k_star in (0, 100) or q == 1


def test_ds_direction_follows_histogram_peak():
    # flat-topped data: histogram peak lower than the Laplace fit's peak -> b_R > b_E
    u = (si.uniform01(3, si.STREAM_VALUE, 0, 20000) * 2 - 1).astype(np.float32)
    st = oracle.stats(u)
    _, res, _, _ = oracle.ds_search(u, st, 2, 0, 100, 100)
    assert res.b_r > res.b_e and res.b_e <= res.b_star <= res.b_r
    assert 1.0 / (2 * res.b_e) > 0.5                              # max(D_E) = 1/(2 b_E) = 1 > max(D_R) ~ 0.5
    # sharply peaked mixture: most mass in a narrow spike -> b_R < b_E
    spike = np.concatenate([0.01 * si.flat_iid(18000, 4, "laplace"), 3.0 * si.flat_iid(2000, 5, "laplace")]).astype(np.float32)
    st = oracle.stats(spike)
    _, res, _, _ = oracle.ds_search(spike, st, 2, 0, 100, 2048)
    assert res.b_r < res.b_e and res.b_r <= res.b_star <= res.b_e
    assert res.mse_star <= res.mse_e


def _gauss_F_numeric(q):
    """Minimiser of the normal clipping-plus-rounding model, by SciPy (independent of the oracle's bisection)."""
    from scipy.optimize import minimize_scalar
    from scipy.stats import norm
    model = lambda a: 2.0 * ((1.0 + a * a) * norm.sf(a) - a * norm.pdf(a)) + a * a / (3.0 * 4.0 ** q)
    return minimize_scalar(model, bounds=(0.1, 12.0), method="bounded", options={"xatol": 1e-12}).x


@pytest.mark.parametrize("q,seed,nb", [(2, 1, 100), (4, 2, 100), (3, 3, 256)])
def test_ds_search_gaussian_model(q, seed, nb):
    """bmode | 0x20: the directed search with the normal density's scale and peak, against an
    independent evaluation of its 101 candidates."""
    x = si.vit_activation((1, 16, 256), seed, outlier_frac=0.02 if seed % 2 else 0.0).reshape(-1)
    st = oracle.stats(x)
    rc, res, qp, curve = oracle.ds_search(x, st, q, 0x20, 100, nb)
    assert rc == 0
    counts, _ = np.histogram(x.astype(np.float64), bins=nb, range=(st.min, st.max))
    peak_ref = counts.max() / (x.size * (st.max - st.min) / nb)
    assert res.b_e == math.sqrt(st.var)                                          # sigma_E
    assert res.b_r == pytest.approx(1.0 / (math.sqrt(2.0 * math.pi) * peak_ref), rel=0.02)   # sigma_R
    F = _gauss_F_numeric(q)
    mses = np.array([_numpy_candidate_mse(x, st.mean, F * (res.b_e + k * (res.b_r - res.b_e) / 100), q)
                     for k in range(101)])
    assert np.allclose(curve, mses, rtol=1e-5)              # F from two solvers: alpha agrees to ~1e-8
    k_ref = int(np.argmin(mses))
    assert res.k_star == k_ref or abs(mses[res.k_star] - mses[k_ref]) <= 1e-6 * mses[k_ref]
    assert res.mse_star <= res.mse_e
    assert res.alpha_e == pytest.approx(F * math.sqrt(st.var), rel=1e-6)       # a numeric minimiser finds F to ~1e-8
    assert res.alpha_star == pytest.approx(F * res.b_star, rel=1e-6)
    # step 0 is plain Gaussian ACIQ
    _, alpha0, qp0 = oracle.aciq_alpha(st, q, dist=1)
    assert alpha0 == res.alpha_e and curve[0] == oracle.quant_mse(x, qp0)
    assert oracle.quant_mse(x, qp) == res.mse_star


def test_ds_search_gaussian_peak_relation_and_direction():
    # normal data: the histogram peak estimates 1 / (sigma sqrt(2 pi)), so sigma_R ~ sigma_E
    g = (0.7 * si.flat_iid(1 << 20, 11, "normal")).astype(np.float32)
    st = oracle.stats(g)
    _, res, _, _ = oracle.ds_search(g, st, 4, 0x20, 100, 256)
    assert res.b_e == pytest.approx(0.7, rel=0.01) and res.b_r == pytest.approx(res.b_e, rel=0.05)
    # the Laplace-model search on the same data sees a peak below a Laplace fit's: b_R > b_E
    _, res_l, _, _ = oracle.ds_search(g, st, 4, 0, 100, 256)
    assert res_l.b_r > res_l.b_e
    # uniform data is flatter than a normal of the same variance: sigma_R = 2a / sqrt(2 pi) > a / sqrt(3)
    u = (si.uniform01(3, si.STREAM_VALUE, 0, 200000) * 2 - 1).astype(np.float32)
    st = oracle.stats(u)
    _, res, _, _ = oracle.ds_search(u, st, 2, 0x20, 100, 100)
    assert res.b_e == pytest.approx(1 / math.sqrt(3), rel=0.01)
    # the fullest of 100 bins of 2000 expected counts lies ~2.5 Poisson deviations above the mean (+6 %)
    assert 0.93 * 2 / math.sqrt(2 * math.pi) < res.b_r <= 2 / math.sqrt(2 * math.pi) and res.b_r > res.b_e
    # Laplace data is more peaked than a normal of the same variance: sigma_R < sigma_E
    lap = si.flat_iid(1 << 18, 12, "laplace")
    st = oracle.stats(lap)
    _, res, _, _ = oracle.ds_search(lap, st, 2, 0x20, 100, 256)
    assert res.b_r < res.b_e and res.b_r <= res.b_star <= res.b_e
    # the literal-formula scale has no Gaussian counterpart; flags combine with the mid-rise grid
    assert oracle.ds_search(lap, st, 2, 0x21)[0] == oracle.ERR_ARG
    rc, res_m, qp_m, _ = oracle.ds_search(lap, st, 2, 0x30, 100, 256)
    assert rc == 0 and res_m.b_e == res.b_e and res_m.b_r == res.b_r


def test_ds_degenerate_and_arguments():
    c = np.full(100, 2.5, dtype=np.float32)
    st = oracle.stats(c)
    rc, res, qp, curve = oracle.ds_search(c, st, 2)
    assert rc == oracle.WARN_DEGENERATE and res.k_star == 0 and res.b_star == res.b_e == 0.0
    assert qp.flags == 1 and res.mse_star == 0.0
    x = si.flat_iid(1000, 1, "laplace")
    st = oracle.stats(x)
    assert oracle.ds_search(x, st, 16)[0] == oracle.ERR_BITS
    assert oracle.ds_search(x, st, 4, steps=0)[0] == oracle.ERR_ARG
    # literal b_E = sum|x|/N when asked
    _, res, _, _ = oracle.ds_search(x, st, 4, bmode=1)
    assert res.b_e == st.mean_abs
    # one-step search: candidates are exactly b_E and b_R
    _, res, _, curve = oracle.ds_search(x, st, 4, steps=1)
    assert len(curve) == 2 and res.k_star in (0, 1)


def test_ds_never_worse_and_monotone_over_bits():
    x = si.config_tensor("c1").reshape(-1)
    st = oracle.stats(x)
    prev = None
    for q in (1, 2, 3, 4, 5, 6, 7, 8):
        _, res, _, _ = oracle.ds_search(x, st, q)
        assert res.mse_star <= res.mse_e
        if prev is not None:
            assert res.mse_star <= prev
        prev = res.mse_star


# -------------------------------------------------------------- select_bits

def _phases():
    rows = []
    for line in open(os.path.join(GOLDEN, "adaptive_phases.txt")):
        if line.strip() and not line.startswith("#"):
            mbps, bits = line.split()
            rows.append((float(mbps), int(bits)))
    return rows


def test_eq2_reproduces_paper_phases():
    n = 64 * 197 * 768
    for r_target in (85.0, 100.0, 160.0):
        for q_now in (32, 16, 8, 2):                      # Eq. 2 rescales V to fp32 size first
            v_bytes = n * q_now / 8.0
            for mbps, bits in _phases():
                bw = 1e12 if mbps == 0 else mbps * 1e6
                rc, q = oracle.select_bits_eq2(v_bytes, q_now, 64, r_target, bw)
                assert rc == 0 and q == bits, (r_target, q_now, mbps)


def test_eq2_by_hand():
    # c = 309.854208e6 / (0.64 * 200e6) = 2.4207 -> ceil(log2) = 2 -> 32/4 = 8
    assert oracle.select_bits_eq2(64 * 197 * 768 * 4, 32, 64, 100, 200e6) == (0, 8)
    assert oracle.select_bits_eq2(1000, 32, 1, 1, 8000.0) == (0, 32)       # c = 1 exactly: fits
    assert oracle.select_bits_eq2(1000, 32, 1, 1, 7999.0) == (0, 16)
    assert oracle.select_bits_eq2(1000, 32, 1, 1, 1.0) == (0, 1)           # clamped below
    assert oracle.select_bits_eq2(0, 32, 1, 1, 1.0)[0] == oracle.ERR_ARG


def test_select_bits_principle():
    n = 64 * 197 * 768
    budget = 0.64
    allowed = (32, 16, 8, 6, 4, 2)
    # the paper's phases with the table's bit-width set: same settled answers as Eq. 2
    for mbps, bits in _phases():
        bw = 1e12 if mbps == 0 else mbps * 1e6
        assert oracle.select_bits(bw, budget, n, 0, allowed) == (0, bits)
    # 6 bits is chosen in a band below 8 bits' threshold (the transient of phase 3)
    assert oracle.select_bits(100e6, budget, n, 0, allowed) == (0, 6)
    # exact thresholds: payload bits <= capacity
    need = 8 * ((n * 6 + 7) // 8)
    assert oracle.select_bits(need / budget * (1 + 1e-12), budget, n, 0, allowed)[1] == 6
    assert oracle.select_bits(need / budget * (1 - 1e-9), budget, n, 0, allowed)[1] == 4
    assert oracle.select_bits(need / budget * (1 + 1e-12), budget, n, 1, allowed)[1] == 4   # header bytes count
    # monotone in bandwidth, infeasible -> smallest with a warning
    last = 0
    for bw in np.linspace(1e6, 600e6, 400):
        rc, q = oracle.select_bits(bw, budget, n, 0, allowed)
        assert q >= last
        last = q
        assert (rc == oracle.WARN_INFEASIBLE) == (8 * ((n * 2 + 7) // 8) > bw * budget)
    assert oracle.select_bits(1.0, budget, n, 0, (4, 2, 8)) == (oracle.WARN_INFEASIBLE, 2)
    assert oracle.select_bits(1e6, 1.0, 10, 0, ())[0] == oracle.ERR_ARG
    assert oracle.select_bits(1e6, 1.0, 10, 0, (0,))[0] == oracle.ERR_ARG


# ------------------------------------------------------------- clip range by method

def test_naive_ptq_range_is_min_max_hand_example():
    """Sec. 3: naive PTQ divides the tensor's own range into equal intervals.  By hand: the values
    0, 0.9, 2.2, 3 at 2 bits have range [0, 3], four levels 0, 1, 2, 3 -> codes 0, 1, 2, 3 and
    reconstructions 0, 1, 2, 3."""
    x = np.array([0.0, 0.9, 2.2, 3.0], dtype=np.float32)
    rc, lo, hi, q = oracle.clip_range(oracle.stats(x), 2, oracle.CLIP_MINMAX)
    assert rc == 0 and (lo, hi) == (0.0, 3.0) and q.scale == 1.0
    codes = oracle.quantize(x, q)
    assert codes.tolist() == [0, 1, 2, 3]
    assert oracle.dequantize(codes, q).tolist() == [0.0, 1.0, 2.0, 3.0]
    # the extremes always take the end codes and are reconstructed exactly
    y = si.flat_iid(10000, 9, "laplace")
    for bits in (1, 3, 8, 16):
        rc, lo, hi, q = oracle.clip_range(oracle.stats(y), bits, oracle.CLIP_MINMAX)
        c = oracle.quantize(y, q)
        assert c[np.argmin(y)] == 0 and c[np.argmax(y)] == (1 << bits) - 1
        d = oracle.dequantize(c, q)
        assert d[np.argmin(y)] == y.min() and abs(d[np.argmax(y)] - y.max()) <= 2e-7 * abs(y.max())
        # nothing is clipped; the position on the grid is an fp32 number of up to 2^bits, so half a
        # step is met up to its rounding
        assert np.max(np.abs(d - y)) <= (0.5 + 2.0 ** -22 * (1 << bits)) * q.scale


def test_clip_range_aciq_equals_aciq_alpha_and_intersection_properties():
    y = si.flat_iid(50000, 10, "laplace") * np.float32(0.7) + np.float32(0.3)
    st = oracle.stats(y)
    for bits in (2, 4, 8, 16):
        rc, alpha, q_a = oracle.aciq_alpha(st, bits)
        rc, lo, hi, q = oracle.clip_range(st, bits, oracle.CLIP_ACIQ)
        assert (lo, hi) == (st.mean - alpha, st.mean + alpha) and bytes(q) == bytes(q_a)
        rc, lo_i, hi_i, q_i = oracle.clip_range(st, bits, oracle.CLIP_ACIQ, intersect=True)
        assert lo_i == max(lo, st.min) and hi_i == min(hi, st.max)       # never wider, never inside the data
        if lo > st.min and hi < st.max:
            assert bytes(q_i) == bytes(q)                                # alpha inside the data: nothing changes
    # at 16 bits alpha = F(16) b reaches far past this sample's extremes: the cut range is naive PTQ's
    rc, lo_i, hi_i, q_i = oracle.clip_range(st, 16, oracle.CLIP_ACIQ, intersect=True)
    rc, lo_n, hi_n, q_n = oracle.clip_range(st, 16, oracle.CLIP_MINMAX)
    assert (lo_i, hi_i) == (lo_n, hi_n) == (st.min, st.max) and bytes(q_i) == bytes(q_n)
    # and it lowers the error there (same clipping error - none - and a smaller step)
    rc, lo, hi, q = oracle.clip_range(st, 16, oracle.CLIP_ACIQ)
    assert oracle.quant_mse(y, q_i) < 0.5 * oracle.quant_mse(y, q)
    # a one-sided cut: shift the data so that only the lower end of the ACIQ range passes the minimum
    z = np.abs(y).astype(np.float32)
    sz = oracle.stats(z)
    rc, lo, hi, q = oracle.clip_range(sz, 3, oracle.CLIP_ACIQ)
    rc, lo_i, hi_i, q_i = oracle.clip_range(sz, 3, oracle.CLIP_ACIQ, intersect=True)
    assert lo < sz.min and hi < sz.max and lo_i == sz.min and hi_i == hi
    assert oracle.quant_mse(z, q_i) < oracle.quant_mse(z, q)
    assert oracle.clip_range(st, 9)[0] == oracle.ERR_BITS
    assert oracle.clip_range(st, 4, 1)[0] == oracle.ERR_ARG               # the search is not a closed form
    assert oracle.clip_range(st, 4, oracle.CLIP_MINMAX, intersect=True)[0] == oracle.ERR_ARG


# ------------------------------------------------------------------- mid-rise grid

def test_midrise_hand_example_and_bin_centres():
    """[0, 4] at 2 bits: four bins of width 1 with centres 0.5, 1.5, 2.5, 3.5 (by hand).  As a clip range that
    is [0.5, 3.5] with step 1: 0.9 -> 0.5, 1.1 -> 1.5, 2.49 -> 2.5, 3.99 -> 3.5, and the ends 0 and 4 go to the
    outermost centres."""
    assert oracle.midrise_range(0.0, 4.0, 2) == (0.5, 3.5)
    q = oracle.make_qparams(*oracle.midrise_range(0.0, 4.0, 2), 2)[1]
    assert q.scale == 1.0
    x = np.array([0.0, 0.9, 1.1, 2.49, 2.51, 3.99, 4.0, -7.0, 9.0], dtype=np.float32)
    back = oracle.dequantize(oracle.quantize(x, q), q)
    assert back.tolist() == [0.5, 0.5, 1.5, 2.5, 2.5, 3.5, 3.5, 0.5, 3.5]
    # every element inside the range lies in the bin whose centre it is given: |x - x^| <= w / 2
    for bits in (1, 3, 8):
        lo, hi = -1.25, 2.75
        w = (hi - lo) / 2 ** bits
        qb = oracle.make_qparams(*oracle.midrise_range(lo, hi, bits), bits)[1]
        y = np.linspace(lo, hi, 20001).astype(np.float32)
        codes = oracle.quantize(y, qb)
        back = oracle.dequantize(codes, qb).astype(np.float64)
        assert np.max(np.abs(back - y)) <= w / 2 * (1 + 1e-5) + 1e-6
        assert codes.min() == 0 and codes.max() == 2 ** bits - 1
        inner = (y > lo + 1e-3) & (y < hi - 1e-3) & (np.abs((y - lo) / w - np.round((y - lo) / w)) > 1e-3)
        assert np.array_equal(codes[inner], np.floor((y[inner].astype(np.float64) - lo) / w).astype(np.uint32))


def test_midrise_matches_the_aciq_noise_model():
    """The ACIQ multiplier minimises 2 b^2 exp(-alpha / b) + alpha^2 / (3 * 4^q) (Sec. 3; the second term is
    the rounding noise w^2 / 12 of 2^q bins of width w = 2 alpha / 2^q, the first the clipping error).  The
    expression treats the density as flat inside a bin, so it is an approximation that gets better with
    more bits: on Laplace data the measured MSE of the mid-rise grid follows it to a few percent from 5
    bits on (3 % at 6 bits)."""
    y = si.flat_iid(400000, 21, "laplace")
    st = oracle.stats(y)
    for bits, tol in ((5, 0.08), (6, 0.04), (8, 0.07)):
        rc, lo, hi, q_mr = oracle.clip_range(st, bits, oracle.CLIP_ACIQ, midrise=True)
        rc, lo0, hi0, q_mt = oracle.clip_range(st, bits, oracle.CLIP_ACIQ)
        alpha = (hi0 - lo0) / 2
        assert (hi - lo) / 2 == pytest.approx(alpha * (1 - 2.0 ** -bits), rel=1e-12)     # half a bin in on each side
        model = 2 * st.mad ** 2 * math.exp(-alpha / st.mad) + alpha ** 2 / (3 * 4 ** bits)
        assert abs(oracle.quant_mse(y, q_mr) - model) <= tol * model, (bits, oracle.quant_mse(y, q_mr), model)
    # uniform data over the range: no clipping, MSE = w^2 / 12
    u = (np.random.default_rng(5).random(400000) * 6.0 - 1.0).astype(np.float32)
    for bits in (2, 5):
        w = 6.0 / 2 ** bits
        q = oracle.make_qparams(*oracle.midrise_range(-1.0, 5.0, bits), bits)[1]
        assert oracle.quant_mse(u, q) == pytest.approx(w * w / 12, rel=0.01)


def test_midrise_in_the_search_and_with_the_other_flags():
    y = si.vit_activation((2, 197, 96), 22, outlier_frac=0.02).reshape(-1)
    st = oracle.stats(y)
    rc, res, q, curve = oracle.ds_search(y, st, 3, oracle.B_MIDRISE)
    rc0, res0, q0, curve0 = oracle.ds_search(y, st, 3, 0)
    assert (res.b_e, res.b_r) == (res0.b_e, res0.b_r)                  # same candidates b_k, another grid
    F = oracle.aciq_F(3, 0)
    for k in (0, res.k_star, 100):
        alpha = F * (res.b_e + k * (res.b_r - res.b_e) / 100)
        qk = oracle.make_qparams(*oracle.midrise_range(st.mean - alpha, st.mean + alpha, 3), 3)[1]
        assert curve[k] == oracle.quant_mse(y, qk)
    assert curve[res.k_star] == curve.min() and bytes(q) != bytes(q0)
    # order of the flags: cut back to the data first, then the half-bin shift
    rc, lo, hi, qa = oracle.clip_range(st, 8, oracle.CLIP_ACIQ, intersect=True, midrise=True)
    rc, lo_i, hi_i, _ = oracle.clip_range(st, 8, oracle.CLIP_ACIQ, intersect=True)
    assert (lo, hi) == oracle.midrise_range(lo_i, hi_i, 8)
    rc, lo, hi, qn = oracle.clip_range(st, 4, oracle.CLIP_MINMAX, midrise=True)
    assert (lo, hi) == oracle.midrise_range(st.min, st.max, 4)
    assert oracle.clip_range(st, 4, oracle.CLIP_MINMAX, intersect=True, midrise=True)[0] == oracle.ERR_ARG


# ------------------------------------------------------- per-channel quantization

def test_channels_hand_example_two_scales():
    """Two channels whose scales differ by ten: channel 0 holds 0, 1, 2, 3 and channel 1 holds 0, 10, 20,
    30.  With the min/max range at 2 bits each channel has its own four levels, so every value is a level
    and is reconstructed exactly; one range for the whole tensor, [0, 30] with levels 0, 10, 20, 30, sends
    channel 0's 1, 2, 3 to 0 (by hand)."""
    x = np.array([[0, 0], [1, 10], [2, 20], [3, 30]], dtype=np.float32)
    st = oracle.stats_channels(x, 2)
    assert [(s.min, s.max, s.n) for s in st] == [(0.0, 3.0, 4), (0.0, 30.0, 4)]
    rc, qp = oracle.clip_channels(st, 2, oracle.CLIP_MINMAX)
    assert rc == 0 and (qp[0].scale, qp[1].scale) == (1.0, 10.0)
    codes = oracle.quantize_channels(x, 2, qp)
    assert codes.reshape(4, 2).tolist() == [[0, 0], [1, 1], [2, 2], [3, 3]]
    assert np.array_equal(oracle.dequantize_channels(codes, 2, qp).reshape(4, 2), x)
    whole = oracle.clip_range(oracle.stats(x), 2, oracle.CLIP_MINMAX)[3]
    assert oracle.dequantize(oracle.quantize(x, whole), whole).reshape(4, 2)[:, 0].tolist() == [0.0, 0.0, 0.0, 0.0]


def test_channels_statistics_against_numpy_columns():
    x = si.vit_activation((3, 50, 24), 11, outlier_frac=0.1).reshape(-1, 24)
    x[5, 3] = np.nan
    x[7, 3] = np.inf
    st = oracle.stats_channels(x, 24)
    x64 = x.astype(np.float64)
    for c in range(24):
        col = x64[:, c]
        col = col[np.isfinite(col)]
        assert st[c].n == 150 and st[c].nonfinite == (2 if c == 3 else 0)
        assert st[c].mean == pytest.approx(col.mean(), rel=1e-12, abs=1e-15)
        assert st[c].mean_abs == pytest.approx(np.abs(col).mean(), rel=1e-12)
        assert st[c].mad == pytest.approx(np.abs(col - col.mean()).mean(), rel=1e-12)
        assert st[c].var == pytest.approx(col.var(), rel=1e-12)
        assert (st[c].min, st[c].max) == (col.min(), col.max())


def test_channels_one_channel_is_the_per_tensor_path_and_symmetries():
    y = si.flat_iid(6000, 12, "laplace")
    # a single channel: exactly the per-tensor functions
    st1 = oracle.stats_channels(y, 1)
    assert bytes(st1[0]) == bytes(oracle.stats(y))
    for bits in (2, 4, 8):
        rc, qp1 = oracle.clip_channels(st1, bits)
        q = oracle.aciq_alpha(oracle.stats(y), bits)[2]
        assert bytes(qp1[0]) == bytes(q)
        assert np.array_equal(oracle.quantize_channels(y, 1, qp1), oracle.quantize(y, q))
        assert np.array_equal(oracle.dequantize_channels(oracle.quantize(y, q), 1, qp1), oracle.dequantize(oracle.quantize(y, q), q))
    # element i belongs to channel i mod C (not i div rows): transposing the roles must change the answer
    x = si.vit_activation((1, 40, 6), 13, outlier_frac=0.2).reshape(40, 6)
    st = oracle.stats_channels(x, 6)
    assert all(st[c].mean == pytest.approx(float(x[:, c].astype(np.float64).mean()), rel=1e-12) for c in range(6))
    rc, qp = oracle.clip_channels(st, 4)
    codes = oracle.quantize_channels(x, 6, qp).reshape(40, 6)
    # channels do not interact: scaling one channel by a power of two scales its range and leaves all codes alone
    x2 = x.copy()
    x2[:, 2] *= np.float32(8.0)
    st2 = oracle.stats_channels(x2, 6)
    rc, qp2 = oracle.clip_channels(st2, 4)
    assert (qp2[2].lo, qp2[2].hi, qp2[2].scale) == (8 * qp[2].lo, 8 * qp[2].hi, 8 * qp[2].scale)
    assert all(bytes(qp2[c]) == bytes(qp[c]) for c in range(6) if c != 2)
    assert np.array_equal(oracle.quantize_channels(x2, 6, qp2).reshape(40, 6), codes)
    # permuting the channels permutes statistics, quantizers and codes
    perm = np.array([3, 0, 5, 1, 4, 2])
    xp = np.ascontiguousarray(x[:, perm])
    stp = oracle.stats_channels(xp, 6)
    rc, qpp = oracle.clip_channels(stp, 4)
    assert all(bytes(qpp[j]) == bytes(qp[perm[j]]) for j in range(6))
    assert np.array_equal(oracle.quantize_channels(xp, 6, qpp).reshape(40, 6), codes[:, perm])
    # with outlier channels, channel-wise ranges lower the error of the whole tensor
    z = si.vit_activation((2, 197, 64), 14, outlier_frac=0.05).reshape(-1, 64)
    stz = oracle.stats_channels(z, 64)
    rc, qz = oracle.clip_channels(stz, 4)
    err_c = np.mean((oracle.dequantize_channels(oracle.quantize_channels(z, 64, qz), 64, qz).astype(np.float64) - z.reshape(-1)) ** 2)
    q_t = oracle.aciq_alpha(oracle.stats(z), 4)[2]
    assert err_c < 0.5 * oracle.quant_mse(z, q_t)
    # a constant channel is degenerate: code 0, reconstructed exactly, and the call says so
    z[:, 7] = np.float32(1.5)
    rc, qz = oracle.clip_channels(oracle.stats_channels(z, 64), 4)
    assert rc == oracle.WARN_DEGENERATE and qz[7].flags == 1
    back = oracle.dequantize_channels(oracle.quantize_channels(z, 64, qz), 64, qz).reshape(-1, 64)
    assert np.all(back[:, 7] == np.float32(1.5))


def test_channels_directed_search():
    """The search per channel: every column gets what the per-tensor search gives for it alone."""
    C_, rows = 5, 3000
    x = si.vit_activation((1, rows, C_), 15, outlier_frac=0.2).reshape(rows, C_)
    st = oracle.stats_channels(x, C_)
    rc, res, qp, curves = oracle.ds_search_channels(x, C_, st, 2, 0, 100, 64)
    assert rc == 0 and curves.shape == (C_, 101)
    F = float(np.real(scipy.special.lambertw(3.0 * 4.0 ** 2)))
    for c in range(C_):
        col = np.ascontiguousarray(x[:, c])
        # independent evaluation of the column's candidates (NumPy histogram and quantizer)
        counts, _ = np.histogram(col.astype(np.float64), bins=64, range=(st[c].min, st[c].max))
        peak = counts.max() / (rows * (st[c].max - st[c].min) / 64)
        assert res[c].b_e == st[c].mad and res[c].b_r == pytest.approx(1.0 / (2.0 * peak), rel=0.03)
        mses = np.array([_numpy_candidate_mse(col, st[c].mean, F * (res[c].b_e + k * (res[c].b_r - res[c].b_e) / 100), 2)
                         for k in range(101)])
        assert np.allclose(curves[c], mses, rtol=1e-9)
        k_ref = int(np.argmin(mses))
        assert res[c].k_star == k_ref or abs(mses[res[c].k_star] - mses[k_ref]) <= 1e-12 * mses[k_ref]
        assert qp[c].lo == np.float32(st[c].mean - res[c].alpha_star) and qp[c].hi == np.float32(st[c].mean + res[c].alpha_star)
        assert res[c].mse_star <= res[c].mse_e
    # the searched quantizers lower the whole tensor's error below the channel-wise ACIQ ranges
    back = oracle.dequantize_channels(oracle.quantize_channels(x, C_, qp), C_, qp).astype(np.float64)
    err_ds = np.mean((back - x.reshape(-1)) ** 2)
    _, qa = oracle.clip_channels(st, 2)
    back_a = oracle.dequantize_channels(oracle.quantize_channels(x, C_, qa), C_, qa).astype(np.float64)
    assert err_ds <= np.mean((back_a - x.reshape(-1)) ** 2)
    assert err_ds == pytest.approx(np.mean([res[c].mse_star for c in range(C_)]), rel=1e-12)
    # one channel: the per-tensor search, byte for byte
    y = np.ascontiguousarray(x[:, 3])
    st1 = oracle.stats_channels(y, 1)
    _, res1, qp1, curve1 = oracle.ds_search_channels(y, 1, st1, 3, 0x10, 50, 100)
    _, res_t, qp_t, curve_t = oracle.ds_search(y, oracle.stats(y), 3, 0x10, 50, 100)
    assert bytes(res1[0]) == bytes(res_t) and bytes(qp1[0]) == bytes(qp_t) and np.array_equal(curve1[0], curve_t)
    # channels do not interact; a constant channel is reported and keeps b_E = 0
    x2 = x.copy()
    x2[:, 1] = np.float32(-2.0)
    rc2, res2, qp2, _ = oracle.ds_search_channels(x2, C_, oracle.stats_channels(x2, C_), 2, 0, 100, 64)
    assert rc2 == oracle.WARN_DEGENERATE and qp2[1].flags == 1 and res2[1].k_star == 0
    assert all(bytes(res2[c]) == bytes(res[c]) and bytes(qp2[c]) == bytes(qp[c]) for c in range(C_) if c != 1)
    assert oracle.ds_search_channels(x, C_, st, 16)[0] == oracle.ERR_BITS


# ------------------------------------------------------------------- inputs

def test_generator_is_counter_based_and_shaped():
    a = si.flat_iid(5000, 4, "laplace")
    b = si.laplace01(4, si.STREAM_VALUE, 1234, 100).astype(np.float32)
    assert np.array_equal(a[1234:1334], b)
    x = si.config_tensor("c1")
    assert x.shape == (1, 197, 768) and x.dtype == np.float32
    mu, s = si.channel_params(0, 768)
    assert np.all(np.abs(x.reshape(-1, 768).mean(0) - mu) <= 6 * s * math.sqrt(2.0 / 197))
    x3 = si.vit_activation((4, 197, 1024), 2, outlier_frac=0.01)
    sd = x3.reshape(-1, 1024).std(0)
    assert (sd > 8 * np.median(sd)).sum() >= 5
    h = si.to_bf16_bits(a)
    assert np.array_equal(oracle.widen_bf16(h), si.bf16_bits_to_f32(h))
    assert np.max(np.abs(si.bf16_bits_to_f32(h) - a) / np.maximum(np.abs(a), 1e-30)) <= 2.0 ** -8
    bw = si.bandwidth_trace(3, 100)
    assert bw.min() >= 5e6 and bw.max() <= 200e6 and len(np.unique(bw)) == 100


# ------------------------------------------------------- per-token quantization

def test_tokens_hand_example_two_scales():
    """Two tokens whose scales differ by ten: token 0 holds 0, 1, 2, 3 and token 1 holds 0, 10, 20, 30.
    With the min/max range at 2 bits every token has its own four levels, so every value is a level and
    is reconstructed exactly; one range for the whole tensor, [0, 30], sends token 0's 1, 2, 3 to 0."""
    x = np.array([[0, 1, 2, 3], [0, 10, 20, 30]], dtype=np.float32)
    st = oracle.stats_tokens(x, 4)
    assert [(s.min, s.max, s.n) for s in st] == [(0.0, 3.0, 4), (0.0, 30.0, 4)]
    rc, qp = oracle.clip_tokens(st, 2, oracle.CLIP_MINMAX)
    assert rc == 0 and (qp[0].scale, qp[1].scale) == (1.0, 10.0)
    codes = oracle.quantize_tokens(x, 4, qp)
    assert codes.reshape(2, 4).tolist() == [[0, 1, 2, 3], [0, 1, 2, 3]]
    assert np.array_equal(oracle.dequantize_tokens(codes, 4, qp).reshape(2, 4), x)
    whole = oracle.clip_range(oracle.stats(x), 2, oracle.CLIP_MINMAX)[3]
    assert oracle.dequantize(oracle.quantize(x, whole), whole).reshape(2, 4)[0].tolist() == [0.0, 0.0, 0.0, 0.0]


def test_tokens_against_numpy_rows_and_against_the_channel_functions_on_the_transpose():
    x = si.vit_activation((1, 37, 24), 16, outlier_frac=0.1).reshape(37, 24)
    x[5, 3] = np.nan
    x[5, 7] = -np.inf
    st = oracle.stats_tokens(x, 24)
    x64 = x.astype(np.float64)
    for t in range(37):
        row = x64[t][np.isfinite(x64[t])]
        assert st[t].n == 24 and st[t].nonfinite == (2 if t == 5 else 0)
        assert st[t].mean == pytest.approx(row.mean(), rel=1e-12, abs=1e-15)
        assert st[t].mad == pytest.approx(np.abs(row - row.mean()).mean(), rel=1e-12)
        assert st[t].var == pytest.approx(row.var(), rel=1e-12)
        assert (st[t].min, st[t].max) == (row.min(), row.max())
    # the tokens of X are the channels of its transpose: statistics, quantizers, codes and reconstructions
    # must be those of the (separately pinned) channel-wise functions on the transposed tensor
    xt = np.ascontiguousarray(x.T)                           # [24, 37]: 37 channels
    st_c = oracle.stats_channels(xt, 37)
    assert all(bytes(st[t]) == bytes(st_c[t]) for t in range(37))
    for bits, method, cut, mid in ((4, oracle.CLIP_ACIQ, False, False), (2, oracle.CLIP_MINMAX, False, True),
                                   (8, oracle.CLIP_ACIQ, True, False)):
        rc, qp = oracle.clip_tokens(st, bits, method, cut, midrise=mid)
        rc_c, qp_c = oracle.clip_channels(st_c, bits, method, cut, midrise=mid)
        assert rc == rc_c and all(bytes(qp[t]) == bytes(qp_c[t]) for t in range(37))
        codes = oracle.quantize_tokens(x, 24, qp).reshape(37, 24)
        codes_c = oracle.quantize_channels(xt, 37, qp_c).reshape(24, 37)
        assert np.array_equal(codes, codes_c.T)
        y = oracle.dequantize_tokens(codes.reshape(-1), 24, qp).reshape(37, 24)
        y_c = oracle.dequantize_channels(codes_c.reshape(-1), 37, qp_c).reshape(24, 37)
        assert np.array_equal(y, y_c.T)


def test_tokens_one_token_is_the_per_tensor_path_and_tokens_do_not_interact():
    y = si.flat_iid(5000, 17, "laplace")
    st1 = oracle.stats_tokens(y, y.size)                     # a single token: exactly the per-tensor functions
    assert bytes(st1[0]) == bytes(oracle.stats(y))
    for bits in (2, 4, 8, 16):
        rc, qp1 = oracle.clip_tokens(st1, bits)
        q = oracle.aciq_alpha(oracle.stats(y), bits)[2]
        assert bytes(qp1[0]) == bytes(q)
        assert np.array_equal(oracle.quantize_tokens(y, y.size, qp1), oracle.quantize(y, q))
        assert np.array_equal(oracle.pack(oracle.quantize_tokens(y, y.size, qp1), bits), oracle.quantize_pack(y, q))
    x = si.vit_activation((1, 30, 16), 18, outlier_frac=0.2).reshape(30, 16)
    st = oracle.stats_tokens(x, 16)
    rc, qp = oracle.clip_tokens(st, 4)
    codes = oracle.quantize_tokens(x, 16, qp).reshape(30, 16)
    x2 = x.copy()
    x2[11] *= np.float32(4.0)                                # a power of two: token 11's range scales, nothing else moves
    st2 = oracle.stats_tokens(x2, 16)
    rc, qp2 = oracle.clip_tokens(st2, 4)
    assert (qp2[11].lo, qp2[11].hi, qp2[11].scale) == (4 * qp[11].lo, 4 * qp[11].hi, 4 * qp[11].scale)
    assert all(bytes(qp2[t]) == bytes(qp[t]) for t in range(30) if t != 11)
    assert np.array_equal(oracle.quantize_tokens(x2, 16, qp2).reshape(30, 16), codes)
    x[7] = np.float32(-2.5)                                  # a constant token is degenerate: code 0, exact
    rc, qz = oracle.clip_tokens(oracle.stats_tokens(x, 16), 4)
    assert rc == oracle.WARN_DEGENERATE and qz[7].flags == 1
    back = oracle.dequantize_tokens(oracle.quantize_tokens(x, 16, qz), 16, qz).reshape(30, 16)
    assert np.all(back[7] == np.float32(-2.5))
