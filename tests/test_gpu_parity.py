"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.

Tolerances (the targets this library is built to):
  statistics      1e-5 relative   (mean: relative to max(|mean|, mad), since the mean of a
                                   centred tensor is near zero)
  clipping value  1e-4 relative, or the oracle's MSE at the GPU's step within 1e-6 of the
                  minimum (two steps of the search can tie to that level); every candidate's
                  error within 2e-6 of the oracle's error for the same quantizer
  packed codes    bit-exact given the same clip range and scale
  dequantized     1e-6 absolute
"""
import ctypes
import numpy as np
import pytest
import torch

import oracle
import oracle_par
import paper_2211_04515_b200 as qp
import synth_inputs as si

pytestmark = pytest.mark.gpu

ALL_BITS = [1, 2, 3, 4, 5, 6, 7, 8, 16]
RAGGED = [1, 7, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 4099, 100003]


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available()
    c = qp.Context(0)
    yield c
    assert c.qp_get_status() >= 0
    c.close()


def to_qp(o):
    return qp.QParams(o.lo, o.hi, o.scale, o.inv_scale, o.bits, o.flags)


def dev(x_np):
    return torch.from_numpy(np.ascontiguousarray(x_np)).cuda()


def guarded(nbytes, fill=0xA5, guard=256):
    """Device byte buffer with canaries on both sides; returns (whole, view)."""
    whole = torch.full((nbytes + 2 * guard,), fill, dtype=torch.uint8, device="cuda")
    return whole, whole[guard:guard + nbytes]


def canaries_intact(whole, nbytes, fill=0xA5, guard=256):
    h = whole.cpu().numpy()
    return (h[:guard] == fill).all() and (h[guard + nbytes:] == fill).all()


def check_stats(st, st_o):
    assert st.n == st_o.n and st.nonfinite == st_o.nonfinite
    assert st.min == st_o.min and st.max == st_o.max
    assert abs(st.mean - st_o.mean) <= 1e-5 * max(abs(st_o.mean), st_o.mad)
    for f in ("mean_abs", "mad", "var"):
        a, b = getattr(st, f), getattr(st_o, f)
        assert abs(a - b) <= 1e-5 * abs(b), (f, a, b)


# ------------------------------------------------------------------ statistics

STATS_PATHS = [qp.QP_STATS_FUSED, qp.QP_STATS_TWO_KERNELS]     # one cooperative launch / one kernel per pass


@pytest.fixture(params=STATS_PATHS, ids=["fused", "two_kernels"])
def sctx(ctx, request):
    """The module's context with the statistics forced down one of their two paths."""
    ctx.qp_set_stats_path(request.param)
    yield ctx
    ctx.qp_set_stats_path(qp.QP_STATS_AUTO)


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_stats_configs(sctx, name):
    ctx = sctx
    x = si.config_tensor(name).reshape(-1)
    st = ctx.read_stats(ctx.qp_stats(dev(x)))
    st_o = oracle.stats(x)
    check_stats(st, st_o)
    assert st.hist_bins == 0
    # bit-reproducible: fixed merge order
    st2 = ctx.read_stats(ctx.qp_stats(dev(x)))
    assert bytes(st) == bytes(st2)
    # histogram carried along by the second pass: integer-identical peak count
    for nb in (100, 7, 2048, 4096):
        sth = ctx.read_stats(ctx.qp_stats(dev(x), hist_bins=nb))
        _, counts = oracle.hist_peak(x, st_o.min, st_o.max, nb)
        assert sth.hist_bins == nb and sth.hist_peak == int(counts.max())
        assert (sth.mean, sth.mad, sth.var) == (st.mean, st.mad, st.var)
    assert ctx.read_stats(ctx.qp_stats(dev(x), hist_bins=8192)).hist_bins == 0      # too many bins to fuse
    xs = dev(x)[1:]                                                                  # not 16-byte aligned: not fused
    assert ctx.read_stats(ctx.qp_stats(xs, hist_bins=100)).hist_bins == 0
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_stats(dev(x), hist_bins=-1)


@pytest.mark.parametrize("n", RAGGED + [262144 + 5])
def test_stats_ragged_and_misaligned(sctx, n):
    ctx = sctx
    x = si.vit_activation((1, n + 3, 1), 40 + n % 7).reshape(-1) * 3.0 + 0.25
    x = x.astype(np.float32)
    d = dev(x)
    for off in (0, 1, 3):
        st = ctx.read_stats(ctx.qp_stats(d[off:off + n]))
        check_stats(st, oracle.stats(x[off:off + n]))


def test_stats_special(sctx):
    ctx = sctx
    st = ctx.read_stats(ctx.qp_stats(torch.empty(0, device="cuda")))
    assert (st.n, st.nonfinite, st.mean, st.mad, st.min, st.max) == (0, 0, 0.0, 0.0, 0.0, 0.0)
    x = si.flat_iid(50000, 9, "laplace")
    x[[5, 777, 49999]] = [np.nan, np.inf, -np.inf]
    st = ctx.read_stats(ctx.qp_stats(dev(x)))
    check_stats(st, oracle.stats(x))
    assert st.nonfinite == 3
    assert ctx.qp_get_status() & qp.QP_DEV_NONFINITE
    xl = si.flat_iid(300000, 9, "laplace")
    xl[[5, 777, 299999]] = [np.nan, np.inf, -np.inf]
    stl = ctx.read_stats(ctx.qp_stats(dev(xl), hist_bins=64))
    sto = oracle.stats(xl)
    check_stats(stl, sto)
    assert stl.hist_peak == int(oracle.hist_peak(xl, sto.min, sto.max, 64)[1].max())
    ctx.qp_get_status()
    c = np.full(3000, -1.5, dtype=np.float32)
    st = ctx.read_stats(ctx.qp_stats(dev(c)))
    assert (st.mean, st.mad, st.var, st.min, st.max) == (-1.5, 0.0, 0.0, -1.5, -1.5)
    big = (np.float32(4096.0) + si.flat_iid(300000, 3, "normal")).astype(np.float32)     # mean >> spread
    check_stats(ctx.read_stats(ctx.qp_stats(dev(big))), oracle.stats(big))
    allbad = np.full(100, np.nan, dtype=np.float32)
    st = ctx.read_stats(ctx.qp_stats(dev(allbad)))
    assert st.nonfinite == 100 and st.mean == 0.0 and st.mad == 0.0
    ctx.qp_get_status()


def test_stats_bf16(sctx):
    ctx = sctx
    x = si.vit_activation((8, 197, 96), 12).reshape(-1)
    h = si.to_bf16_bits(x)
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    for off, n in ((0, h.size), (3, h.size - 11), (1, 77), (8, h.size - 8)):
        st = ctx.read_stats(ctx.qp_stats(d[off:off + n]))
        check_stats(st, oracle.stats(oracle.widen_bf16(h[off:off + n])))


# tiles of the one-launch statistics are 32 KB = 8192 fp32 elements; a B200 has 148 SMs and every block
# keeps 6 tiles resident: fewer tiles than blocks, one per block, a few per block (all resident), more than
# stay resident, and ragged tails behind the last whole tile
@pytest.mark.parametrize("tiles,tail", [(4, 0), (5, 777), (147, 1), (148, 0), (149, 8191), (6 * 148, 5), (6 * 148 + 1, 0),
                                         (7 * 148 + 75, 33), (13 * 148 + 3, 4099)])
def test_stats_one_launch_against_oracle_and_two_kernels(ctx, tiles, tail):
    n = tiles * 8192 + tail
    x = si.vit_activation((1, n, 1), 200 + tiles % 11).reshape(-1) * np.float32(1.5) - np.float32(0.75)
    d = dev(x)
    st_o = oracle.stats(x)
    _, counts = oracle.hist_peak(x, st_o.min, st_o.max, 100)
    got = {}
    for path in STATS_PATHS:
        ctx.qp_set_stats_path(path)
        try:
            before = ctx.qp_launch_count()
            st = ctx.read_stats(ctx.qp_stats(d, hist_bins=100))
            launches = ctx.qp_launch_count() - before
            again = ctx.read_stats(ctx.qp_stats(d, hist_bins=100))
            plain = ctx.read_stats(ctx.qp_stats(d))
        finally:
            ctx.qp_set_stats_path(qp.QP_STATS_AUTO)
        assert launches == (2 if path == qp.QP_STATS_TWO_KERNELS else 1)
        check_stats(st, st_o)
        assert st.hist_bins == 100 and st.hist_peak == int(counts.max())
        assert bytes(st) == bytes(again)                              # fixed merge order: bit-reproducible
        assert plain.hist_bins == 0 and (plain.mean, plain.mad, plain.var) == (st.mean, st.mad, st.var)
        got[path] = st
    a, b = got[qp.QP_STATS_FUSED], got[qp.QP_STATS_TWO_KERNELS]
    assert (a.n, a.nonfinite, a.min, a.max, a.hist_peak) == (b.n, b.nonfinite, b.min, b.max, b.hist_peak)
    for f in ("mean_abs", "mad", "var"):         # fp32 sums over 16 elements, grouped differently by the two tile sizes
        assert abs(getattr(a, f) - getattr(b, f)) <= 1e-7 * abs(getattr(b, f))
    assert ctx.qp_get_status() == 0


def test_stats_hard_tensors(sctx):
    """Tensors that are hard on a streaming reduction: sorted (every block sees another level), a third
    of the elements exactly at the mean, constant, two levels, a shifted mixture, a mean far from zero,
    a tiny scale."""
    ctx = sctx
    n = 1500 * 8192 + 77
    base = si.flat_iid(n, 77, "laplace")
    cases = {
        "sorted": np.sort(base),
        "mass_at_mean": np.where(np.arange(n) % 3 == 0, np.float32(0.0),            # 0, +a, -a, 0, +b, -b, ...: mean exactly 0
                                 np.where(np.arange(n) % 3 == 1, 1.0, -1.0) * np.abs(np.repeat(base[:n // 3 + 1], 3)[:n])
                                 ).astype(np.float32),
        "constant": np.full(n, 3.25, dtype=np.float32),
        "two_levels": np.where(np.arange(n) % 2 == 0, np.float32(-1.0), np.float32(2.0)).astype(np.float32),
        "mixture": (base + np.where(np.arange(n) % 5 == 0, 40.0, 0.0)).astype(np.float32),
        "large_offset": (np.float32(4096.0) + base).astype(np.float32),
        "tiny_scale": (base * np.float32(1e-20)).astype(np.float32),
    }
    for name, x in cases.items():
        st = ctx.read_stats(ctx.qp_stats(dev(x)))
        st_o = oracle.stats(x)
        assert (st.min, st.max, st.n) == (st_o.min, st_o.max, st_o.n), name
        if st_o.mad > 0:
            check_stats(st, st_o)
        else:
            assert st.mad == 0.0 and st.var == 0.0 and st.mean == st_o.mean, name
    assert ctx.qp_get_status() == 0


# ------------------------------------------------------------- quantize + pack

def run_pack_unpack(ctx, x_np, d_x, qp_o, bits, out_bf16=False):
    n = x_np.size
    qp_h = to_qp(qp_o)
    nbytes = qp.qp_packed_bytes(n, bits)
    whole, view = guarded(nbytes)
    ctx.qp_quantize_pack(d_x, bits, qp_h, out=view)
    ref = oracle.quantize_pack(x_np, qp_o)
    got = view.cpu().numpy()
    assert got.size == ref.size
    assert np.array_equal(got, ref), f"bits={bits} n={n}: first diff at byte {np.flatnonzero(got != ref)[:4]}"
    assert canaries_intact(whole, nbytes)
    # receiver
    ywhole, yview = guarded(4 * n)
    y = yview.view(torch.float32)
    ctx.qp_unpack_dequantize(view, n, bits, qp_h, out=y)
    y_o = oracle.unpack_dequantize(ref, n, qp_o)
    if n:
        assert np.max(np.abs(y.cpu().numpy().astype(np.float64) - y_o.astype(np.float64))) <= 1e-6
    assert canaries_intact(ywhole, 4 * n)
    # output that is only 4-byte aligned: the scalar path must give the same values
    if n in (33, 1025, 4099):
        zwhole, zview = guarded(4 * (n + 1))
        z = zview[4:].view(torch.float32)
        ctx.qp_unpack_dequantize(view, n, bits, qp_h, out=z)
        assert torch.equal(z, y) and canaries_intact(zwhole, 4 * (n + 1))
        assert (zview[:4].cpu().numpy() == 0xA5).all()
    return view


@pytest.mark.parametrize("bits", ALL_BITS)
def test_pack_unpack_c1(ctx, bits):
    x = si.config_tensor("c1").reshape(-1)
    st = oracle.stats(x)
    _, _, qp_o = oracle.aciq_alpha(st, bits)
    run_pack_unpack(ctx, x, dev(x), qp_o, bits)
    # naive min/max range (Sec. 3, naive PTQ) through the same kernels
    _, qp_n = oracle.make_qparams(st.min, st.max, bits)
    run_pack_unpack(ctx, x, dev(x), qp_n, bits)


@pytest.mark.parametrize("bits", ALL_BITS)
def test_pack_unpack_ragged_and_misaligned(ctx, bits):
    base = si.vit_activation((1, 1, 110000), 17).reshape(-1)
    d = dev(base)
    st = oracle.stats(base)
    _, _, qp_o = oracle.aciq_alpha(st, bits)
    for n in RAGGED:
        for off in (0, 1) if n > 1024 or n in (33, 1023) else (0,):
            run_pack_unpack(ctx, base[off:off + n], d[off:off + n], qp_o, bits)


@pytest.mark.parametrize("bits", [1, 3, 4, 8, 16])
def test_pack_special_values_and_degenerate(ctx, bits):
    x = si.flat_iid(5000, 23, "normal")
    x[[0, 1, 2, 3, 4097, 4999]] = [np.nan, np.inf, -np.inf, -0.0, np.nan, 1e38]
    _, qp_o = oracle.make_qparams(-1.75, 2.25, bits)
    run_pack_unpack(ctx, x, dev(x), qp_o, bits)
    rc, qp_d = oracle.make_qparams(0.5, 0.5, bits)
    assert rc == oracle.WARN_DEGENERATE
    packed = run_pack_unpack(ctx, x, dev(x), qp_d, bits)
    assert not packed.cpu().numpy().any()
    # exact ties: positions k + 0.5 must round to the even level
    L1 = 2 ** bits - 1
    ties = (np.arange(min(L1, 4096), dtype=np.float32) + np.float32(0.5))
    _, qp_t = oracle.make_qparams(0.0, float(L1), bits)
    assert qp_t.scale == 1.0 and qp_t.inv_scale == 1.0
    run_pack_unpack(ctx, ties, dev(ties), qp_t, bits)


@pytest.mark.parametrize("bits", [2, 5, 8, 16])
def test_pack_bf16_input_and_output(ctx, bits):
    x = si.vit_activation((3, 197, 64), 31).reshape(-1)
    h = si.to_bf16_bits(x)
    xw = oracle.widen_bf16(h)
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    _, _, qp_o = oracle.aciq_alpha(oracle.stats(xw), bits)
    for off, n in ((0, h.size), (0, 8 * 1024 + 5), (1, 2049)):
        packed = ctx.qp_quantize_pack(d[off:off + n], bits, to_qp(qp_o))
        ref = oracle.quantize_pack(xw[off:off + n], qp_o)
        assert np.array_equal(packed.cpu().numpy(), ref)
        y = ctx.qp_unpack_dequantize(packed, n, bits, to_qp(qp_o), out_dtype=torch.bfloat16)
        y_o = si.to_bf16_bits(oracle.unpack_dequantize(ref, n, qp_o))
        assert np.array_equal(y.view(torch.int16).cpu().numpy().view(np.uint16), y_o)


def test_pack_argument_errors(ctx):
    x = torch.zeros(1000, device="cuda")
    _, qp_h = qp.qp_make_qparams(-1.0, 1.0, 4)
    with pytest.raises(qp.QuantPipeError) as e:
        ctx.qp_quantize_pack(x, 4, qp_h, out=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == qp.QP_ERR_BUFFER_TOO_SMALL
    with pytest.raises(qp.QuantPipeError) as e:
        ctx.qp_quantize_pack(x, 9, qp_h)
    assert e.value.status == qp.QP_ERR_UNSUPPORTED_BITS
    with pytest.raises(qp.QuantPipeError) as e:
        ctx.qp_quantize_pack(x, 8, qp_h)                       # quantizer made for 4 bits
    assert e.value.status == qp.QP_ERR_INVALID_ARG
    with pytest.raises(qp.QuantPipeError) as e:
        ctx.qp_quantize_pack(x, 4, qp_h, out=torch.empty(1024, dtype=torch.uint8, device="cuda")[1:])
    assert e.value.status == qp.QP_ERR_ALIGNMENT
    with pytest.raises(qp.QuantPipeError) as e:
        ctx.qp_quantize_pack(x.double(), 4, qp_h)
    assert e.value.status == qp.QP_ERR_UNSUPPORTED_DTYPE
    assert ctx.qp_quantize_pack(x[:0], 4, qp_h).numel() == 0
    # device-resident quantizer with other bits than the call: flagged in the status word
    d_qp = torch.from_numpy(np.frombuffer(bytes(qp_h), dtype=np.uint8).copy()).cuda()
    ctx.qp_get_status()
    ctx.qp_quantize_pack(x, 2, d_qp)
    assert ctx.qp_get_status() & qp.QP_DEV_BITS_MISMATCH


# ------------------------------------------------------------ ACIQ on device

@pytest.mark.parametrize("bits", ALL_BITS)
def test_aciq_device_chain(ctx, bits):
    """stats -> clip -> quantize with no host round trip; equals the oracle's chain."""
    x = si.config_tensor("c1").reshape(-1)
    d = dev(x)
    d_stats = ctx.qp_stats(d)
    st_o = oracle.stats(x)
    for dist, bmode in ((0, 0), (0, 1), (1, 0)):
        d_qp = ctx.qp_aciq_qparams_device(d_stats, bits, dist, bmode)
        got = ctx.read_qparams(d_qp)
        _, alpha_o, qp_o = oracle.aciq_alpha(st_o, bits, dist, bmode)
        assert got.bits == bits and got.flags == 0
        alpha_g = 0.5 * (float(got.hi) - float(got.lo))
        assert abs(alpha_g - alpha_o) <= 1e-4 * alpha_o
        assert abs(got.lo - qp_o.lo) <= 1e-5 * alpha_o and abs(got.hi - qp_o.hi) <= 1e-5 * alpha_o
    d_qp = ctx.qp_aciq_qparams_device(d_stats, bits)
    got = ctx.read_qparams(d_qp)
    packed = ctx.qp_quantize_pack(d, bits, d_qp)
    o = oracle.QParams(got.lo, got.hi, got.scale, got.inv_scale, got.bits, got.flags)
    assert np.array_equal(packed.cpu().numpy(), oracle.quantize_pack(x, o))
    y = ctx.qp_unpack_dequantize(packed, x.size, bits, d_qp)
    assert np.max(np.abs(y.cpu().numpy() - oracle.unpack_dequantize(packed.cpu().numpy(), x.size, o))) <= 1e-6


# ------------------------------------------------------------ directed search

BOTH_PATHS = [qp.QP_SEARCH_CANDIDATES, qp.QP_SEARCH_INTERVALS, qp.QP_SEARCH_INTERVALS_PLAIN]


CURVE_RTOL = 2e-6        # a candidate's error against the oracle's error for the same quantizer
TIE_RTOL = 1e-6          # two steps whose errors differ by less are both right (reading A5)
ALPHA_RTOL = 1e-4        # the chosen clipping value


def oracle_candidate_ends(st_o, res_o, bits, bmode, steps, k):
    """Clip range of step k as the oracle's search forms it: (lo, hi, alpha)."""
    gauss, midrise = bool(bmode & qp.QP_B_GAUSS), bool(bmode & qp.QP_B_MIDRISE)
    alpha = oracle.aciq_F(bits, 1 if gauss else 0) * (res_o.b_e + k * (res_o.b_r - res_o.b_e) / steps)
    lo, hi = st_o.mean - alpha, st_o.mean + alpha
    if midrise:
        lo, hi = oracle.midrise_range(lo, hi, bits)
    return lo, hi, alpha


def as_oracle_qp(c):
    return oracle.QParams(c.lo, c.hi, c.scale, c.inv_scale, c.bits, c.flags)


def check_candidates_and_pick(x_np, st_o, res_o, curve_o, res, curve, cand, bits, bmode, steps, exact_steps=None,
                              strict_winner=False):
    """The search's result against the oracle, step by step.

    The clip ends are fp32.  Two correct implementations whose statistics differ in the last
    bits can round an end to neighbouring floats, and for a tensor whose mean is far from zero
    one such ulp moves a candidate's error by far more than the error tolerance.  So the curve
    is compared where it is well defined: the library reports the quantizer of every candidate
    (qp_dsaciq_candidates), each is checked against the oracle's own clip range for that step
    (an fp32 ulp, or 1e-5 of the clipping value), and the oracle scores exactly those
    quantizers (orc_quant_mse).  Against that curve the library's errors must agree to 2e-6 and
    its winner must be the first minimum or tie with it to 1e-6; the winning clipping value
    must be the oracle's for that step to 1e-4.  exact_steps: score only these steps that way
    (full-size tensors) and compare the others with the oracle's own curve."""
    fin = np.isfinite(curve_o)
    assert np.array_equal(np.isfinite(curve), fin)
    ks = [int(k) for k in np.flatnonzero(fin)]
    for k in ks:
        lo_o, hi_o, alpha = oracle_candidate_ends(st_o, res_o, bits, bmode, steps, k)
        ulp = float(np.spacing(np.float32(max(abs(lo_o), abs(hi_o)))))
        tol = max(1e-5 * alpha, ulp) + 1e-30
        assert abs(cand[k].lo - lo_o) <= tol and abs(cand[k].hi - hi_o) <= tol, (k, cand[k].lo, lo_o, cand[k].hi, hi_o)
        _, again = oracle.make_qparams(cand[k].lo, cand[k].hi, bits)      # scale and reciprocal follow from the ends
        assert (again.scale, again.inv_scale, again.flags) == (cand[k].scale, cand[k].inv_scale, cand[k].flags), k
    scored = ks if exact_steps is None else sorted(set(k for k in exact_steps if k in ks) | {res.k_star, 0})
    exact = dict(zip(scored, oracle_par.run_all([(lambda k=k: oracle.quant_mse(x_np, as_oracle_qp(cand[k]))) for k in scored],
                                                parallel=x_np.size >= 100000)))
    for k in ks:
        want = exact.get(k, curve_o[k])
        assert abs(curve[k] - want) <= CURVE_RTOL * want + 1e-300, (k, curve[k], want, k in exact)
    ref = np.array([exact.get(k, curve_o[k]) if fin[k] else np.inf for k in range(steps + 1)])
    k_ref = int(np.argmin(ref))                                        # first minimum
    assert res.k_star == k_ref or ref[res.k_star] <= ref[k_ref] * (1 + TIE_RTOL), (res.k_star, k_ref)
    _, _, alpha_k = oracle_candidate_ends(st_o, res_o, bits, bmode, steps, res.k_star)
    assert abs(res.alpha_star - alpha_k) <= ALPHA_RTOL * abs(alpha_k) + 1e-300
    if strict_winner:                                                  # the benchmark's configurations: no tie escape
        assert res.k_star == res_o.k_star, (res.k_star, res_o.k_star)
        assert abs(res.alpha_star - res_o.alpha_star) <= ALPHA_RTOL * abs(res_o.alpha_star)


def check_search(ctx, x_np, d_x, bits, bmode=0, steps=100, nb=100, path=qp.QP_SEARCH_AUTO, exact_steps=None,
                 strict_winner=False, oracle_result=None):
    # statistics with the histogram carried along, except when the candidate-scoring path is
    # forced (then the search counts its own histogram): both ways are exercised
    d_stats = ctx.qp_stats(d_x, hist_bins=0 if path == qp.QP_SEARCH_CANDIDATES else nb)
    ctx.qp_set_search_path(path)
    try:
        d_res, d_qp = ctx.qp_dsaciq_search(d_x, d_stats, bits, bmode, steps, nb)
    finally:
        ctx.qp_set_search_path(qp.QP_SEARCH_AUTO)
    res, got_qp = ctx.read_ds_result(d_res), ctx.read_qparams(d_qp)
    curve = np.array(ctx.qp_dsaciq_curve(steps))
    cand = ctx.qp_dsaciq_candidates(steps)
    st_o = oracle.stats(x_np)
    rc_o, res_o, qp_o, curve_o = oracle_result if oracle_result is not None else oracle.ds_search(x_np, st_o, bits, bmode, steps, nb)
    assert (res.steps, res.hist_bins, res.bits) == (steps, nb, bits)
    assert abs(res.b_e - res_o.b_e) <= 1e-5 * abs(res_o.b_e) + 1e-300
    # the histogram counts are integers computed with the same fp32 expression; b_R can
    # differ only through the fp64 statistics it is scaled by
    assert abs(res.b_r - res_o.b_r) <= 1e-9 * abs(res_o.b_r) + 1e-300
    check_candidates_and_pick(x_np, st_o, res_o, curve_o, res, curve, cand, bits, bmode, steps, exact_steps, strict_winner)
    # the quantizer written for the packer is the winning candidate's
    w = cand[res.k_star]
    assert (got_qp.lo, got_qp.hi, got_qp.scale, got_qp.inv_scale, got_qp.bits) == (w.lo, w.hi, w.scale, w.inv_scale, bits)
    assert res.mse_star <= res.mse_e and res.mse_star == curve[res.k_star] and res.mse_e == curve[0]
    assert abs(res.alpha_e - res_o.alpha_e) <= 1e-5 * res_o.alpha_e + 1e-300
    return res, res_o


@pytest.mark.parametrize("path", BOTH_PATHS)
@pytest.mark.parametrize("bits", [1, 2, 3, 4, 5, 6, 7, 8])
def test_search_c1(ctx, bits, path):
    x = si.config_tensor("c1").reshape(-1)
    d = dev(x)
    check_search(ctx, x, d, bits, path=path)
    first = ctx.qp_dsaciq_curve(100)
    check_search(ctx, x, d, bits, path=path)
    assert ctx.qp_dsaciq_curve(100) == first          # fixed merge order / integer sums: bit-reproducible


@pytest.mark.parametrize("path", BOTH_PATHS)
@pytest.mark.parametrize("nb", [1, 64, 256, 2048, 16384])
def test_search_hist_bins_and_modes(ctx, nb, path):
    x = si.vit_activation((4, 197, 256), 2, outlier_frac=0.02).reshape(-1)
    d = dev(x)
    check_search(ctx, x, d, 2, nb=nb, path=path)
    check_search(ctx, x, d, 4, bmode=1, nb=nb, path=path)


@pytest.mark.parametrize("path", BOTH_PATHS)
@pytest.mark.parametrize("steps", [1, 7, 8, 9, 100, 250, 1023])
def test_search_steps(ctx, steps, path):
    x = si.vit_activation((1, 64, 192), 5).reshape(-1)
    check_search(ctx, x, dev(x), 3, steps=steps, path=path)    # 1023 steps: the interval tables do not fit, falls back
    check_search(ctx, x, dev(x), 1, steps=steps, path=path)


@pytest.mark.parametrize("path", BOTH_PATHS)
@pytest.mark.parametrize("n", [1, 5, 33, 1000, 4099, 100003])
def test_search_ragged_misaligned_nonfinite(ctx, n, path):
    x = si.vit_activation((1, n + 2, 1), 60 + n % 5).reshape(-1).astype(np.float32)
    d = dev(x)
    for off in (0, 1):
        if n > 1:
            check_search(ctx, x[off:off + n], d[off:off + n], 2, path=path)
    if n >= 1000:
        x[[3, n // 2]] = [np.nan, np.inf]
        check_search(ctx, x[:n], dev(x[:n]), 4, path=path)
        ctx.qp_get_status()


@pytest.mark.parametrize("path", BOTH_PATHS)
def test_search_large_offset_and_outliers(ctx, path):
    """Mean far from zero (few floats per grid cell) and heavy outliers on both sides."""
    # At |mean| = 4096 one fp32 ulp of a clip end is 4.9e-4, i.e. ~1e-4 of the clip width; the
    # oracle scores the library's own fp32 clip ends (check_candidates_and_pick), so the usual
    # tolerances hold here too.
    big = (np.float32(4096.0) + si.flat_iid(200000, 3, "normal")).astype(np.float32)
    check_search(ctx, big, dev(big), 2, path=path)
    check_search(ctx, big, dev(big), 4, nb=2048, path=path)
    x = si.vit_activation((2, 197, 512), 2, outlier_frac=0.03).reshape(-1)
    x[::1000] *= -50.0
    for bits in (1, 2, 3, 4):
        check_search(ctx, x, dev(x), bits, path=path)


def test_search_degenerate_and_errors(ctx):
    c = np.full(5000, 2.5, dtype=np.float32)
    d = dev(c)
    d_stats = ctx.qp_stats(d)
    for path in BOTH_PATHS:
        ctx.qp_set_search_path(path)
        d_res, d_qp = ctx.qp_dsaciq_search(d, d_stats, 2)
        res, q = ctx.read_ds_result(d_res), ctx.read_qparams(d_qp)
        assert res.k_star == 0 and res.b_star == 0.0 and res.mse_star == 0.0 and q.flags == 1
        assert ctx.qp_get_status() & qp.QP_DEV_DEGENERATE
        two = np.array([1.0, 1.0, 1.0, 3.0], dtype=np.float32)          # two distinct values
        check_search(ctx, two, dev(two), 2, path=path)
        ctx.qp_get_status()
    ctx.qp_set_search_path(qp.QP_SEARCH_AUTO)
    packed = ctx.qp_quantize_pack(d, 2, d_qp)
    assert not packed.cpu().numpy().any()
    assert np.array_equal(ctx.qp_unpack_dequantize(packed, c.size, 2, d_qp).cpu().numpy(), c)
    for bad in (dict(bits=16), dict(bits=0), dict(steps=0), dict(steps=1024), dict(hist_bins=0), dict(hist_bins=16385)):
        kw = dict(bits=2, steps=100, hist_bins=100)
        kw.update(bad)
        with pytest.raises(qp.QuantPipeError):
            ctx.qp_dsaciq_search(d, d_stats, kw["bits"], 0, kw["steps"], kw["hist_bins"])


@pytest.mark.parametrize("path", BOTH_PATHS)
@pytest.mark.parametrize("bits", [1, 2, 4, 6])
def test_search_midrise_grid(ctx, bits, path):
    """Every candidate on the mid-rise grid (bmode | QP_B_MIDRISE): same b_E, b_R and steps, other ranges."""
    x = si.config_tensor("c1").reshape(-1)
    res, res_o = check_search(ctx, x, dev(x), bits, bmode=qp.QP_B_MIDRISE, path=path)
    plain, _ = check_search(ctx, x, dev(x), bits, path=path)
    assert (res.b_e, res.b_r) == (plain.b_e, plain.b_r) and res.mse_e != plain.mse_e
    y = si.vit_activation((5, 197, 200), 55, outlier_frac=0.02).reshape(-1)
    check_search(ctx, y, dev(y), bits, bmode=qp.QP_B_MEAN_ABS | qp.QP_B_MIDRISE, path=path)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_dsaciq_search(dev(y), ctx.qp_stats(dev(y)), bits, 0x80)


@pytest.mark.parametrize("path", BOTH_PATHS)
@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_search_gaussian_model(ctx, bits, path):
    """QP_B_GAUSS: scale = standard deviation, sigma_R from the normal density's peak, F of the normal model."""
    x = si.config_tensor("c1").reshape(-1)
    res, res_o = check_search(ctx, x, dev(x), bits, bmode=qp.QP_B_GAUSS, path=path)
    plain, _ = check_search(ctx, x, dev(x), bits, path=path)
    st_o = oracle.stats(x)
    assert abs(res.b_e - np.sqrt(st_o.var)) <= 1e-5 * res.b_e
    assert abs(res.b_r / plain.b_r - 2.0 / np.sqrt(2.0 * np.pi)) <= 1e-9      # the same peak count, another model
    g = (0.3 + 0.7 * si.flat_iid(200003, 17, "normal")).astype(np.float32)     # normal data, ragged size
    check_search(ctx, g, dev(g), bits, bmode=qp.QP_B_GAUSS | qp.QP_B_MIDRISE, nb=256, path=path)
    with pytest.raises(qp.QuantPipeError):                                     # the printed formula has no normal form
        ctx.qp_dsaciq_search(dev(g), ctx.qp_stats(dev(g)), bits, qp.QP_B_MEAN_ABS | qp.QP_B_GAUSS)


@pytest.mark.parametrize("path", BOTH_PATHS)
def test_search_histogram_promise(ctx, path):
    """QP_B_HIST_IN_STATS: no histogram pass of its own, same result; a broken promise is reported."""
    x = si.vit_activation((8, 197, 256), 21).reshape(-1)              # 1.6 MB: the statistics carry the histogram
    d = dev(x)
    assert qp.qp_stats_carries_histogram(d, 100) and not qp.qp_stats_carries_histogram(d[1:], 100)
    assert not qp.qp_stats_carries_histogram(d, 8192) and not qp.qp_stats_carries_histogram(d[:1000], 100)
    ctx.qp_set_search_path(path)
    try:
        d_stats = ctx.qp_stats(d, hist_bins=100)
        n0 = ctx.qp_launch_count()
        d_res, d_qp = ctx.qp_dsaciq_search(d, d_stats, 2, qp.QP_B_MAD, 100, 100)
        n1 = ctx.qp_launch_count()
        d_res2, d_qp2 = ctx.qp_dsaciq_search(d, d_stats, 2, qp.QP_B_MAD | qp.QP_B_HIST_IN_STATS, 100, 100)
        n2 = ctx.qp_launch_count()
        assert bytes(ctx.read_ds_result(d_res)) == bytes(ctx.read_ds_result(d_res2))
        assert bytes(ctx.read_qparams(d_qp)) == bytes(ctx.read_qparams(d_qp2))
        assert (n1 - n0) - (n2 - n1) == 1                              # one launch fewer
        assert ctx.qp_get_status() == 0
        # statistics without the histogram, yet the promise: reported, and b_E is kept
        d_plain = ctx.qp_stats(d, hist_bins=0)
        d_res3, _ = ctx.qp_dsaciq_search(d, d_plain, 2, qp.QP_B_MAD | qp.QP_B_HIST_IN_STATS, 100, 100)
        res3 = ctx.read_ds_result(d_res3)
        assert ctx.qp_get_status() & qp.QP_DEV_HIST_MISSING
        assert res3.k_star == 0 and res3.b_star == res3.b_e
    finally:
        ctx.qp_set_search_path(qp.QP_SEARCH_AUTO)


@pytest.mark.parametrize("path", BOTH_PATHS)
def test_search_bf16(ctx, path):
    x = si.vit_activation((4, 197, 128), 8).reshape(-1)
    h = si.to_bf16_bits(x)
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    check_search(ctx, oracle.widen_bf16(h), d, 2, path=path)
    check_search(ctx, oracle.widen_bf16(h[1:-2]), d[1:-2], 4, path=path)


# ----------------------------------------------------------- whole-sender calls

@pytest.mark.parametrize("bits,use_ds", [(2, True), (4, True), (8, False), (16, False), (3, False)])
def test_sender_device_equals_separate_calls(ctx, bits, use_ds):
    x = si.vit_activation((6, 197, 256), 77).reshape(-1)
    d = dev(x)
    d_stats = ctx.qp_stats(d, hist_bins=100 if use_ds else 0)
    if use_ds:
        _, d_qp = ctx.qp_dsaciq_search(d, d_stats, bits)
    else:
        d_qp = ctx.qp_aciq_qparams_device(d_stats, bits)
    want = ctx.qp_quantize_pack(d, bits, d_qp)
    ctx.qp_set_sender_path(qp.QP_SENDER_CHAIN)               # the chain is bit for bit the separate calls
    try:
        got, got_qp = ctx.qp_sender_device(d, bits, use_ds)
    finally:
        ctx.qp_set_sender_path(qp.QP_SENDER_AUTO)
    assert torch.equal(got, want) and torch.equal(got_qp, d_qp)
    q = ctx.read_qparams(got_qp)
    o = oracle.QParams(q.lo, q.hi, q.scale, q.inv_scale, q.bits, q.flags)
    assert np.array_equal(got.cpu().numpy(), oracle.quantize_pack(x, o))


def check_fused_sender(x_np, d_x, bits, use_ds, bmode=0, steps=100, nb=100):
    """The single-launch sender against the oracle: statistics, clip (every candidate's error and the
    winner as in check_candidates_and_pick), and the packed stream bit for bit under the quantizer
    the kernel chose."""
    from types import SimpleNamespace
    c = qp.Context(0)
    try:
        c.qp_set_sender_path(qp.QP_SENDER_FUSED)
        n = x_np.size
        nbytes = qp.qp_packed_bytes(n, bits)
        whole, packed = guarded(nbytes)
        d_stats = torch.empty(ctypes.sizeof(qp.Stats), dtype=torch.uint8, device="cuda")
        before = c.qp_launch_count()
        _, d_qp = c.qp_sender_device(d_x, bits, use_ds, out_packed=packed, out_stats=d_stats, bmode=bmode, steps=steps,
                                     hist_bins=nb)
        torch.cuda.synchronize()
        assert c.qp_launch_count() - before == 1                      # one kernel did all of it
        assert canaries_intact(whole, nbytes)
        st, st_o = c.read_stats(d_stats), oracle.stats(x_np)
        check_stats(st, st_o)
        got = c.read_qparams(d_qp)
        assert got.bits == bits
        if use_ds:
            assert st.hist_bins == nb
            rc_o, res_o, qp_o, curve_o = oracle.ds_search(x_np, st_o, bits, bmode, steps, nb)
            curve = np.array(c.qp_dsaciq_curve(steps))
            cand = c.qp_dsaciq_candidates(steps)
            # the one launch reports no result record: the winner is the candidate it wrote as quantizer
            hits = [k for k in range(steps + 1) if np.isfinite(curve[k]) and (cand[k].lo, cand[k].hi) == (got.lo, got.hi)]
            assert hits
            res = SimpleNamespace(k_star=hits[0], alpha_star=0.5 * (float(got.hi) - float(got.lo)))
            check_candidates_and_pick(x_np, st_o, res_o, curve_o, res, curve, cand, bits, bmode, steps)
        else:
            rc_o, alpha_o, qp_o = oracle.aciq_alpha(st_o, bits, 0, bmode, 0.0)
            assert abs(got.lo - qp_o.lo) <= 1e-5 * alpha_o + 1e-30 and abs(got.hi - qp_o.hi) <= 1e-5 * alpha_o + 1e-30
        rc2, again = oracle.make_qparams(got.lo, got.hi, bits)        # scale and reciprocal follow from the ends
        assert (again.scale, again.inv_scale, again.flags) == (got.scale, got.inv_scale, got.flags)
        o = oracle.QParams(got.lo, got.hi, got.scale, got.inv_scale, got.bits, got.flags)
        assert np.array_equal(packed.cpu().numpy(), oracle.quantize_pack(x_np, o))
        return c.qp_get_status(), got
    finally:
        c.close()


@pytest.mark.parametrize("bits,use_ds", [(1, True), (2, True), (3, True), (4, True), (8, True), (3, False), (5, False),
                                         (6, False), (8, False), (16, False)])
def test_fused_sender_c1(bits, use_ds):
    x = si.config_tensor("c1").reshape(-1)
    status, _ = check_fused_sender(x, dev(x), bits, use_ds)
    assert status == 0


@pytest.mark.parametrize("n", RAGGED + [151297, (1 << 20) - 5, 1 << 20])
def test_fused_sender_ragged_and_misaligned(n):
    x = si.vit_activation((1, n + 2, 1), 30 + n % 7).reshape(-1).astype(np.float32)
    d = dev(x)
    for off, bits, use_ds in ((0, 2, True), (1, 3, False), (1, 4, True), (0, 16, False), (0, 1, False)):
        if n == 1 and use_ds:
            continue                                                  # one element: nothing to search
        status, _ = check_fused_sender(x[off:off + n], d[off:off + n], bits, use_ds)
        assert status & ~qp.QP_DEV_DEGENERATE == 0


def test_fused_sender_special_values_modes_and_bf16():
    x = si.vit_activation((3, 197, 200), 31, outlier_frac=0.02).reshape(-1)
    x[[0, 77, x.size - 1]] = [np.nan, np.inf, -np.inf]
    for bits, use_ds in ((2, True), (8, False)):
        status, _ = check_fused_sender(x, dev(x), bits, use_ds)
        assert status == qp.QP_DEV_NONFINITE
    x = si.vit_activation((2, 197, 160), 32).reshape(-1)
    check_fused_sender(x, dev(x), 4, True, bmode=1, steps=127, nb=4096)
    check_fused_sender(x, dev(x), 2, True, steps=1, nb=1)
    check_fused_sender(x, dev(x), 6, False, bmode=1)
    const = np.full(3000, -1.25, dtype=np.float32)                    # no spread: code 0 everywhere
    for use_ds in (True, False):
        status, got = check_fused_sender(const, dev(const), 2, use_ds)
        assert status == qp.QP_DEV_DEGENERATE and got.flags == 1
    h = si.to_bf16_bits(x)
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    check_fused_sender(oracle.widen_bf16(h), d, 2, True)
    check_fused_sender(oracle.widen_bf16(h[1:-2]), d[1:-2], 8, False)


def test_fused_sender_range_and_fallback():
    """Forced, the single launch takes a closed-form clip up to what shared memory holds (millions of
    elements) and the search up to 2^20; beyond that, or beyond 127 steps or 4096 bins, the call runs the
    kernel chain.  AUTO switches to the chain earlier (2^21), where the chain is the faster one."""
    c = qp.Context(0)
    x = si.vit_activation((1, 3000000, 1), 33).reshape(-1)
    d = dev(x)
    c.qp_set_sender_path(qp.QP_SENDER_FUSED)
    status, _ = check_fused_sender(x, d, 8, False)                     # 3 M elements, one launch
    assert status == 0
    big = torch.zeros(7000000, device="cuda")
    for t, use_ds, want_one in ((big, False, False), (d[:(1 << 20) + 1], True, False), (d[:1 << 20], True, True),
                                (d[:5000], True, True)):
        before = c.qp_launch_count()
        c.qp_sender_device(t, 2, use_ds)
        assert (c.qp_launch_count() - before == 1) == want_one
    for kw in (dict(steps=128), dict(hist_bins=4097)):
        before = c.qp_launch_count()
        c.qp_sender_device(d[:5000], 2, True, **kw)
        assert c.qp_launch_count() - before > 1
    c.qp_set_sender_path(qp.QP_SENDER_AUTO)
    for n, want_one in ((1 << 21, True), ((1 << 21) + 1, False)):
        before = c.qp_launch_count()
        c.qp_sender_device(d[:n], 8, False)
        assert (c.qp_launch_count() - before == 1) == want_one
    with pytest.raises(qp.QuantPipeError):
        c.qp_set_sender_path(3)
    assert c.qp_get_status() & ~qp.QP_DEV_DEGENERATE == 0              # (the all-zero tensor has no spread)
    c.close()


# clip methods of the sender: ACIQ, ACIQ cut back to the data range, naive PTQ's min/max
CLIP_CASES = [(qp.QP_CLIP_ACIQ, oracle.CLIP_ACIQ, False), (qp.QP_CLIP_ACIQ | qp.QP_CLIP_INTERSECT, oracle.CLIP_ACIQ, True),
              (qp.QP_CLIP_MINMAX, oracle.CLIP_MINMAX, False), (qp.QP_CLIP_ACIQ | qp.QP_CLIP_MIDRISE, oracle.CLIP_ACIQ, False),
              (qp.QP_CLIP_MINMAX | qp.QP_CLIP_MIDRISE, oracle.CLIP_MINMAX, False),
              (qp.QP_CLIP_ACIQ | qp.QP_CLIP_INTERSECT | qp.QP_CLIP_MIDRISE, oracle.CLIP_ACIQ, True)]


@pytest.mark.parametrize("method,o_method,cut", CLIP_CASES)
@pytest.mark.parametrize("path", [qp.QP_SENDER_CHAIN, qp.QP_SENDER_FUSED])
def test_sender_clip_methods(ctx, method, o_method, cut, path):
    x = si.vit_activation((3, 197, 192), 81, outlier_frac=0.01).reshape(-1)
    d = dev(x)
    st_o = oracle.stats(x)
    ctx.qp_set_sender_path(path)
    try:
        for bits in (2, 4, 8, 16):
            d_stats = torch.empty(ctypes.sizeof(qp.Stats), dtype=torch.uint8, device="cuda")
            packed, d_qp = ctx.qp_sender_device(d, bits, method, out_stats=d_stats)
            got = ctx.read_qparams(d_qp)
            rc_o, lo_o, hi_o, q_o = oracle.clip_range(st_o, bits, o_method, cut, midrise=bool(method & qp.QP_CLIP_MIDRISE))
            width = hi_o - lo_o
            assert abs(got.lo - q_o.lo) <= 1e-5 * width and abs(got.hi - q_o.hi) <= 1e-5 * width
            if method & 0xF == qp.QP_CLIP_MINMAX:               # min and max are exact, so is the quantizer
                assert bytes(got) == bytes(to_qp(q_o))
            o = oracle.QParams(got.lo, got.hi, got.scale, got.inv_scale, got.bits, got.flags)
            assert np.array_equal(packed.cpu().numpy(), oracle.quantize_pack(x, o))
            # the device form of the closed-form clip gives the same quantizer from the same statistics
            assert torch.equal(ctx.qp_clip_qparams_device(d_stats, bits, method), d_qp)
    finally:
        ctx.qp_set_sender_path(qp.QP_SENDER_AUTO)
    assert ctx.qp_get_status() == 0


@pytest.mark.parametrize("path", [qp.QP_SENDER_CHAIN, qp.QP_SENDER_FUSED])
def test_sender_search_on_midrise_grid(ctx, path):
    x = si.vit_activation((3, 197, 192), 82, outlier_frac=0.01).reshape(-1)
    d = dev(x)
    st_o = oracle.stats(x)
    ctx.qp_set_sender_path(path)
    try:
        for bits in (2, 4):
            packed, d_qp = ctx.qp_sender_device(d, bits, qp.QP_CLIP_DSACIQ | qp.QP_CLIP_MIDRISE)
            got = ctx.read_qparams(d_qp)
            rc_o, res_o, qp_o, curve_o = oracle.ds_search(x, st_o, bits, oracle.B_MIDRISE)
            curve = np.array(ctx.qp_dsaciq_curve(100))
            assert np.all(np.abs(curve - curve_o) <= 2e-6 * curve_o)
            F = oracle.aciq_F(bits, 0)
            ok = False
            for k in np.flatnonzero(curve_o <= res_o.mse_star * (1 + 1e-6)):
                alpha = F * (res_o.b_e + k * (res_o.b_r - res_o.b_e) / 100)
                lo, hi = oracle.midrise_range(st_o.mean - alpha, st_o.mean + alpha, bits)
                ok = ok or (abs(got.lo - lo) <= 1e-5 * alpha and abs(got.hi - hi) <= 1e-5 * alpha)
            assert ok
            o = oracle.QParams(got.lo, got.hi, got.scale, got.inv_scale, got.bits, got.flags)
            assert np.array_equal(packed.cpu().numpy(), oracle.quantize_pack(x, o))
            plain = ctx.read_qparams(ctx.qp_sender_device(d, bits, qp.QP_CLIP_DSACIQ)[1])
            assert (plain.lo, plain.hi) != (got.lo, got.hi)
    finally:
        ctx.qp_set_sender_path(qp.QP_SENDER_AUTO)
    assert ctx.qp_get_status() == 0


def test_clip_method_errors(ctx):
    x = dev(si.flat_iid(4096, 5, "laplace"))
    d_stats = ctx.qp_stats(x)
    for bad in (qp.QP_CLIP_DSACIQ, 3, qp.QP_CLIP_MINMAX | qp.QP_CLIP_INTERSECT):
        with pytest.raises(qp.QuantPipeError):
            ctx.qp_clip_qparams_device(d_stats, 4, bad)
    for bad in (3, qp.QP_CLIP_DSACIQ | qp.QP_CLIP_INTERSECT, qp.QP_CLIP_MINMAX | qp.QP_CLIP_INTERSECT):
        with pytest.raises(qp.QuantPipeError):
            ctx.qp_sender_device(x, 4, bad)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_sender_device(x, 16, qp.QP_CLIP_DSACIQ)


def test_sender_and_receiver_host_buffers(ctx):
    x = si.vit_activation((2, 197, 384), 78).reshape(-1)
    n = x.size
    hx = torch.from_numpy(x).pin_memory()
    for bits, use_ds in ((2, True), (8, False)):
        nbytes = qp.qp_packed_bytes(n, bits)
        d_x, d_p = torch.empty(n, device="cuda"), torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        h_p = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
        h_qp = qp.QParams()
        ctx.qp_sender_host(hx, bits, use_ds, d_x, d_p, h_p, h_qp)
        torch.cuda.synchronize()
        want, want_qp = ctx.qp_sender_device(dev(x), bits, use_ds)
        assert np.array_equal(h_p.numpy(), want.cpu().numpy())
        assert bytes(h_qp) == bytes(ctx.read_qparams(want_qp))
        d_y, h_y = torch.empty(n, device="cuda"), torch.empty(n).pin_memory()
        ctx.qp_receiver_host(h_p, n, bits, h_qp, d_p, d_y, h_y)
        torch.cuda.synchronize()
        o = oracle.QParams(h_qp.lo, h_qp.hi, h_qp.scale, h_qp.inv_scale, h_qp.bits, h_qp.flags)
        y_o = oracle.unpack_dequantize(h_p.numpy(), n, o)
        assert np.max(np.abs(h_y.numpy().astype(np.float64) - y_o.astype(np.float64))) <= 1e-6


# ----------------------------------------------------- full-size configurations

def full_pack_unpack(ctx, x, d, qp_o, bits, label=""):
    """quantize+pack and unpack+dequantize of a whole large tensor: every packed byte and every
    reconstruction against the oracle (run chunk-wise on the host cores)."""
    qp_h = to_qp(qp_o)
    packed = ctx.qp_quantize_pack(d, bits, qp_h)
    y = ctx.qp_unpack_dequantize(packed, x.size, bits, qp_h)
    same, err = oracle_par.check_pack_unpack(x, qp_o, packed.cpu().numpy(), y.cpu().numpy())
    assert same, (label, bits, "packed bytes differ")
    assert err <= 1e-6, (label, bits, err)


@pytest.mark.parametrize("name", ["c2", "c3", "c4"])
def test_full_size_configs(ctx, name):
    """The benchmark configurations at full size: statistics, the search at every width where the
    paper switches it on (1..4 bits, in the launch configuration the benchmark times: histogram in
    the statistics, interval moments), and pack/unpack at every width 1..8 and 16, all element by
    element against the oracle."""
    x = si.config_tensor(name).reshape(-1)
    d = dev(x)
    st_o = oracle.stats(x)
    check_stats(ctx.read_stats(ctx.qp_stats(d)), st_o)
    ds_bits = [1, 2, 3, 4]
    # the oracle's searches (tens of seconds each at this size) side by side on the host cores
    searches = dict(zip(ds_bits, oracle_par.run_all([(lambda b=b: oracle.ds_search(x, st_o, b)) for b in ds_bits])))
    for bits in ds_bits:
        # every candidate against the oracle's curve; steps spread over the curve, the winner and its
        # neighbours also against the oracle's error for the library's own fp32 clip ends; same winner
        k_o = searches[bits][1].k_star
        check_search(ctx, x, d, bits, oracle_result=searches[bits], strict_winner=True,
                     exact_steps=[0, 25, 50, 75, 100, max(k_o - 1, 0), k_o, min(k_o + 1, 100)])
    if name == "c2":                                                # and the candidate-scoring kernel at full size
        check_search(ctx, x, d, 2, path=qp.QP_SEARCH_CANDIDATES, oracle_result=searches[2], strict_winner=True,
                     exact_steps=[0, 50, 100])
    for bits in ALL_BITS:
        _, _, qp_o = oracle.aciq_alpha(st_o, bits)
        full_pack_unpack(ctx, x, d, qp_o, bits, name)
    assert ctx.qp_get_status() == 0


C5_LOG2 = list(range(18, 29))


@pytest.mark.parametrize("log2n", C5_LOG2)
def test_roofline_sweep_sizes(ctx, log2n):
    """The roofline sweep's tensors, every size 2^18 .. 2^28, both distributions: statistics, and
    pack/unpack at every width of the sweep over the whole buffer; bf16 input of the same element
    count at the widths the sweep times for it."""
    n = 1 << log2n
    for dist in ("laplace", "normal"):
        x = si.flat_iid(n, si.C5_SEED, dist)
        d = dev(x)
        st_o = oracle.stats(x)
        check_stats(ctx.read_stats(ctx.qp_stats(d)), st_o)
        for bits in si.C5_BITS:
            _, _, qp_o = oracle.aciq_alpha(st_o, bits, 1 if dist == "normal" else 0)
            full_pack_unpack(ctx, x, d, qp_o, bits, (log2n, dist))
        if dist == "laplace":                                        # bf16 input of the same element count
            h = si.to_bf16_bits(x)
            del d
            db = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
            xw = oracle.widen_bf16(h)
            st_w = oracle.stats(xw)
            check_stats(ctx.read_stats(ctx.qp_stats(db)), st_w)
            for bits in (2, 4, 8, 16):
                _, _, qp_o = oracle.aciq_alpha(st_w, bits)
                full_pack_unpack(ctx, xw, db, qp_o, bits, (log2n, "bf16"))
            del db, xw, h
        del x
    assert ctx.qp_get_status() == 0


def test_search_beyond_one_wave_against_the_oracle(ctx):
    """2^26 + 3 elements: the second form of the moments pass runs two waves of blocks (its replica
    sums are 32 bit).  The interval path against the oracle itself (the oracle needs about a minute
    here), and the plain form of the pass against the same curve."""
    n = (1 << 26) + 3
    x = si.flat_iid(n, 91, "laplace")
    x[::1000] *= np.float32(6.0)                          # some elements beyond every clip range
    d = dev(x)
    st_o = oracle.stats(x)
    result = oracle.ds_search(x, st_o, 3)
    for path in (qp.QP_SEARCH_INTERVALS, qp.QP_SEARCH_INTERVALS_PLAIN):
        check_search(ctx, x, d, 3, path=path, oracle_result=result, exact_steps=[0, 50, 100, result[1].k_star])
    assert ctx.qp_get_status() == 0


@pytest.mark.parametrize("n", [(1 << 27) + 4099])
def test_search_forms_agree_beyond_two_waves(ctx, n):
    """Three waves of the second form (134 M elements).  The oracle would need minutes here, so the
    three scoring kernels, each checked against the oracle up to 67 M elements, are compared with
    one another: the two forms of the interval pass share the partition and differ only in who
    adds what, the candidate-by-candidate kernel is independent of both."""
    x = si.flat_iid(n, 91, "laplace")
    x[::1000] *= np.float32(6.0)                          # some elements beyond every clip range
    d = dev(x)
    d_stats = ctx.qp_stats(d, hist_bins=100)
    curves, results = {}, {}
    for path in (qp.QP_SEARCH_INTERVALS, qp.QP_SEARCH_INTERVALS_PLAIN, qp.QP_SEARCH_CANDIDATES):
        ctx.qp_set_search_path(path)
        try:
            d_res, d_qp = ctx.qp_dsaciq_search(d, d_stats, 3)
        finally:
            ctx.qp_set_search_path(qp.QP_SEARCH_AUTO)
        results[path] = (bytes(ctx.read_ds_result(d_res)), bytes(ctx.read_qparams(d_qp)))
        curves[path] = np.array(ctx.qp_dsaciq_curve(100))
    # same integer interval sums; the sums beyond the grid and of the squared offsets are fp32 batches
    # folded into fp64 in another grouping, so the curves agree to rounding, not bit for bit
    a, b = curves[qp.QP_SEARCH_INTERVALS], curves[qp.QP_SEARCH_INTERVALS_PLAIN]
    assert np.all(np.abs(a - b) <= 1e-9 * b)
    assert results[qp.QP_SEARCH_INTERVALS][1] == results[qp.QP_SEARCH_INTERVALS_PLAIN][1]       # the same winner
    ref = curves[qp.QP_SEARCH_CANDIDATES]
    assert np.all(np.abs(curves[qp.QP_SEARCH_INTERVALS] - ref) <= 2e-6 * ref)
    res_iv = qp.DSResult.from_buffer_copy(results[qp.QP_SEARCH_INTERVALS][0])
    res_c = qp.DSResult.from_buffer_copy(results[qp.QP_SEARCH_CANDIDATES][0])
    assert res_iv.k_star == res_c.k_star or ref[res_iv.k_star] <= ref[res_c.k_star] * (1 + 1e-6)
    assert ctx.qp_get_status() == 0


# ------------------------------------------------------------------ graph replay (execution option)

@pytest.mark.parametrize("n_images,path", [(6, qp.QP_SEARCH_CANDIDATES), (40, qp.QP_SEARCH_AUTO)])
def test_graph_replay_gives_the_same_bytes(n_images, path):
    """With replay on, a repeated call launches the graph recorded by the first one.  The
    results must be the bytes of the plain launches, also after the input buffer's CONTENTS
    changed between replays, and the launch counter must advance as if launched one by one."""
    plain, replay = qp.Context(0), qp.Context(0)
    for c in (plain, replay):
        c.qp_set_search_path(path)
    replay.qp_set_graph_replay(True)
    inputs = [si.vit_activation((n_images, 197, 256), 90 + i, outlier_frac=0.002 * i).reshape(-1) for i in range(3)]
    n = inputs[0].size
    d_x = torch.empty(n, device="cuda")
    st, res, dq = (torch.empty(k, dtype=torch.uint8, device="cuda")
                   for k in (ctypes.sizeof(qp.Stats), ctypes.sizeof(qp.DSResult), ctypes.sizeof(qp.QParams)))
    packed = torch.empty(qp.qp_packed_bytes(n, 2), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    per_call = None
    for i, x in enumerate(inputs + inputs[:1]):
        d_x.copy_(torch.from_numpy(x))
        want_st = plain.qp_stats(d_x, hist_bins=100)
        want_res, want_qp = plain.qp_dsaciq_search(d_x, want_st, 2)
        want_packed, want_qp2 = plain.qp_sender_device(d_x, 2, True)
        torch.cuda.synchronize()
        before = replay.qp_launch_count()
        with torch.cuda.stream(side):
            replay.qp_stats(d_x, out=st, hist_bins=100)
            replay.qp_dsaciq_search(d_x, st, 2, out_result=res, out_qp=dq)
            replay.qp_sender_device(d_x, 2, True, out_packed=packed, out_qp=dq)
        side.synchronize()
        launched = replay.qp_launch_count() - before
        per_call = launched if per_call is None else per_call
        assert launched == per_call and launched >= 5
        assert replay.qp_graph_replays() == 3 * i
        assert torch.equal(st, want_st) and torch.equal(res, want_res)
        assert torch.equal(dq, want_qp2) and torch.equal(want_qp, want_qp2) and torch.equal(packed, want_packed)
        o = oracle.QParams(*[getattr(replay.read_qparams(dq), f) for f in ("lo", "hi", "scale", "inv_scale", "bits", "flags")])
        assert np.array_equal(packed.cpu().numpy(), oracle.quantize_pack(x, o))
    # the legacy default stream cannot be captured: the call is enqueued directly and still right
    hits = replay.qp_graph_replays()
    replay.qp_stats(d_x, out=st, hist_bins=100)
    torch.cuda.synchronize()
    assert replay.qp_graph_replays() == hits and torch.equal(st, want_st)
    # a refused call records nothing and leaves the stream usable
    with torch.cuda.stream(side):
        with pytest.raises(qp.QuantPipeError):
            replay.qp_dsaciq_search(d_x, st, 9, out_result=res, out_qp=dq)
        replay.qp_stats(d_x, out=st, hist_bins=100)
    side.synchronize()
    assert torch.equal(st, want_st)
    # switching replay off drops the graphs; calls go back to plain launches
    replay.qp_set_graph_replay(False)
    hits = replay.qp_graph_replays()
    with torch.cuda.stream(side):
        replay.qp_stats(d_x, out=st, hist_bins=100)
    side.synchronize()
    assert replay.qp_graph_replays() == hits and torch.equal(st, want_st)
    assert replay.qp_get_status() == 0 and plain.qp_get_status() == 0
    plain.close(); replay.close()


# ------------------------------------------------------------------ channel-wise variant

def _read_array(t, ctype, count):
    raw = t.cpu().numpy().tobytes()
    return (ctype * count).from_buffer_copy(raw)


def check_channels(ctx, x_np, d_x, channels, bits, method=qp.QP_CLIP_ACIQ, out_bf16=False):
    """Statistics, quantizers, packed stream and reconstruction of the channel-wise calls against the
    oracle.  The statistics are compared at 1e-5; the packed stream bit for bit under the quantizers the
    kernels produced, and those quantizers against the oracle's per channel."""
    rows = x_np.size // channels
    d_stats = ctx.qp_stats_channels(d_x, channels)
    st = _read_array(d_stats, qp.Stats, channels)
    st_o = oracle.stats_channels(x_np, channels)
    for c in range(channels):
        check_stats(st[c], st_o[c])
    o_method, cut = (oracle.CLIP_MINMAX, False) if method & 0xF == qp.QP_CLIP_MINMAX else (oracle.CLIP_ACIQ, bool(method & qp.QP_CLIP_INTERSECT))
    d_qp = ctx.qp_clip_qparams_channels_device(d_stats, channels, bits, method)
    got = _read_array(d_qp, qp.QParams, channels)
    rc_o, qp_o = oracle.clip_channels(st_o, bits, o_method, cut, midrise=bool(method & qp.QP_CLIP_MIDRISE))
    for c in range(channels):
        width = max(qp_o[c].hi - qp_o[c].lo, 1e-30)
        assert abs(got[c].lo - qp_o[c].lo) <= 1e-5 * width and abs(got[c].hi - qp_o[c].hi) <= 1e-5 * width, c
        assert got[c].bits == bits and got[c].flags == qp_o[c].flags
        rc2, again = oracle.make_qparams(got[c].lo, got[c].hi, bits)
        assert (again.scale, again.inv_scale) == (got[c].scale, got[c].inv_scale)
    mine = (oracle.QParams * channels)(*[oracle.QParams(g.lo, g.hi, g.scale, g.inv_scale, g.bits, g.flags) for g in got])
    nbytes = qp.qp_packed_bytes(x_np.size, bits)
    whole, packed = guarded(nbytes)
    ctx.qp_quantize_pack_channels(d_x, channels, bits, d_qp, out=packed)
    codes_o = oracle.quantize_channels(x_np, channels, mine)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack(codes_o, bits))
    assert canaries_intact(whole, nbytes)
    esz = 2 if out_bf16 else 4
    whole_y, y_bytes = guarded(x_np.size * esz)
    y = y_bytes.view(torch.bfloat16 if out_bf16 else torch.float32)
    ctx.qp_unpack_dequantize_channels(packed, rows, channels, bits, d_qp, out=y)
    y_o = oracle.dequantize_channels(codes_o, channels, mine)
    if out_bf16:
        want = si.bf16_bits_to_f32(si.to_bf16_bits(y_o))
        assert np.array_equal(y.float().cpu().numpy(), want)
    else:
        assert np.max(np.abs(y.cpu().numpy().astype(np.float64) - y_o.astype(np.float64)), initial=0.0) <= 1e-6
    assert canaries_intact(whole_y, x_np.size * esz)
    return got


@pytest.mark.parametrize("bits", ALL_BITS)
def test_channels_vit_shapes(ctx, bits):
    x = si.vit_activation((2, 197, 768), 101, outlier_frac=0.01).reshape(-1)
    check_channels(ctx, x, dev(x), 768, bits)
    assert ctx.qp_get_status() == 0


@pytest.mark.parametrize("channels,rows", [(1, 5000), (3, 777), (4, 1), (20, 411), (64, 2049), (1000, 37), (1280, 300),
                                            (4096, 9)])
def test_channels_shapes_ragged_and_methods(ctx, channels, rows):
    x = si.vit_activation((1, rows, channels), 102 + channels % 5, outlier_frac=0.05).reshape(-1)
    d = dev(x)
    for bits, method in ((2, qp.QP_CLIP_ACIQ), (5, qp.QP_CLIP_MINMAX), (8, qp.QP_CLIP_ACIQ | qp.QP_CLIP_INTERSECT),
                         (16, qp.QP_CLIP_ACIQ), (4, qp.QP_CLIP_ACIQ | qp.QP_CLIP_MIDRISE),
                         (3, qp.QP_CLIP_MINMAX | qp.QP_CLIP_MIDRISE)):
        check_channels(ctx, x, d, channels, bits, method)
    ctx.qp_get_status()                                         # single-row tensors have no spread: degenerate


def test_channels_misaligned_nonfinite_bf16(ctx):
    x = si.vit_activation((1, 301, 96), 107, outlier_frac=0.03).reshape(-1).astype(np.float32)
    big = dev(np.concatenate([np.zeros(1, np.float32), x]))
    check_channels(ctx, x, big[1:], 96, 4)                      # 4-byte aligned only: scalar paths
    x[[5, 96 * 7 + 5, 96 * 100 + 17]] = [np.nan, np.inf, -np.inf]
    check_channels(ctx, x, dev(x), 96, 3)
    assert ctx.qp_get_status() & qp.QP_DEV_NONFINITE
    h = si.to_bf16_bits(si.vit_activation((1, 150, 256), 108).reshape(-1))
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    check_channels(ctx, oracle.widen_bf16(h), d, 256, 4)
    check_channels(ctx, oracle.widen_bf16(h), d, 256, 8, out_bf16=True)
    check_channels(ctx, oracle.widen_bf16(h[:150 * 100]), d[:150 * 100], 100, 6, out_bf16=True)   # 100 % 8 != 0
    const = np.tile(np.array([1.5, -2.0, 0.0, 7.25], dtype=np.float32), 500)                      # every channel constant
    got = check_channels(ctx, const, dev(const), 4, 4)
    assert all(g.flags == 1 for g in got) and ctx.qp_get_status() & qp.QP_DEV_DEGENERATE


def test_channels_errors_and_empty(ctx):
    x = dev(si.flat_iid(4096, 6, "laplace"))
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_stats_channels(torch.zeros(2 * 8192, device="cuda"), 8192)      # beyond QP_MAX_CHANNELS
    d_stats = ctx.qp_stats_channels(x, 64)
    for bad in (qp.QP_CLIP_DSACIQ, 3):
        with pytest.raises(qp.QuantPipeError):
            ctx.qp_clip_qparams_channels_device(d_stats, 64, 4, bad)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_clip_qparams_channels_device(d_stats, 64, 9)
    d_qp = ctx.qp_clip_qparams_channels_device(d_stats, 64, 4)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_quantize_pack_channels(x, 64, 4, d_qp, out=torch.empty(16, dtype=torch.uint8, device="cuda"))
    ctx.qp_quantize_pack_channels(x, 64, 8, d_qp)               # quantizers made for 4 bits: flagged on the device
    assert ctx.qp_get_status() & qp.QP_DEV_BITS_MISMATCH
    empty = torch.empty(0, device="cuda")
    st = _read_array(ctx.qp_stats_channels(empty, 16), qp.Stats, 16)
    assert all(s.n == 0 and s.mean == 0.0 for s in st)


def test_channels_full_size_c2_sampled(ctx):
    """ViT-Base micro-batch of 64 images, 768 channels: statistics of sampled channels and the packed
    words of sampled rows against the oracle."""
    x = si.config_tensor("c2").reshape(-1, 768)
    d = dev(x.reshape(-1))
    d_stats = ctx.qp_stats_channels(d, 768)
    st = _read_array(d_stats, qp.Stats, 768)
    for c in (0, 1, 255, 500, 767):
        check_stats(st[c], oracle.stats(np.ascontiguousarray(x[:, c])))
    d_qp = ctx.qp_clip_qparams_channels_device(d_stats, 768, 4)
    got = _read_array(d_qp, qp.QParams, 768)
    mine = (oracle.QParams * 768)(*[oracle.QParams(g.lo, g.hi, g.scale, g.inv_scale, g.bits, g.flags) for g in got])
    packed = ctx.qp_quantize_pack_channels(d, 768, 4, d_qp).cpu().numpy()
    y = ctx.qp_unpack_dequantize_channels(torch.from_numpy(packed).cuda(), x.shape[0], 768, 4, d_qp).cpu().numpy().reshape(-1, 768)
    for r0 in (0, 4097, x.shape[0] - 3):
        rows = x[r0:r0 + 3]
        codes = oracle.quantize_channels(rows, 768, mine)
        nb = 3 * 768 * 4 // 8
        assert np.array_equal(packed[r0 * 768 // 2: r0 * 768 // 2 + nb], oracle.pack(codes, 4)[:nb])
        assert np.max(np.abs(y[r0:r0 + 3].reshape(-1) - oracle.dequantize_channels(codes, 768, mine))) <= 1e-6
    assert ctx.qp_get_status() == 0


def test_channels_sender_in_one_call(ctx):
    x = si.vit_activation((2, 197, 384), 109, outlier_frac=0.02).reshape(-1)
    d = dev(x)
    for bits, method in ((4, qp.QP_CLIP_ACIQ), (8, qp.QP_CLIP_MINMAX | qp.QP_CLIP_MIDRISE)):
        d_stats = ctx.qp_stats_channels(d, 384)
        d_qp = ctx.qp_clip_qparams_channels_device(d_stats, 384, bits, method)
        want = ctx.qp_quantize_pack_channels(d, 384, bits, d_qp)
        got, got_qp = ctx.qp_sender_channels_device(d, 384, bits, method)            # statistics kept by the context
        assert torch.equal(got, want) and torch.equal(got_qp, d_qp)
        st_out = torch.empty(384 * ctypes.sizeof(qp.Stats), dtype=torch.uint8, device="cuda")
        got2, _ = ctx.qp_sender_channels_device(d, 384, bits, method, out_stats=st_out)
        assert torch.equal(got2, want) and torch.equal(st_out, d_stats)
    # with the directed search per channel
    for bits, method, bmode in ((2, qp.QP_CLIP_DSACIQ, 0), (4, qp.QP_CLIP_DSACIQ | qp.QP_CLIP_MIDRISE, qp.QP_B_MIDRISE)):
        d_stats = ctx.qp_stats_channels(d, 384)
        _, d_qp = ctx.qp_dsaciq_search_channels(d, 384, d_stats, bits, bmode)
        want = ctx.qp_quantize_pack_channels(d, 384, bits, d_qp)
        got, got_qp = ctx.qp_sender_channels_device(d, 384, bits, method)
        assert torch.equal(got, want) and torch.equal(got_qp, d_qp)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_sender_channels_device(d, 384, 16, qp.QP_CLIP_DSACIQ)
    assert ctx.qp_get_status() & ~qp.QP_DEV_DEGENERATE == 0


# ------------------------------------------------- channel-wise directed search

def check_search_channels(ctx, x_np, d_x, channels, bits, bmode=0, steps=100, nb=100):
    """Every channel's search against the oracle's search of that column, as check_search: the
    candidates' clip ranges, every candidate's error for exactly the quantizer the library scored
    (2e-6), the winner (first minimum, or a tie at 1e-6) and its clipping value (1e-4).  Both forms
    of the library's search: interval moments (the default where they apply) and the scoring of
    every candidate."""
    rows = x_np.size // channels
    st_o = oracle.stats_channels(x_np, channels)
    rc_o, res_o, qp_o, curves_o = oracle.ds_search_channels(x_np, channels, st_o, bits, bmode, steps, nb)
    cols = x_np.reshape(rows, channels)
    rsz, qsz = ctypes.sizeof(qp.DSResult), ctypes.sizeof(qp.QParams)
    try:
        for path in (qp.QP_SEARCH_AUTO, qp.QP_SEARCH_CANDIDATES):
            ctx.qp_set_search_path(path)
            d_stats = ctx.qp_stats_channels(d_x, channels)
            d_res, d_qp = ctx.qp_dsaciq_search_channels(d_x, channels, d_stats, bits, bmode, steps, nb)
            raw_res = d_res.cpu().numpy().tobytes()
            raw_qp = d_qp.cpu().numpy().tobytes()
            cand_all = ctx.qp_dsaciq_candidates_channels(channels, steps)
            for c in range(channels):
                res = qp.DSResult.from_buffer_copy(raw_res[c * rsz:(c + 1) * rsz])
                got = qp.QParams.from_buffer_copy(raw_qp[c * qsz:(c + 1) * qsz])
                ro = res_o[c]
                assert (res.steps, res.hist_bins, res.bits) == (steps, nb, bits)
                assert abs(res.b_e - ro.b_e) <= 1e-5 * abs(ro.b_e) + 1e-300
                assert abs(res.b_r - ro.b_r) <= 1e-9 * abs(ro.b_r) + 1e-300         # integer-identical histogram
                curve = np.array(ctx.qp_dsaciq_curve_channels(c, steps))
                cand = cand_all[c * (steps + 1):(c + 1) * (steps + 1)]
                check_candidates_and_pick(np.ascontiguousarray(cols[:, c]), st_o[c], ro, curves_o[c], res, curve, cand, bits,
                                          bmode, steps)
                w = cand[res.k_star]
                assert (got.lo, got.hi, got.scale, got.inv_scale, got.bits) == (w.lo, w.hi, w.scale, w.inv_scale, bits)
                assert got.flags == qp_o[c].flags
                assert res.mse_star == curve[res.k_star] and res.mse_e == curve[0]
    finally:
        ctx.qp_set_search_path(qp.QP_SEARCH_AUTO)
    # the quantizers feed the channel-wise packer: bit-exact codes under the library's own quantizers
    mine = (oracle.QParams * channels)()
    for c in range(channels):
        g = qp.QParams.from_buffer_copy(raw_qp[c * qsz:(c + 1) * qsz])
        mine[c] = oracle.QParams(g.lo, g.hi, g.scale, g.inv_scale, g.bits, g.flags)
    packed = ctx.qp_quantize_pack_channels(d_x, channels, bits, d_qp)
    codes_o = oracle.quantize_channels(x_np, channels, mine)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack(codes_o, bits))
    return rc_o


@pytest.mark.parametrize("bits", [1, 2, 3, 4, 8])
def test_search_channels_vit(ctx, bits):
    x = si.vit_activation((2, 197, 96), 131, outlier_frac=0.03).reshape(-1)
    check_search_channels(ctx, x, dev(x), 96, bits)
    ctx.qp_get_status()


@pytest.mark.parametrize("channels,rows", [(1, 5000), (3, 777), (5, 1), (33, 100), (70, 2049), (1280, 64)])
def test_search_channels_shapes_and_modes(ctx, channels, rows):
    x = si.vit_activation((1, rows, channels), 140 + channels % 7, outlier_frac=0.05).reshape(-1)
    d = dev(x)
    check_search_channels(ctx, x, d, channels, 2, nb=64)
    check_search_channels(ctx, x, d, channels, 4, bmode=qp.QP_B_MEAN_ABS | qp.QP_B_MIDRISE, steps=37, nb=256)
    check_search_channels(ctx, x, d, channels, 3, bmode=qp.QP_B_GAUSS, steps=127, nb=1)
    ctx.qp_get_status()


def test_search_channels_special_values_bf16_and_errors(ctx):
    channels, rows = 12, 3000
    x = si.vit_activation((1, rows, channels), 151).reshape(rows, channels).copy()
    x[:, 4] = np.float32(0.5)                                   # a constant channel: degenerate, b_E kept
    x[[7, 100, 2999], [0, 3, 11]] = [np.nan, np.inf, -np.inf]
    flat = x.reshape(-1)
    assert check_search_channels(ctx, flat, dev(flat), channels, 2) == oracle.WARN_DEGENERATE
    assert ctx.qp_get_status() & qp.QP_DEV_DEGENERATE
    h = si.to_bf16_bits(si.vit_activation((1, 500, 40), 152).reshape(-1))
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    check_search_channels(ctx, oracle.widen_bf16(h), d, 40, 4)
    y = dev(flat)
    st = ctx.qp_stats_channels(y, channels)
    for bad in (dict(bits=16), dict(bits=2, steps=128), dict(bits=2, hist_bins=257), dict(bits=2, bmode=qp.QP_B_HIST_IN_STATS),
                dict(bits=2, steps=0)):
        with pytest.raises(qp.QuantPipeError):
            ctx.qp_dsaciq_search_channels(y, channels, st, **bad)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_dsaciq_search_channels(y, y.numel(), st, 2)          # 36000 channels: beyond QP_MAX_CHANNELS
    ctx.qp_get_status()


@pytest.mark.parametrize("name,bits", [("c3", 4), ("c4", 2)])
def test_search_channels_full_size_sampled(ctx, name, bits):
    """Full-size configs (c3: outlier channels; c4: the largest, 9 channels per block of the interval pass):
    sampled channels against the oracle's search of the column, the whole curve on the library's own
    quantizers, both forms of the search."""
    C = si.CONFIGS[name]["shape"][-1]
    x = si.config_tensor(name).reshape(-1, C)
    d = dev(x.reshape(-1))
    d_stats = ctx.qp_stats_channels(d, C)
    rsz = ctypes.sizeof(qp.DSResult)
    sample = (0, 17, C // 2 - 1, C - 1)
    ref = {}
    for c in sample:
        col = np.ascontiguousarray(x[:, c])
        st_c = oracle.stats(col)
        ref[c] = (col, st_c) + tuple(oracle.ds_search(col, st_c, bits)[i] for i in (1, 3))
    try:
        for path in (qp.QP_SEARCH_AUTO, qp.QP_SEARCH_CANDIDATES):
            ctx.qp_set_search_path(path)
            d_res, d_qp = ctx.qp_dsaciq_search_channels(d, C, d_stats, bits)
            raw = d_res.cpu().numpy().tobytes()
            cand_all = ctx.qp_dsaciq_candidates_channels(C, 100)
            for c in sample:
                col, st_c, ro, curve_o = ref[c]
                res = qp.DSResult.from_buffer_copy(raw[c * rsz:(c + 1) * rsz])
                assert abs(res.b_r - ro.b_r) <= 1e-9 * ro.b_r
                curve = np.array(ctx.qp_dsaciq_curve_channels(c, 100))
                check_candidates_and_pick(col, st_c, ro, curve_o, res, curve, cand_all[c * 101:(c + 1) * 101], bits, 0, 100)
    finally:
        ctx.qp_set_search_path(qp.QP_SEARCH_AUTO)
    assert ctx.qp_get_status() & ~qp.QP_DEV_DEGENERATE == 0


@pytest.mark.parametrize("rows", [65535, 65536])
def test_search_channels_at_the_row_limit_of_the_interval_form(ctx, rows):
    """65535 rows is the most the interval form's 16-bit counts hold; one more row and the call scores every
    candidate on every element instead.  A constant-heavy channel puts nearly all rows into one interval."""
    channels = 3
    x = si.vit_activation((1, rows, channels), 161).reshape(rows, channels).copy()
    x[: rows - 40, 1] = np.float32(-0.25)                       # one interval holds rows - 40 elements
    flat = x.reshape(-1)
    check_search_channels(ctx, flat, dev(flat), channels, 2)
    ctx.qp_get_status()


# ------------------------------------------------------------------ token-wise variant

def check_tokens(ctx, x_np, d_x, channels, bits, method=qp.QP_CLIP_ACIQ, out_bf16=False):
    """Statistics, quantizers, packed stream and reconstruction of the token-wise calls against the oracle:
    statistics at 1e-5; the packed stream bit for bit under the quantizers the kernels produced, and those
    quantizers against the oracle's per token; reconstruction at 1e-6 (bf16: the rounded oracle value)."""
    tokens = x_np.size // channels
    d_stats = ctx.qp_stats_tokens(d_x, channels)
    st = _read_array(d_stats, qp.Stats, tokens)
    st_o = oracle.stats_tokens(x_np, channels)
    for t in range(tokens):
        check_stats(st[t], st_o[t])
    o_method, cut = (oracle.CLIP_MINMAX, False) if method & 0xF == qp.QP_CLIP_MINMAX else (oracle.CLIP_ACIQ, bool(method & qp.QP_CLIP_INTERSECT))
    d_qp = ctx.qp_clip_qparams_tokens_device(d_stats, tokens, bits, method)
    got = _read_array(d_qp, qp.QParams, tokens)
    rc_o, qp_o = oracle.clip_tokens(st_o, bits, o_method, cut, midrise=bool(method & qp.QP_CLIP_MIDRISE))
    for t in range(tokens):
        width = max(qp_o[t].hi - qp_o[t].lo, 1e-30)
        assert abs(got[t].lo - qp_o[t].lo) <= 1e-5 * width and abs(got[t].hi - qp_o[t].hi) <= 1e-5 * width, t
        assert got[t].bits == bits and got[t].flags == qp_o[t].flags
        rc2, again = oracle.make_qparams(got[t].lo, got[t].hi, bits)
        assert (again.scale, again.inv_scale) == (got[t].scale, got[t].inv_scale)
    mine = (oracle.QParams * tokens)(*[oracle.QParams(g.lo, g.hi, g.scale, g.inv_scale, g.bits, g.flags) for g in got])
    nbytes = qp.qp_packed_bytes(x_np.size, bits)
    whole, packed = guarded(nbytes)
    ctx.qp_quantize_pack_tokens(d_x, channels, bits, d_qp, out=packed)
    codes_o = oracle.quantize_tokens(x_np, channels, mine)
    assert np.array_equal(packed.cpu().numpy(), oracle.pack(codes_o, bits))
    assert canaries_intact(whole, nbytes)
    esz = 2 if out_bf16 else 4
    whole_y, y_bytes = guarded(x_np.size * esz)
    y = y_bytes.view(torch.bfloat16 if out_bf16 else torch.float32)
    ctx.qp_unpack_dequantize_tokens(packed, tokens, channels, bits, d_qp, out=y)
    y_o = oracle.dequantize_tokens(codes_o, channels, mine)
    if out_bf16:
        assert np.array_equal(y.float().cpu().numpy(), si.bf16_bits_to_f32(si.to_bf16_bits(y_o)))
    else:
        assert np.max(np.abs(y.cpu().numpy().astype(np.float64) - y_o.astype(np.float64)), initial=0.0) <= 1e-6
    assert canaries_intact(whole_y, x_np.size * esz)
    # the one-call sender gives the same stream and quantizers
    got_packed, got_qp = ctx.qp_sender_tokens_device(d_x, channels, bits, method)
    assert torch.equal(got_packed, packed) and torch.equal(got_qp, d_qp)
    return got


@pytest.mark.parametrize("bits", ALL_BITS)
def test_tokens_vit_shapes(ctx, bits):
    x = si.vit_activation((2, 197, 768), 161, outlier_frac=0.01).reshape(-1)
    check_tokens(ctx, x, dev(x), 768, bits)
    assert ctx.qp_get_status() == 0


@pytest.mark.parametrize("channels,tokens", [(1, 700), (3, 777), (4, 1), (20, 411), (64, 2049), (100, 333), (1000, 37),
                                              (1280, 300), (5000, 9)])
def test_tokens_shapes_ragged_and_methods(ctx, channels, tokens):
    x = si.vit_activation((1, tokens, channels), 162 + channels % 5, outlier_frac=0.05).reshape(-1)
    d = dev(x)
    for bits, method in ((2, qp.QP_CLIP_ACIQ), (5, qp.QP_CLIP_MINMAX), (8, qp.QP_CLIP_ACIQ | qp.QP_CLIP_INTERSECT),
                         (16, qp.QP_CLIP_ACIQ), (4, qp.QP_CLIP_ACIQ | qp.QP_CLIP_MIDRISE),
                         (3, qp.QP_CLIP_MINMAX | qp.QP_CLIP_MIDRISE)):
        check_tokens(ctx, x, d, channels, bits, method)
    ctx.qp_get_status()                                         # one-channel tokens have no spread: degenerate


def test_tokens_misaligned_nonfinite_bf16_and_errors(ctx):
    x = si.vit_activation((1, 301, 96), 167, outlier_frac=0.03).reshape(-1).astype(np.float32)
    big = dev(np.concatenate([np.zeros(1, np.float32), x]))
    check_tokens(ctx, x, big[1:], 96, 4)                        # 4-byte aligned only: scalar paths
    x[[5, 96 * 7 + 5, 96 * 100 + 17]] = [np.nan, np.inf, -np.inf]
    check_tokens(ctx, x, dev(x), 96, 3)
    assert ctx.qp_get_status() & qp.QP_DEV_NONFINITE
    h = si.to_bf16_bits(si.vit_activation((1, 150, 256), 168).reshape(-1))
    d = torch.from_numpy(h.view(np.int16)).cuda().view(torch.bfloat16)
    check_tokens(ctx, oracle.widen_bf16(h), d, 256, 4)
    check_tokens(ctx, oracle.widen_bf16(h), d, 256, 8, out_bf16=True)
    check_tokens(ctx, oracle.widen_bf16(h[:150 * 100]), d[:150 * 100], 100, 6, out_bf16=True)   # 100 % 8 != 0
    const = np.repeat(np.array([1.5, -2.0, 0.0, 7.25], dtype=np.float32), 500)                  # every token constant
    got = check_tokens(ctx, const, dev(const), 500, 4)
    assert all(g.flags == 1 for g in got) and ctx.qp_get_status() & qp.QP_DEV_DEGENERATE
    y = dev(si.flat_iid(4096, 6, "laplace"))
    d_stats = ctx.qp_stats_tokens(y, 64)
    for bad in (qp.QP_CLIP_DSACIQ, 3):
        with pytest.raises(qp.QuantPipeError):
            ctx.qp_clip_qparams_tokens_device(d_stats, 64, 4, bad)
    d_qp = ctx.qp_clip_qparams_tokens_device(d_stats, 64, 4)
    with pytest.raises(qp.QuantPipeError):
        ctx.qp_quantize_pack_tokens(y, 64, 4, d_qp, out=torch.empty(16, dtype=torch.uint8, device="cuda"))
    ctx.qp_quantize_pack_tokens(y, 64, 8, d_qp)                 # quantizers made for 4 bits: flagged on the device
    assert ctx.qp_get_status() & qp.QP_DEV_BITS_MISMATCH


def test_tokens_full_size_c2_sampled(ctx):
    """ViT-Base micro-batch of 64 images (12 608 tokens of 768 channels): every token's statistics, and the
    packed words and reconstructions of sampled tokens, against the oracle."""
    x = si.config_tensor("c2").reshape(-1, 768)
    tokens = x.shape[0]
    d = dev(x.reshape(-1))
    d_stats = ctx.qp_stats_tokens(d, 768)
    st = _read_array(d_stats, qp.Stats, tokens)
    st_o = oracle.stats_tokens(x.reshape(-1), 768)
    for t in range(0, tokens, 97):
        check_stats(st[t], st_o[t])
    d_qp = ctx.qp_clip_qparams_tokens_device(d_stats, tokens, 4)
    got = _read_array(d_qp, qp.QParams, tokens)
    packed = ctx.qp_quantize_pack_tokens(d, 768, 4, d_qp)
    y = ctx.qp_unpack_dequantize_tokens(packed, tokens, 768, 4, d_qp).cpu().numpy().reshape(-1, 768)
    packed = packed.cpu().numpy()
    for t0 in (0, 4097, tokens - 3):
        rows = np.ascontiguousarray(x[t0:t0 + 3])
        mine = (oracle.QParams * 3)(*[oracle.QParams(g.lo, g.hi, g.scale, g.inv_scale, g.bits, g.flags) for g in got[t0:t0 + 3]])
        codes = oracle.quantize_tokens(rows, 768, mine)
        nb = 3 * 768 * 4 // 8
        assert np.array_equal(packed[t0 * 768 // 2: t0 * 768 // 2 + nb], oracle.pack(codes, 4)[:nb])
        assert np.max(np.abs(y[t0:t0 + 3].reshape(-1) - oracle.dequantize_tokens(codes, 768, mine))) <= 1e-6
    assert ctx.qp_get_status() == 0
