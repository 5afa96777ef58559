"""The library's behaviour when something goes wrong on the device, and options that must not
change results: bounded waits that run out (made to run out by shortening the limit, never by
withholding work: nothing here faults, traps or hangs), and graph replay keyed by every argument.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2211_04515_b200 as qp
import synth_inputs as si

pytestmark = pytest.mark.gpu


def dev(x_np):
    return torch.from_numpy(np.ascontiguousarray(x_np)).cuda()


def stats_close(st, st_o):
    assert st.n == st_o.n and st.nonfinite == st_o.nonfinite and st.min == st_o.min and st.max == st_o.max
    assert abs(st.mean - st_o.mean) <= 1e-5 * max(abs(st_o.mean), st_o.mad)
    for f in ("mean_abs", "mad", "var"):
        assert abs(getattr(st, f) - getattr(st_o, f)) <= 1e-5 * abs(getattr(st_o, f)), f


@pytest.mark.parametrize("path", [qp.QP_STATS_FUSED, qp.QP_STATS_TWO_KERNELS])
def test_tile_wait_that_runs_out_is_reported_and_the_context_stays_usable(path):
    """Wait limit 0: the first look at the first tile finds its copy still in flight, the block gives
    up, waits (with the normal limit) for the copies it has in flight, and the kernel returns.
    qp_get_status reports QP_ERR_TIMEOUT; with the limit restored the same call is right again."""
    c = qp.Context(0)
    x = si.vit_activation((6, 197, 768), 301).reshape(-1)            # 3.6 MB: both streamed forms apply
    d = dev(x)
    st_o = oracle.stats(x)
    c.qp_set_stats_path(path)
    c.qp_set_wait_limit_for_testing(tile_wait_cycles=0)
    c.qp_stats(d, hist_bins=100)
    with pytest.raises(qp.QuantPipeError) as e:
        c.qp_get_status()
    assert e.value.status == qp.QP_ERR_TIMEOUT and "timed out" in str(e.value)
    assert c.qp_get_status() == 0                                    # the word was cleared with the report
    c.qp_set_wait_limit_for_testing()                                # defaults again
    for _ in range(2):
        st = c.read_stats(c.qp_stats(d, hist_bins=100))
        stats_close(st, st_o)
        assert st.hist_peak == int(oracle.hist_peak(x, st_o.min, st_o.max, 100)[1].max())
    assert c.qp_get_status() == 0
    c.close()


def test_grid_barrier_that_runs_out_is_reported_and_the_context_stays_usable():
    """A short poll limit together with a barrier that waits for one arrival more than there are
    blocks: every block's wait runs out after a fraction of a millisecond and every block leaves.
    Both cooperative kernels (statistics, whole sender); afterwards ordinary calls are right."""
    c = qp.Context(0)
    x = si.config_tensor("c1").reshape(-1)
    big = si.vit_activation((6, 197, 768), 302).reshape(-1)
    d, d_big = dev(x), dev(big)
    c.qp_set_stats_path(qp.QP_STATS_FUSED)
    c.qp_set_sender_path(qp.QP_SENDER_FUSED)
    c.qp_set_wait_limit_for_testing(barrier_polls=500, barrier_extra_arrivals=1)
    # statistics: the kernel's exit path leaves its scratch clean, so even without reading the status ...
    sentinel = torch.full((ctypes.sizeof(qp.Stats),), 0xEE, dtype=torch.uint8, device="cuda")
    c.qp_stats(d_big, out=sentinel)
    torch.cuda.synchronize()
    assert (sentinel.cpu().numpy() == 0xEE).all()                    # no output was written
    c.qp_set_wait_limit_for_testing()
    stats_close(c.read_stats(c.qp_stats(d_big)), oracle.stats(big))  # ... the next launch is right
    with pytest.raises(qp.QuantPipeError) as e:
        c.qp_get_status()
    assert e.value.status == qp.QP_ERR_TIMEOUT
    # whole sender in one launch
    c.qp_set_wait_limit_for_testing(barrier_polls=500, barrier_extra_arrivals=1)
    before = c.qp_launch_count()
    c.qp_sender_device(d, 2, True)
    assert c.qp_launch_count() - before == 1
    with pytest.raises(qp.QuantPipeError) as e:
        c.qp_get_status()                                            # also clears the barrier scratch
    assert e.value.status == qp.QP_ERR_TIMEOUT
    c.qp_set_wait_limit_for_testing()
    packed, d_qp = c.qp_sender_device(d, 2, True)
    q = c.read_qparams(d_qp)
    o = oracle.QParams(q.lo, q.hi, q.scale, q.inv_scale, q.bits, q.flags)
    assert np.array_equal(packed.cpu().numpy(), oracle.quantize_pack(x, o))
    _, res_o, _, curve_o = oracle.ds_search(x, oracle.stats(x), 2)
    cand = c.qp_dsaciq_candidates(100)
    k = [i for i in range(101) if (cand[i].lo, cand[i].hi) == (q.lo, q.hi)][0]
    assert k == res_o.k_star or curve_o[k] <= res_o.mse_star * (1 + 1e-6)
    assert c.qp_get_status() == 0
    with pytest.raises(qp.QuantPipeError):
        c.qp_set_wait_limit_for_testing(barrier_extra_arrivals=2)
    c.close()


def test_graph_replay_keeps_calls_with_different_options_apart():
    """Stored graphs are keyed by every argument.  Pairs of calls that differ only in the clip method
    and the histogram's bin count (fields that once shared bits of one key word) must each replay
    their own recording: with replay on, every call gives the bytes of the plain call."""
    plain, replay = qp.Context(0), qp.Context(0)
    replay.qp_set_graph_replay(True)
    for c in (plain, replay):
        c.qp_set_sender_path(qp.QP_SENDER_CHAIN)
    x = si.vit_activation((40, 197, 256), 303, outlier_frac=0.01).reshape(-1)     # 8 MB: interval search
    d = dev(x)
    n = x.size
    side = torch.cuda.Stream()
    calls = [(qp.QP_CLIP_DSACIQ, 8292), (qp.QP_CLIP_DSACIQ | qp.QP_CLIP_MIDRISE, 100), (qp.QP_CLIP_ACIQ, 512),
             (qp.QP_CLIP_MINMAX, 0), (qp.QP_CLIP_DSACIQ, 100), (qp.QP_CLIP_DSACIQ, 356), (qp.QP_CLIP_ACIQ | qp.QP_CLIP_MIDRISE, 0)]
    packed = torch.empty(qp.qp_packed_bytes(n, 4), dtype=torch.uint8, device="cuda")
    dq = torch.empty(ctypes.sizeof(qp.QParams), dtype=torch.uint8, device="cuda")
    for rounds in range(2):                                          # second round: every call is a replay
        for method, nb in calls:
            want, want_qp = plain.qp_sender_device(d, 4, method, hist_bins=max(nb, 1))
            torch.cuda.synchronize()
            packed.zero_()
            with torch.cuda.stream(side):
                replay.qp_sender_device(d, 4, method, out_packed=packed, out_qp=dq, hist_bins=max(nb, 1))
            side.synchronize()
            assert torch.equal(dq, want_qp) and torch.equal(packed, want), (rounds, method, nb)
    assert replay.qp_graph_replays() >= len(calls)
    assert plain.qp_get_status() == 0 and replay.qp_get_status() == 0
    plain.close(); replay.close()
