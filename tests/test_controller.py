"""The adaptive controller (window averaging + bit-width decision, paper Sec. 3 "Adaptive PDA"
and Sec. 4.2): library and oracle replay the paper's five-phase bandwidth scenario on a
simulated link and must pass through the widths the paper reports."""
import os

import pytest

import oracle
import paper_2211_04515_b200 as qp

N = 64 * 197 * 768
S, R, WINDOW = 64.0, 100.0, 50
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "adaptive_replay.txt")


def scenario():
    phases, total, expect = [], 0, {}
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "phase":
            phases.append((int(t[1]), float(t[2]) * 1e6))
        elif t[0] == "microbatches":
            total = int(t[1])
        elif t[0].startswith("expect_"):
            expect[t[0][7:]] = [int(v) for v in t[1:]]
    return phases, total, expect


def link_bps(phases, i):
    bw = phases[0][1]
    for start, b in phases:
        if i >= start:
            bw = b
    return bw


def payload(bits):
    return (N * bits + 7) // 8


def replay(observe, phases, total):
    """observe(bytes, seconds) -> (bits, decided).  Returns the widths in force after each change, the
    width in force at every microbatch, and the microbatches at which a decision was taken."""
    bits, changes, trace, decided_at = 32, [32], [], []
    for i in range(total):
        nbytes = payload(bits)
        new_bits, decided = observe(float(nbytes), nbytes * 8.0 / link_bps(phases, i))
        if decided:
            decided_at.append(i)
        if new_bits != bits:
            changes.append(new_bits)
            bits = new_bits
        trace.append(bits)
    return changes, trace, decided_at


@pytest.mark.parametrize("mode,key", [(0, "fit"), (1, "eq2")])
def test_five_phase_replay(mode, key):
    phases, total, expect = scenario()
    c_o = oracle.controller_init(WINDOW, S, R, N, 0, (32, 16, 8, 6, 4, 2), mode, 0.0, 32)
    changes_o, trace_o, dec_o = replay(lambda b, s: oracle.controller_observe(c_o, b, s), phases, total)
    assert changes_o == expect[key]
    rc, c = qp.qp_controller_init(WINDOW, S, R, N, 0, None, mode, 0.0, 32)
    assert rc == 0

    def obs(b, s):
        rc, bits, decided = qp.qp_controller_observe(c, b, s)
        assert rc >= 0
        return bits, decided

    changes, trace, dec = replay(obs, phases, total)
    assert changes == expect[key] and trace == trace_o and dec == dec_o
    assert all((i + 1) % WINDOW == 0 for i in dec)         # decisions only when a window closes
    # the settled widths are the paper's: 400 Mbps -> 16, 50 -> 2, 200 -> 8, not limited -> 32
    assert trace[199] == 32 and trace[399] == 16 and trace[599] == 2 and trace[799] == 8 and trace[999] == 32
    # the new width is in force one window after the link changed (plus the straddling one for 200 Mbps)
    assert trace[249] == 16 and trace[449] == 2 and trace[699] == 8 and trace[849] == 32


def test_significant_change_threshold_and_window():
    phases, total, _ = scenario()
    rc, c = qp.qp_controller_init(WINDOW, S, R, N, 0, None, qp.QP_CTRL_FIT, 0.25, 32)
    c_o = oracle.controller_init(WINDOW, S, R, N, 0, (32, 16, 8, 6, 4, 2), 0, 0.25, 32)
    bits, n_decided = 32, 0
    for i in range(total):
        nbytes = payload(bits)
        sec = nbytes * 8.0 / link_bps(phases, i)
        rc, b, decided = qp.qp_controller_observe(c, float(nbytes), sec)
        assert (b, decided) == oracle.controller_observe(c_o, float(nbytes), sec)
        assert not decided or (i + 1) % WINDOW == 0                      # only at window ends
        n_decided += decided
        bits = b
    # a decision only when the window bandwidth moved by more than 25 %: first window + 5 changes
    assert n_decided == 6
    assert c.count == 0 and c.bits == 32


def test_controller_arguments_and_payload():
    rc, c = qp.qp_controller_init(10, 64, 100, 1000, 24, (8, 4, 2), qp.QP_CTRL_FIT, 0.0, 8)
    assert rc == 0 and c.n_allowed == 3 and c.bits == 8
    assert qp.qp_controller_payload_bytes(c, 8) == 1024 and qp.qp_controller_payload_bytes(c, 3) == 375 + 24
    assert qp.qp_controller_payload_bytes(c, 32) == 4024 and qp.qp_controller_payload_bytes(c, 0) == 0
    # nothing fits: the smallest allowed width, with a warning
    for _ in range(9):
        assert qp.qp_controller_observe(c, 1024.0, 10.0) == (0, 8, False)
    assert qp.qp_controller_observe(c, 1024.0, 10.0) == (qp.QP_WARN_INFEASIBLE, 2, True)
    for bad in (dict(window=0), dict(s=0.0), dict(r=-1.0), dict(allowed=(0,)), dict(allowed=tuple(range(1, 10))),
                dict(mode=2), dict(rel=-0.1), dict(initial=33)):
        kw = dict(window=10, s=64.0, r=100.0, allowed=(8, 4), mode=0, rel=0.0, initial=8)
        kw.update(bad)
        rc, _ = qp.qp_controller_init(kw["window"], kw["s"], kw["r"], 1000, 0, kw["allowed"], kw["mode"], kw["rel"],
                                      kw["initial"])
        assert rc == qp.QP_ERR_INVALID_ARG, bad
    rc, c = qp.qp_controller_init(2, 64, 100, 1000)
    assert qp.qp_controller_observe(c, -1.0, 1.0)[0] == qp.QP_ERR_INVALID_ARG
    # a window in which nothing was measured keeps the width
    assert qp.qp_controller_observe(c, 0.0, 0.0)[1:] == (32, False)
    assert qp.qp_controller_observe(c, 0.0, 0.0)[1:] == (32, False)
