"""The CPU oracle, as it stands, on several host cores at once (test infrastructure).

The oracle is single-threaded C; ctypes releases the interpreter lock while it runs, so plain
threads are enough (no process pool, nothing forked after CUDA is up).  Independent oracle
calls run side by side (`run_all`), and the element-wise stages of a large tensor are cut into
chunks: a chunk that starts at a multiple of 128 elements starts on a byte boundary of the
packed stream for every bit-width (128 * bits / 8 = 16 * bits bytes), so quantize+pack of the
chunk is the corresponding slice of the whole stream.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

import oracle

WORKERS = max(1, min(32, os.cpu_count() or 1))
CHUNK = 1 << 21                      # elements; a multiple of 128


def run_all(jobs, parallel: bool = True):
    """Results of the callables in `jobs`, run on WORKERS threads (in this thread if not `parallel`)."""
    if len(jobs) <= 1 or WORKERS == 1 or not parallel:
        return [f() for f in jobs]
    with ThreadPoolExecutor(WORKERS) as ex:
        return list(ex.map(lambda f: f(), jobs))


def check_pack_unpack(x: np.ndarray, qp, got_packed: np.ndarray, got_y: np.ndarray | None, chunk: int = CHUNK):
    """Whole-buffer comparison in chunks: (all packed bytes equal, max |y - y_oracle|).

    x: the host tensor; qp: oracle.QParams; got_packed: the library's packed stream (all
    qp_packed_bytes of it); got_y: the library's reconstruction as fp32 (or None)."""
    n, bits = x.size, qp.bits
    assert chunk % 128 == 0 and got_packed.size == oracle.packed_bytes(n, bits)

    def job(s0):
        s1 = min(n, s0 + chunk)
        ref = oracle.quantize_pack(x[s0:s1], qp)
        b0 = s0 * bits // 8
        if s1 == n:                                       # the last chunk carries the pad bytes
            same = np.array_equal(got_packed[b0:], ref)
        else:
            nb = (s1 - s0) * bits // 8
            same = np.array_equal(got_packed[b0:b0 + nb], ref[:nb])
        err = 0.0
        if got_y is not None and s1 > s0:
            y_o = oracle.unpack_dequantize(ref, s1 - s0, qp)
            err = float(np.max(np.abs(got_y[s0:s1].astype(np.float64) - y_o.astype(np.float64))))
        return same, err

    res = run_all([(lambda s0=s0: job(s0)) for s0 in range(0, max(n, 1), chunk)])
    return all(r[0] for r in res), max(r[1] for r in res)
