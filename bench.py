#!/usr/bin/env python
"""Benchmark of the activation-quantization path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole path over one batch of the ViT-Huge-shaped workload
(fp32 [128,197,1280], 129 MB): bit-width from the step's link bandwidth (qp_select_bits on a
seeded 100-step trace), statistics, clip (directed search at <= 4 bits, plain ACIQ above),
quantize+pack, and the receiver's unpack+dequantize.  `value` is GB/s of fp32 input pushed
through the whole step with inputs resident in HBM; `e2e` is the same through the
host-buffer entry points with the host<->device copies inside the timed region.

`--impl reference` times the CPU oracle (as it stands, single thread) on a bounded sample of
the same workload and prints the same line shape.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synth_inputs as si  # noqa: E402

WORKLOAD = "c4"
METRIC = "quantize+pack and unpack+dequant throughput, fp32 in, whole path per step"
UNIT = "GB/s"
SAMPLE_IMAGES = 8              # CPU legs: the first 8 images of the batch (2.0 M elements) per step
ORACLE_US_PER_ELEM = 0.31      # rough cost of one oracle step per element (search on ~half the steps)
MIN_TIMED_S = 0.5              # the K-step region is repeated until this much device time has been measured

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum per launch) of each stage's main kernel on
# this workload, from one ncu capture each.  Every entry names the capture's summary and carries a
# digest of the kernel's source files at capture time: when those files have changed since, the entry
# is stale and the benchmark reports traffic = null.
NCU_TRAFFIC = {
    "stats": {"bytes": 176.7e6, "kernel": "stats_fused_kernel<float, 0>", "summary": "profiles/stats_fused_kernel_c4.md",
              "files": ("qp_stats.cu", "qp_stream.cuh", "qp_gridbar.cuh"), "digest": "6be59a35b2bfd17e"},
    "clip": {"bytes": 133.1e6, "kernel": "iv_moments2_kernel<float>", "summary": "profiles/kernels_c4_ncu_full.md",
             "files": ("qp_search_fast.cu",), "digest": "619ca87dc8596b84"},
    "quantize_pack": {"bytes": 141.5e6, "kernel": "pack_kernel<8, float>", "summary": "profiles/kernels_c4_ncu_full.md",
                      "files": ("qp_pack.cu",), "digest": "90a28547ba456cdf"},
    "unpack_dequantize": {"bytes": 99.3e6, "kernel": "unpack_kernel<8, float>", "summary": "profiles/kernels_c4_ncu_full.md",
                          "files": ("qp_unpack.cu",), "digest": "5b1421f640e0f472"},
}


def source_digest(files) -> str:
    import hashlib
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2211_04515_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def traffic_of(stage: str):
    """(bytes or None, source label) of the ncu DRAM traffic recorded for a stage's main kernel."""
    e = NCU_TRAFFIC.get(stage)
    if e is None or e["bytes"] is None:
        return None, "no capture of the current kernel"
    if source_digest(e["files"]) != e["digest"]:
        return None, f"stale: {', '.join(e['files'])} changed since the capture in {e['summary']}"
    return e["bytes"], f"ncu capture of {e['kernel']} summarised in {e['summary']} (source digest {e['digest']})"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return 6650.0, 1965.0, "fallback"


def step_bits(n_elems: int, select):
    """Bit-width of every step of the bandwidth trace (host, O(1) per step)."""
    trace = si.bandwidth_trace(si.CONFIGS[WORKLOAD]["seed"], si.C4_TRACE_STEPS)
    out = []
    for bw in trace:
        rc, q = select(float(bw), si.C4_BUDGET_S, n_elems, 24, si.C4_ALLOWED_BITS)
        out.append(q)
    return out


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while running."""

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=1.0)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "period_ms": self.period * 1e3}


def replica_throughput(local_ms: float, steps: int, bytes_per_step: float, world: int, device=None):
    """Whole-job GB/s of `world` independent replicas: every rank processed steps*bytes_per_step,
    the job took as long as its slowest rank (MAX over ranks of the device time)."""
    ms = float(local_ms)
    if world > 1:
        import torch
        import torch.distributed as dist
        t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return world * steps * bytes_per_step / (ms * 1e-3) / 1e9, ms


# --------------------------------------------------------------------- CPU oracle legs

def oracle_step(oracle, x, bits, use_ds):
    """One pass of the path in the oracle on host array x; returns nothing (timed by caller)."""
    st = oracle.stats(x)
    if use_ds:
        _, _, qp, _ = oracle.ds_search(x, st, bits)
    else:
        _, _, qp = oracle.aciq_alpha(st, bits)
    packed = oracle.quantize_pack(x, qp)
    oracle.unpack_dequantize(packed, x.size, qp)


def sample_images_for(steps: int, budget_s: float = 150.0) -> int:
    """Images per step of the CPU legs: SAMPLE_IMAGES, fewer only where `steps` oracle steps on that
    many images would take more than about budget_s seconds."""
    per_image = 197 * 1280 * ORACLE_US_PER_ELEM * 1e-6
    return int(max(1, min(SAMPLE_IMAGES, budget_s / (max(steps, 1) * per_image))))


def run_oracle_steps(first_step: int, count: int, bits_of_step, images: int = SAMPLE_IMAGES):
    import oracle
    x = si.vit_activation((images, 197, 1280), si.CONFIGS[WORKLOAD]["seed"]).reshape(-1)
    oracle.lib()
    t0 = time.perf_counter()
    for t in range(first_step, first_step + count):
        q = bits_of_step[t % len(bits_of_step)]
        oracle_step(oracle, x, q, 1 <= q <= 4)
    dt = time.perf_counter() - t0
    return dt, x.size


def sample_text(images: int, n_sample: int) -> str:
    return f"first {images} images of the batch ({n_sample} elements) per step, steps of the same trace"


def oracle_all_cores(x, bits_list=(4, 8)):
    """quantize+pack and unpack+dequantize of the oracle, as it stands, chunk-parallel over the host
    cores (a chunk that starts at a multiple of 128 elements starts on a byte boundary of the packed
    stream; ctypes releases the interpreter lock, so threads suffice).  GB/s of fp32 in (out)."""
    from concurrent.futures import ThreadPoolExecutor

    import oracle
    cores = os.cpu_count() or 1
    n = x.size
    chunk = max(128, (n // (4 * cores)) // 128 * 128)
    st = oracle.stats(x[:1 << 20])
    out = {"cores": cores, "sample": f"the whole batch ({n} elements), chunks of {chunk} elements on {cores} threads"}
    with ThreadPoolExecutor(cores) as ex:
        for bits in bits_list:
            _, _, qp_o = oracle.aciq_alpha(st, bits)
            starts = list(range(0, n, chunk))
            t0 = time.perf_counter()
            packed = list(ex.map(lambda s0: oracle.quantize_pack(x[s0:s0 + chunk], qp_o), starts))
            t1 = time.perf_counter()
            list(ex.map(lambda a: oracle.unpack_dequantize(a[1], min(chunk, n - a[0]), qp_o), zip(starts, packed)))
            t2 = time.perf_counter()
            out[f"quantize_pack@{bits}b"] = round(4.0 * n / (t1 - t0) / 1e9, 3)
            out[f"unpack_dequantize@{bits}b"] = round(4.0 * n / (t2 - t1) / 1e9, 3)
    out["unit"] = UNIT
    return out


def reference_main(args):
    """The CPU oracle as the reference arm: same metric, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    shape = si.CONFIGS[WORKLOAD]["shape"]
    n_full = int(np.prod(shape))
    bits_of_step = step_bits(n_full, oracle.select_bits)
    images = sample_images_for(args.steps + args.warmup)
    run_oracle_steps(0, args.warmup, bits_of_step, images)
    dt, n_sample = run_oracle_steps(args.warmup, args.steps, bits_of_step, images)
    gbs = args.steps * 4.0 * n_sample / dt / 1e9
    sample = sample_text(images, n_sample)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: fp32 {list(shape)} ViT-Huge activations, adaptive bits from a 100-step "
                               f"bandwidth trace; timed on a sample: {sample}"},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------- CUDA arm

def time_groups(torch, fn, nbuf, reps=20, warm=5, groups=5):
    """Median per-launch time (ms) over `groups` groups of `reps` back-to-back launches of fn(i % nbuf)
    (events around each group on the current stream, no host synchronisation inside a group)."""
    for i in range(warm):
        fn(i % nbuf)
    torch.cuda.synchronize()
    ts, k = [], warm
    for _ in range(groups):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn(k % nbuf)
            k += 1
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b) / reps)
    ts.sort()
    return ts[len(ts) // 2]


def cold_kernels(torch, qp, ctx, x_host, hbm_peak, peak_kind):
    """The metric's two kernels alone and cold: quantize+pack and unpack+dequantize on the workload at
    2, 4 and 8 bits, and on a 1 GiB tensor at 4 bits; on the workload also the statistics call (without and
    with the histogram) and the search call at 1-4 bits.  Consecutive launches use different input and
    output buffers, rotating through more than 4x the L2 capacity (126 MB) between reuses, so no
    launch finds its lines in L2."""
    out = {}

    def row(name, q, n, ms):
        alg = (4.0 + q / 8.0) * n
        g = alg / (ms * 1e-3) / 1e9
        out[f"{name}@{q}b"] = {"us": round(ms * 1e3, 2), "n": n, "gbs_fp32": round(4.0 * n / (ms * 1e-3) / 1e9, 1),
                               "achieved": round(g, 1), "unit": "GB/s", "frac": round(g / hbm_peak, 4),
                               "peak": hbm_peak, "peak_kind": peak_kind, "frac_of_8000": round(g / 8000.0, 4)}

    def read_row(name, n, ms):                                      # a stage whose algorithmic traffic is one read of x
        g = 4.0 * n / (ms * 1e-3) / 1e9
        out[name] = {"us": round(ms * 1e3, 2), "n": n, "achieved": round(g, 1), "unit": "GB/s",
                     "frac": round(g / hbm_peak, 4), "peak": hbm_peak, "peak_kind": peak_kind}

    def run(tag, xh, rot, widths, reductions=False):
        n = xh.numel()
        xs = [xh.cuda() for _ in range(rot)]
        ys = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(rot)]
        st = ctx.read_stats(ctx.qp_stats(xs[0]))
        if reductions:                                              # the statistics and the search call, alone too
            nb = qp.QP_DEFAULT_HIST_BINS
            d_st = [ctx.qp_stats(x, hist_bins=nb) for x in xs]
            d_res = torch.empty(72, dtype=torch.uint8, device="cuda")
            d_qp = torch.empty(24, dtype=torch.uint8, device="cuda")
            read_row(f"{tag}stats", n, time_groups(torch, lambda i: ctx.qp_stats(xs[i], hist_bins=0, out=d_st[i]), rot))
            read_row(f"{tag}stats+hist", n,
                     time_groups(torch, lambda i: ctx.qp_stats(xs[i], hist_bins=nb, out=d_st[i]), rot))
            for q in (1, 2, 3, 4):
                read_row(f"{tag}clip@{q}b", n, time_groups(
                    torch, lambda i: ctx.qp_dsaciq_search(xs[i], d_st[i], q, bmode=qp.QP_B_MAD | qp.QP_B_HIST_IN_STATS,
                                                          out_result=d_res, out_qp=d_qp), rot))
        for q in widths:
            _, _, qp_h = qp.qp_aciq_alpha(st, q)
            pk = [torch.empty(qp.qp_packed_bytes(n, q), dtype=torch.uint8, device="cuda") for _ in range(rot)]
            ms = time_groups(torch, lambda i: ctx.qp_quantize_pack(xs[i], q, qp_h, out=pk[i]), rot)
            row(f"{tag}quantize_pack", q, n, ms)
            ms = time_groups(torch, lambda i: ctx.qp_unpack_dequantize(pk[i], n, q, qp_h, out=ys[i]), rot)
            row(f"{tag}unpack_dequantize", q, n, ms)
            del pk
        del xs, ys
        torch.cuda.empty_cache()

    run("", x_host, 5, (2, 4, 8), reductions=True)                  # 5 x 129 MB in, 5 x 129 MB out
    big = torch.from_numpy(si.flat_iid(1 << 28, si.C5_SEED, "laplace"))
    run("2^28:", big, 2, (4,))                                       # every launch moves > 1 GiB: nothing survives in L2
    out["method"] = ("each kernel alone, buffers rotating through > 4x L2 between reuses; median per-launch time of 5 "
                     "groups of 20 back-to-back launches after 5 warm-ups; achieved = (4 + q/8) n bytes / time "
                     "(stats, stats+hist, clip: 4 n bytes / time of the whole call, graph replay as in the step)")
    return out


def ours_main(args):
    import torch
    import torch.distributed as dist

    import paper_2211_04515_b200 as qp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    hbm_peak, sm_max_mhz, peak_kind = peaks()

    cfg = si.CONFIGS[WORKLOAD]
    shape = cfg["shape"]
    n = int(np.prod(shape))
    bits_of_step = step_bits(n, qp.qp_select_bits)
    ctx = qp.Context(local)

    # inputs: ROT rotating copies so that a step never finds its input in L2 from the step before
    ROT = 3
    x_host = torch.empty(n, dtype=torch.float32, pin_memory=True)
    si.config_tensor(WORKLOAD, out=x_host.numpy())
    xs = [x_host.cuda(non_blocking=True) for _ in range(ROT)]
    max_packed = qp.qp_packed_bytes(n, 16)
    packed = torch.empty(max_packed, dtype=torch.uint8, device="cuda")
    y = torch.empty(n, dtype=torch.float32, device="cuda")
    d_stats = torch.empty(80, dtype=torch.uint8, device="cuda")
    d_qp = torch.empty(24, dtype=torch.uint8, device="cuda")
    d_res = torch.empty(72, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()

    assert all(qp.qp_stats_carries_histogram(x, qp.QP_DEFAULT_HIST_BINS) for x in xs)
    stage_names = ("stats", "clip", "quantize_pack", "unpack_dequantize")

    def step(t):
        # The step as a user runs it: the sender as the library's single call (statistics -> clip ->
        # quantize+pack, replayed as one recorded graph), then the receiver.  No events inside.
        q, x = bits_of_step[t % len(bits_of_step)], xs[t % ROT]
        ctx.qp_sender_device(x, q, qp.qp_policy_use_ds(q), out_packed=packed, out_qp=d_qp, out_stats=d_stats)
        ctx.qp_unpack_dequantize(packed, n, q, d_qp, out=y)

    def step_by_stage(t, events):
        # The same kernels called stage by stage with a CUDA event between the stages (each event makes
        # the stream drain, about 3.5 us): used only for the per-stage times, after the headline run.
        q, x = bits_of_step[t % len(bits_of_step)], xs[t % ROT]
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        marks[0].record()
        use_ds = qp.qp_policy_use_ds(q)
        ctx.qp_stats(x, out=d_stats, hist_bins=qp.QP_DEFAULT_HIST_BINS if use_ds else 0)
        marks[1].record()
        if use_ds:      # the statistics just written carry the histogram (checked above): the search need not look
            ctx.qp_dsaciq_search(x, d_stats, q, bmode=qp.QP_B_MAD | qp.QP_B_HIST_IN_STATS, out_result=d_res, out_qp=d_qp)
        else:
            ctx.qp_aciq_qparams_device(d_stats, q, out=d_qp)
        marks[2].record()
        ctx.qp_quantize_pack(x, q, d_qp, out=packed)
        marks[3].record()
        ctx.qp_unpack_dequantize(packed, n, q, d_qp, out=y)
        marks[4].record()
        events.append((q, marks))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # The step runs on a stream of its own with graph replay on: each multi-kernel call is recorded
    # once per (input buffer, bit-width) during warm-up and replayed afterwards.
    sampler = ClockSampler(local)
    sampler.start()                                      # before warm-up: the clocks of the whole run under load
    main_stream = torch.cuda.Stream()
    ctx.qp_set_graph_replay(True)
    torch.cuda.set_stream(main_stream)
    seen = set()
    for t in range(len(bits_of_step) * ROT):             # untimed: every (bit-width, input buffer) pair once, so that
        pair = (bits_of_step[t % len(bits_of_step)], t % ROT)   # every kernel is loaded and every graph recorded
        if pair not in seen:
            seen.add(pair)
            step(t)
            step_by_stage(t, [])
    for t in range(args.warmup):
        step(t)
    barrier()
    assert ctx.qp_get_status() & ~qp.QP_DEV_NONFINITE == 0

    # ---- timed region: exactly K steps between two events, bracketed by barrier + synchronize; the region
    # is repeated until MIN_TIMED_S of device time has been measured, and the median repeat is reported
    repeats = []
    launches = graph_hits = 0
    total_ms = 0.0
    while total_ms < MIN_TIMED_S * 1e3 and len(repeats) < 200:
        launches0, hits0 = ctx.qp_launch_count(), ctx.qp_graph_replays()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for t in range(args.warmup, args.warmup + args.steps):
            step(t)
        e1.record()
        barrier()
        ms_r = e0.elapsed_time(e1)
        _, ms_r = replica_throughput(ms_r, args.steps, 4.0 * n, world, "cuda")     # MAX over ranks
        repeats.append(ms_r)
        total_ms += ms_r
        launches = ctx.qp_launch_count() - launches0
        graph_hits = ctx.qp_graph_replays() - hits0
    ms = statistics.median(repeats)
    value = world * args.steps * 4.0 * n / (ms * 1e-3) / 1e9

    # ---- the same K steps with the receiver of step t beside the sender of step t + 1 (two streams, two
    # contexts, packed stream and quantizer double-buffered): what a pipeline stage sustains when it does not
    # wait for the far end.  Reported beside the headline, which stays the one-stream figure.
    pipelined = None
    if world == 1:
        ctx_r = qp.Context(local)
        side = torch.cuda.Stream()
        pk2 = [packed, torch.empty(max_packed, dtype=torch.uint8, device="cuda")]
        qp2 = [d_qp, torch.empty(24, dtype=torch.uint8, device="cuda")]
        free = [None, None]                                      # receiver done with buffer pair i

        def step2(t):
            q, x, i = bits_of_step[t % len(bits_of_step)], xs[t % ROT], t & 1
            if free[i] is not None:
                main_stream.wait_event(free[i])
            ctx.qp_sender_device(x, q, qp.qp_policy_use_ds(q), out_packed=pk2[i], out_qp=qp2[i], out_stats=d_stats)
            sent = torch.cuda.Event()
            sent.record(main_stream)
            side.wait_event(sent)
            with torch.cuda.stream(side):
                ctx_r.qp_unpack_dequantize(pk2[i], n, q, qp2[i], out=y)
                free[i] = torch.cuda.Event()
                free[i].record(side)

        for t in range(2 * len(bits_of_step) * ROT):            # untimed: graphs for the second buffer pair too
            step2(t)
        barrier()
        reps2, tot2 = [], 0.0
        while tot2 < MIN_TIMED_S * 1e3 and len(reps2) < 200:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(main_stream)
            for t in range(args.warmup, args.warmup + args.steps):
                step2(t)
            main_stream.wait_stream(side)
            e1.record(main_stream)
            barrier()
            reps2.append(e0.elapsed_time(e1))
            tot2 += reps2[-1]
        ms2 = statistics.median(reps2)
        assert ctx_r.qp_get_status() == 0
        pipelined = {"value": args.steps * 4.0 * n / (ms2 * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms2 / args.steps,
                     "repeats": len(reps2), "streams": 2,
                     "note": "receiver of step t on a second stream and context beside the sender of step t+1; "
                             "packed stream and quantizer double-buffered; not the headline"}
        del ctx_r

    # ---- per-stage device times: a separate instrumented pass over the trace (events between the stages)
    events = []
    inst_steps = max(args.steps, len(bits_of_step))
    for t in range(args.warmup, args.warmup + inst_steps):
        step_by_stage(t, events)
    barrier()
    clocks = sampler.stop()
    torch.cuda.set_stream(torch.cuda.default_stream())
    per = {}
    for q, m in events:
        for i, name in enumerate(stage_names):
            per.setdefault((name, q), []).append(m[i].elapsed_time(m[i + 1]))
    stage_ms = {name: sum(sum(v) for (nm, q), v in per.items() if nm == name) for name in stage_names}
    kernels = {}
    for (name, q), v in sorted(per.items()):
        avg = sum(v) / len(v)
        if name == "stats":
            bytes_alg = 4.0 * n
        elif name == "quantize_pack" or name == "unpack_dequantize":
            bytes_alg = (4.0 + q / 8.0) * n
        else:
            bytes_alg = None
        key = f"{name}@{q}b"
        if bytes_alg is not None:
            gbs = bytes_alg / (avg * 1e-3) / 1e9
            kernels[key] = {"ms": round(avg, 4), "bound": "hbm", "achieved": round(gbs, 1), "peak": hbm_peak,
                            "unit": "GB/s", "frac": round(gbs / hbm_peak, 4), "calls": len(v)}
            if name != "stats":
                kernels[key]["note"] = ("in the chain, L2-warm: the pass before it left part of x (of the packed stream) "
                                        "in L2; the cold figures are in kernels_cold")
        elif qp.qp_policy_use_ds(q):
            # the search reads x once (interval moments); it is limited by shared-memory atomics, and
            # is reported against the HBM time of that one pass
            gbs = 4.0 * n / (avg * 1e-3) / 1e9
            kernels[key] = {"ms": round(avg, 4), "bound": "hbm", "achieved": round(gbs, 1), "peak": hbm_peak,
                            "unit": "GB/s", "frac": round(gbs / hbm_peak, 4), "calls": len(v),
                            "note": "one read of x is the algorithmic traffic; limited by instruction issue and shared-memory atomics"}
        else:
            kernels[key] = {"ms": round(avg, 4), "calls": len(v)}
    # the dominant kernel of the step (largest share of device time)
    dom = max(stage_ms, key=stage_ms.get)
    dom_keys = [k for k in kernels if k.startswith(dom + "@") and "achieved" in kernels[k]]
    tot_ms = sum(kernels[k]["ms"] * kernels[k]["calls"] for k in dom_keys)
    ach = sum(kernels[k]["achieved"] * kernels[k]["ms"] * kernels[k]["calls"] for k in dom_keys) / tot_ms
    first = kernels[dom_keys[0]]
    traffic, traffic_source = traffic_of(dom)
    roofline = {"kernel": dom, "bound": first["bound"], "achieved": round(ach, 3), "peak": first["peak"],
                "unit": first["unit"], "frac": round(ach / first["peak"], 4), "peak_kind": peak_kind,
                "traffic": traffic, "traffic_source": traffic_source,
                "share_of_step_time": round(stage_ms[dom] / sum(stage_ms.values()), 3),
                "measured": f"CUDA events around the stage's call on the launching stream, {inst_steps} instrumented steps "
                            "after the headline run (algorithmic bytes per call / average call time)"}

    # ---- the metric's kernels alone and cold (rank 0 of a 1-GPU run: it needs ~5 GB of buffers)
    cold = None
    if rank == 0 and world == 1 and not args.no_cold:
        cold = cold_kernels(torch, qp, ctx, x_host, hbm_peak, peak_kind)

    # ---- end to end through the host-buffer entry points (pinned host memory, copies timed).
    # Sender and receiver are two parties with their own context, stream and buffers, as on two
    # pipeline stages; the receiver of step t-1 runs while the sender of step t does, so the
    # host->device copy of one tensor overlaps the device->host copy of the previous one.
    e2e_steps = max(3, min(args.steps, 40))
    ctx_r = qp.Context(local)
    s_send, s_recv = torch.cuda.Stream(), torch.cuda.Stream()
    SLOTS = 4                                                # host slots for packed stream + quantizer in flight
    h_packed = [torch.empty(max_packed, dtype=torch.uint8, pin_memory=True) for _ in range(SLOTS)]
    h_qps = [qp.QParams() for _ in range(SLOTS)]
    sent = [torch.cuda.Event() for _ in range(SLOTS)]
    consumed = [torch.cuda.Event() for _ in range(SLOTS)]
    h_y = torch.empty(n, dtype=torch.float32, pin_memory=True)
    d_x_work = xs[0]
    packed_r = torch.empty(max_packed, dtype=torch.uint8, device="cuda")

    def send(t):
        q = bits_of_step[t % len(bits_of_step)]
        with torch.cuda.stream(s_send):
            ctx.qp_sender_host(x_host, q, qp.qp_policy_use_ds(q), d_x_work, packed, h_packed[t % SLOTS],
                               h_qps[t % SLOTS])
            sent[t % SLOTS].record()
        return 4 * n + qp.qp_packed_bytes(n, q), qp.qp_packed_bytes(n, q) + 24

    def receive(t):
        q = bits_of_step[t % len(bits_of_step)]
        sent[t % SLOTS].synchronize()                        # packed stream and quantizer are on the host
        with torch.cuda.stream(s_recv):
            ctx_r.qp_receiver_host(h_packed[t % SLOTS], n, q, h_qps[t % SLOTS], packed_r, y, h_y)
            consumed[t % SLOTS].record()
        return qp.qp_packed_bytes(n, q), 4 * n

    def e2e_run(first, count):
        h2d = d2h = 0
        for t in range(first, first + count):
            if t >= first + SLOTS:
                consumed[t % SLOTS].synchronize()            # the receiver is done with this slot
            if t > first:                                    # receiver first: its small copy-in does not queue
                a, b = receive(t - 1)                        # behind the sender's large one
                h2d, d2h = h2d + a, d2h + b
            a, b = send(t)
            h2d, d2h = h2d + a, d2h + b
        a, b = receive(first + count - 1)
        s_send.synchronize()
        s_recv.synchronize()
        return h2d + a, d2h + b

    e2e_run(0, 3)
    barrier()
    t0 = time.perf_counter()
    h2d, d2h = e2e_run(args.warmup, e2e_steps)
    e2e_ms = (time.perf_counter() - t0) * 1e3                # spans two streams: wall clock, both synchronised
    barrier()
    e2e_value, e2e_ms = replica_throughput(e2e_ms, e2e_steps, 4.0 * n, world, "cuda")
    e2e = {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms / e2e_steps,
           "h2d_bytes_per_step": h2d // e2e_steps, "d2h_bytes_per_step": d2h // e2e_steps, "steps": e2e_steps,
           "overlap": "receiver of step t-1 runs beside the sender of step t (two streams, two contexts)"}
    ctx_r.close()

    # ---- CPU oracle beside it (rank 0, N=1 only): bounded sample, same trace; 1 thread for the whole
    # step, and the two element-wise stages also chunk-parallel on every host core
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_steps = 16
        images = sample_images_for(cpu_steps)
        dt, n_sample = run_oracle_steps(args.warmup, cpu_steps, bits_of_step, images)
        cpu = {"value": cpu_steps * 4.0 * n_sample / dt / 1e9, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(),
               "kind": "oracle", "sample": f"{cpu_steps} steps: " + sample_text(images, n_sample) + f", {dt:.1f} s",
               "all_cores": oracle_all_cores(x_host.numpy())}

    if rank == 0:
        med_mhz = clocks.get("sm_mhz")
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: fp32 {list(shape)} ViT-Huge activations (129 MB), adaptive bits "
                                   f"{list(si.C4_ALLOWED_BITS)} from a seeded 100-step bandwidth trace, search at <=4 bits",
                       "replicas": world, "l2": f"inputs larger than L2 (129 MB > 126 MB), {ROT} rotating input buffers",
                       "bits_mix": {str(b): bits_of_step.count(b) for b in sorted(set(bits_of_step))},
                       "timed_region": f"{args.steps} steps (qp_sender_device + qp_unpack_dequantize per step, no events "
                                       f"inside) between two events, repeated {len(repeats)} times "
                                       f"({total_ms:.0f} ms of device time); ms_per_step is the median repeat",
                       "stage_events": f"per-stage times from {inst_steps} separately instrumented steps after the timed "
                                       "region (qp_stats / clip / qp_quantize_pack / qp_unpack_dequantize one by one, an "
                                       "event between them)",
                       "graph_replay": f"on: {graph_hits} multi-kernel calls of one timed region replayed a graph "
                                       "recorded in warm-up"},
            "repeats_ms_per_step": {"min": round(min(repeats) / args.steps, 5), "median": round(ms / args.steps, 5),
                                    "max": round(max(repeats) / args.steps, 5), "count": len(repeats)},
            "ms_per_step_x_sm_mhz": round(ms / args.steps * med_mhz, 2) if med_mhz else None,
            "roofline": roofline, "kernels": kernels, "kernels_cold": cold, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks, "pipelined": pipelined,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    ctx.close()
    return 0


# ------------------------------------------------------------- kernel-by-kernel sweep

def sweep_main(args):
    """Each stage timed alone, cold: the buffers of consecutive launches rotate through more than
    4x the L2 capacity, so no launch finds its input (or output lines) in L2.  One JSON line per
    (workload, dtype, stage, bits): median and best per-launch time over 5 groups of 20
    back-to-back launches after 5 warm-ups."""
    import torch

    import paper_2211_04515_b200 as qp

    assert torch.cuda.is_available(), "the sweep needs a CUDA device"
    torch.cuda.set_device(0)
    hbm_peak, _, peak_kind = peaks()
    ctx, gctx = qp.Context(0), qp.Context(0)
    side = torch.cuda.Stream()
    L2_BYTES = 126e6

    def rotating(make, nbytes):
        count = max(2, int(4 * L2_BYTES // max(nbytes, 1)) + 1)
        return [make() for _ in range(min(count, 64))]

    def timed(fn, nbuf, reps=20, warm=5, groups=5):
        """Median and best per-launch time over `groups` groups of `reps` back-to-back launches
        (events around each group, no host synchronisation inside a group, so the device never
        waits for the host)."""
        for i in range(warm):
            fn(i % nbuf)
        torch.cuda.synchronize()
        ts, k = [], warm
        for _ in range(groups):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn(k % nbuf)
                k += 1
            b.record()
            b.synchronize()
            ts.append(a.elapsed_time(b) / reps)
        ts.sort()
        return ts[len(ts) // 2], ts[0]

    def emit(workload, dtype, stage, bits, n, med, best, alg_bytes):
        row = {"sweep": True, "workload": workload, "dtype": dtype, "stage": stage, "bits": bits, "n": n,
               "us_median": round(med * 1e3, 2), "us_best": round(best * 1e3, 2),
               "gbs_in": round(4.0 * n / (med * 1e-3) / 1e9, 1) if dtype == "f32" else round(2.0 * n / (med * 1e-3) / 1e9, 1)}
        if alg_bytes is not None:
            g = alg_bytes / (med * 1e-3) / 1e9
            row.update({"alg_gbs": round(g, 1), "frac_of_measured_peak": round(g / hbm_peak, 3),
                        "frac_of_8000": round(g / 8000.0, 3), "peak_kind": peak_kind})
        print(json.dumps(row), flush=True)

    def run_workload(name, x_host, bits_list, dtype="f32", search_bits=(), channels=0):
        n = x_host.numel()
        esz = 4 if dtype == "f32" else 2
        xs = rotating(lambda: x_host.cuda(), n * esz)
        nb = len(xs)
        d_stats = [torch.empty(80, dtype=torch.uint8, device="cuda") for _ in range(nb)]
        med, best = timed(lambda i: ctx.qp_stats(xs[i], out=d_stats[i]), nb)
        emit(name, dtype, "stats", 0, n, med, best, esz * n)
        med, best = timed(lambda i: ctx.qp_stats(xs[i], out=d_stats[i], hist_bins=100), nb)
        emit(name, dtype, "stats+hist100", 0, n, med, best, esz * n)
        st = ctx.read_stats(d_stats[0])
        d_qp = torch.empty(24, dtype=torch.uint8, device="cuda")
        d_res = torch.empty(72, dtype=torch.uint8, device="cuda")
        for q in search_bits:
            med, best = timed(lambda i: ctx.qp_dsaciq_search(xs[i], d_stats[i], q, out_result=d_res, out_qp=d_qp), nb)
            emit(name, dtype, "dsaciq_search", q, n, med, best, esz * n)
        # the sender in one call (statistics -> clip -> quantize+pack): the kernel chain and, for small
        # tensors, the single cooperative launch; each launched directly and as a recorded graph (one
        # graph per input buffer, on a stream of its own)
        for q, use_ds in ((2, True), (8, False)):
            pk = [torch.empty(qp.qp_packed_bytes(n, q), dtype=torch.uint8, device="cuda") for _ in range(nb)]
            call = lambda c: (lambda i: c.qp_sender_device(xs[i], q, use_ds, out_packed=pk[i], out_qp=d_qp,
                                                           out_stats=d_stats[i]))
            paths = [("chain", qp.QP_SENDER_CHAIN)] + ([("fused", qp.QP_SENDER_FUSED)] if n <= (1 << 20) else [])
            for label, path in paths:
                stage = f"sender_device[{label}{', search' if use_ds else ''}]"
                ctx.qp_set_sender_path(path)
                med, best = timed(call(ctx), nb)
                emit(name, dtype, stage, q, n, med, best, None)
                ctx.qp_set_sender_path(qp.QP_SENDER_AUTO)
                torch.cuda.synchronize()
                gctx.qp_set_sender_path(path)
                with torch.cuda.stream(side):
                    gctx.qp_set_graph_replay(True)
                    med, best = timed(call(gctx), nb, warm=nb + 5)
                    gctx.qp_set_graph_replay(False)           # drops this workload's graphs
                emit(name, dtype, stage + "+graph", q, n, med, best, None)
            del pk
        # channel-wise variant ([rows, channels], one quantizer per channel), ViT-shaped workloads only
        if channels:
            d_cst = torch.empty(80 * channels, dtype=torch.uint8, device="cuda")
            med, best = timed(lambda i: ctx.qp_stats_channels(xs[i], channels, out=d_cst), nb)
            emit(name, dtype, f"stats_channels[{channels}]", 0, n, med, best, esz * n)
            d_cres = torch.empty(72 * channels, dtype=torch.uint8, device="cuda")
            d_csqp = torch.empty(24 * channels, dtype=torch.uint8, device="cuda")
            for q in (2, 4):                  # every candidate scored on every element: fp32-ALU-bound
                med, best = timed(lambda i: ctx.qp_dsaciq_search_channels(xs[i], channels, d_cst, q, out_result=d_cres,
                                                                          out_qp=d_csqp), nb)
                emit(name, dtype, f"dsaciq_search_channels[{channels}]", q, n, med, best, esz * n)
            for q in (4, 8):
                d_cqp = ctx.qp_clip_qparams_channels_device(d_cst, channels, q)
                pk = rotating(lambda: torch.empty(qp.qp_packed_bytes(n, q), dtype=torch.uint8, device="cuda"),
                              n * esz + qp.qp_packed_bytes(n, q))
                npk = len(pk)
                med, best = timed(lambda i: ctx.qp_quantize_pack_channels(xs[i % nb], channels, q, d_cqp, out=pk[i % npk]),
                                  max(nb, npk))
                emit(name, dtype, f"quantize_pack_channels[{channels}]", q, n, med, best, (esz + q / 8.0) * n)
                if dtype == "f32":
                    ysc = rotating(lambda: torch.empty(n, dtype=torch.float32, device="cuda"), 4 * n)
                    nyc = len(ysc)
                    med, best = timed(lambda i: ctx.qp_unpack_dequantize_channels(pk[i % npk], n // channels, channels, q,
                                                                                  d_cqp, out=ysc[i % nyc]), max(nyc, npk))
                    emit(name, dtype, f"unpack_dequantize_channels[{channels}]", q, n, med, best, (4 + q / 8.0) * n)
                    del ysc
                del pk
            # token-wise variant (one quantizer per row of `channels` contiguous elements)
            tokens = n // channels
            d_tst = torch.empty(80 * tokens, dtype=torch.uint8, device="cuda")
            med, best = timed(lambda i: ctx.qp_stats_tokens(xs[i], channels, out=d_tst), nb)
            emit(name, dtype, f"stats_tokens[{tokens}]", 0, n, med, best, esz * n)
            for q in (4, 8):
                d_tqp = ctx.qp_clip_qparams_tokens_device(d_tst, tokens, q)
                pk = rotating(lambda: torch.empty(qp.qp_packed_bytes(n, q), dtype=torch.uint8, device="cuda"),
                              n * esz + qp.qp_packed_bytes(n, q))
                npk = len(pk)
                med, best = timed(lambda i: ctx.qp_quantize_pack_tokens(xs[i % nb], channels, q, d_tqp, out=pk[i % npk]),
                                  max(nb, npk))
                emit(name, dtype, f"quantize_pack_tokens[{tokens}]", q, n, med, best, (esz + q / 8.0) * n)
                if dtype == "f32":
                    yst = rotating(lambda: torch.empty(n, dtype=torch.float32, device="cuda"), 4 * n)
                    nyt = len(yst)
                    med, best = timed(lambda i: ctx.qp_unpack_dequantize_tokens(pk[i % npk], tokens, channels, q, d_tqp,
                                                                                out=yst[i % nyt]), max(nyt, npk))
                    emit(name, dtype, f"unpack_dequantize_tokens[{tokens}]", q, n, med, best, (4 + q / 8.0) * n)
                    del yst
                del pk
        ys = None
        for q in bits_list:
            rc, alpha, qp_h = qp.qp_aciq_alpha(st, q)
            pk = rotating(lambda: torch.empty(qp.qp_packed_bytes(n, q), dtype=torch.uint8, device="cuda"),
                          n * esz + qp.qp_packed_bytes(n, q))
            npk = len(pk)
            med, best = timed(lambda i: ctx.qp_quantize_pack(xs[i % nb], q, qp_h, out=pk[i % npk]), max(nb, npk))
            emit(name, dtype, "quantize_pack", q, n, med, best, (esz + q / 8.0) * n)
            if dtype == "f32":
                if ys is None:
                    ys = rotating(lambda: torch.empty(n, dtype=torch.float32, device="cuda"), 4 * n)
                ny = len(ys)
                med, best = timed(lambda i: ctx.qp_unpack_dequantize(pk[i % npk], n, q, qp_h, out=ys[i % ny]), max(ny, npk))
                emit(name, dtype, "unpack_dequantize", q, n, med, best, (4 + q / 8.0) * n)
            del pk
        del xs, ys
        torch.cuda.empty_cache()

    only = set(args.sweep_only.split(",")) if args.sweep_only else None
    for name in ("c1", "c2", "c3", "c4"):
        if only is not None and name not in only:
            continue
        cfg = si.CONFIGS[name]
        x = torch.from_numpy(si.config_tensor(name).reshape(-1))
        run_workload(name, x, cfg["bits"], "f32", [b for b in cfg["bits"] if b <= 4][:2], channels=cfg["shape"][-1])
    for log2n in range(18, args.sweep_max_log2 + 1, 2):
        if only is not None and f"2^{log2n}" not in only:
            continue
        for dist in ("laplace", "normal"):
            if dist == "normal" and log2n not in (22, 26):
                continue
            x = torch.from_numpy(si.flat_iid(1 << log2n, si.C5_SEED, dist))
            run_workload(f"c5-{dist}-2^{log2n}", x, si.C5_BITS, "f32", (2,) if dist == "laplace" else ())
            if dist == "laplace" and log2n in (22, 26):
                run_workload(f"c5-{dist}-2^{log2n}", x.to(torch.bfloat16), (2, 4, 8, 16), "bf16")
    ctx.close()
    gctx.close()
    return 0


def quality_main(args):
    """Quantization error of the clip methods on the ViT-shaped configs (context for the paper's Sec. 3
    claim that the directed search lowers the MSE of ACIQ): every number is the MSE between the tensor
    and what the receiver reconstructs, measured on the device from the library's own output."""
    import torch

    import paper_2211_04515_b200 as qp

    if not torch.cuda.is_available():
        raise SystemExit("bench.py --quality needs a CUDA device")
    ctx = qp.Context(0)
    for name in ("c2", "c3"):
        shape = si.CONFIGS[name]["shape"]
        channels = shape[-1]
        x = torch.from_numpy(si.config_tensor(name).reshape(-1)).cuda()
        n = x.numel()
        rows = n // channels

        def mse_of(y):
            return float(((y.double() - x.double()) ** 2).mean())

        for q in (2, 4, 8):
            row = {"quality": True, "workload": name, "bits": q}
            d_stats = ctx.qp_stats(x)
            for label, method in (("naive_minmax", qp.QP_CLIP_MINMAX), ("aciq", qp.QP_CLIP_ACIQ)):
                d_qp = ctx.qp_clip_qparams_device(d_stats, q, method)
                y = ctx.qp_unpack_dequantize(ctx.qp_quantize_pack(x, q, d_qp), n, q, d_qp)
                row[label] = mse_of(y)
            for nb in (100, 2048):
                d_sh = ctx.qp_stats(x, hist_bins=nb)
                d_res, d_qp = ctx.qp_dsaciq_search(x, d_sh, q, hist_bins=nb)
                res = ctx.read_ds_result(d_res)
                y = ctx.qp_unpack_dequantize(ctx.qp_quantize_pack(x, q, d_qp), n, q, d_qp)
                row[f"ds_nb{nb}"] = {"mse_e": res.mse_e, "mse_star": res.mse_star, "k_star": res.k_star,
                                     "b_r_over_b_e": res.b_r / res.b_e, "measured": mse_of(y)}
            d_cst = ctx.qp_stats_channels(x, channels)
            d_cqp = ctx.qp_clip_qparams_channels_device(d_cst, channels, q)
            y = ctx.qp_unpack_dequantize_channels(ctx.qp_quantize_pack_channels(x, channels, q, d_cqp), rows, channels, q, d_cqp)
            row["channels_aciq"] = mse_of(y)
            _, d_cqp = ctx.qp_dsaciq_search_channels(x, channels, d_cst, q)
            y = ctx.qp_unpack_dequantize_channels(ctx.qp_quantize_pack_channels(x, channels, q, d_cqp), rows, channels, q, d_cqp)
            row["channels_ds"] = mse_of(y)
            print(json.dumps(row))
    ctx.qp_get_status()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cold", action="store_true", help="skip the kernels_cold object (it needs ~5 GB of buffers)")
    ap.add_argument("--quality", action="store_true",
                    help="print the quantization MSE of every clip method on the ViT-shaped configs (one GPU)")
    ap.add_argument("--sweep", action="store_true",
                    help="kernel-by-kernel cold-cache table over the configurations (one JSON line per row)")
    ap.add_argument("--sweep-only", default="",
                    help="comma-separated workloads of the sweep to run (c1..c4, 2^18..2^28); default: all")
    ap.add_argument("--sweep-max-log2", type=int, default=28)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return reference_main(args)
    if args.quality:
        return quality_main(args)
    if args.sweep:
        return sweep_main(args)
    return ours_main(args)


if __name__ == "__main__":
    sys.exit(main())
