"""Host-side logic of bench.py that needs no GPU: the aggregation over replicas (two gloo
ranks on CPU), the bit-width trace of the workload, and the reference arm's JSON line."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
import oracle  # noqa: E402
import synth_inputs as si  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow replica
    gbs, ms = bench.replica_throughput(local_ms, steps=5, bytes_per_step=1e9, world=world)
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"gbs": gbs, "ms": ms}, f)
    dist.destroy_process_group()


def test_replicas_aggregate_with_max_over_ranks(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    for g in got:                                               # every rank sees the slowest rank's time
        assert g["ms"] == 25.0
        assert g["gbs"] == pytest.approx(world * 5 * 1e9 / 25e-3 / 1e9)
    gbs1, ms1 = bench.replica_throughput(10.0, 5, 1e9, 1)       # single replica: no collective
    assert ms1 == 10.0 and gbs1 == pytest.approx(500.0)


def test_trace_bits_cover_the_allowed_widths():
    n = 128 * 197 * 1280
    bits = bench.step_bits(n, oracle.select_bits)
    assert len(bits) == si.C4_TRACE_STEPS
    assert set(bits) <= set(si.C4_ALLOWED_BITS) and {1, 2, 3, 4, 6, 8} <= set(bits)
    assert 16 not in bits                                       # never fits the 2 s budget on this trace


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "3"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    # ranks other than 0 print nothing and exit 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2"],
                         capture_output=True, text=True, timeout=60, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
