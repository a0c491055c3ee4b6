"""The N > 1 path of bench.py on CPU: two gloo ranks agree on the max-over-ranks time and the replica
throughput (the path has no exchange step, so ranks are independent replicas; only the timing is reduced)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms = 10.0 + 5.0 * rank                      # rank 1 is slower
    red = bench.reduce_max_ms(ms, torch.device("cpu"), world)
    value = bench.replica_throughput(tokens=32, steps=4, world=world, ms_total=red)
    print(json.dumps({"rank": rank, "ms": red, "value": value}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_reduce_timing_to_the_slowest():
    import socket
    with socket.socket() as sock:                  # a port nobody holds right now
        sock.bind(("127.0.0.1", 0))
        port = str(sock.getsockname()[1])
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
    import tempfile
    with tempfile.NamedTemporaryFile("w", suffix=".py", delete=False) as f:
        f.write(WORKER)
        path = f.name
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", port, path]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=240)
    os.unlink(path)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    import re
    rows = [json.loads(o) for o in re.findall(r"\{[^{}]*\}", out.stdout)]      # two ranks share one pipe: lines may run together
    assert len(rows) == 2
    for r in rows:
        assert r["ms"] == 15.0                                  # max over ranks
        assert abs(r["value"] - 2 * 32 * 4 / 15e-3) < 1e-6      # units of all ranks / slowest time


def test_block_statistics_and_traffic_ratio_helpers():
    """Host logic of bench.py that needs no GPU: the median / best block arithmetic and the lookup of the DRAM-traffic
    ratio recorded with the ncu capture."""
    sys.path.insert(0, ROOT)
    import bench
    st = bench.block_stats([10.0, 12.0, 11.0, 30.0], steps=20)
    assert st["blocks"] == 4 and abs(st["ms_per_step"] - 11.5 / 20) < 1e-12 and abs(st["ms_per_step_best"] - 0.5) < 1e-12
    assert abs(st["timed_seconds"] - 0.063) < 1e-12
    r = bench.traffic_ratio("k_ffn_up_gate")
    assert r is not None and 1.0 <= r["ratio"] < 1.1 and r["source"].startswith("profiles/")
    assert bench.traffic_ratio("no_such_kernel") is None
    hbm, sustained, burst, src = bench.peaks()
    assert hbm > 1000 and burst >= sustained > 100 and src in ("measured", "fallback")
