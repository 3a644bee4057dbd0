"""The benchmark's N > 1 plumbing on CPU: two `gloo` ranks, barrier, MAX of per-rank times, aggregate value.

The data path has no collective (chunks are independent: replicas only), so this is all there is to test
for more than one GPU; it runs without any."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import bench
r = bench.Ranks("gloo", "cpu")
r.barrier()
seconds = 1.0 + r.rank            # rank 0 took 1 s, rank 1 took 2 s
slowest = r.max_over_ranks(seconds)
value = r.aggregate_throughput(10_000, seconds)
r.barrier()
print(json.dumps({{"rank": r.rank, "world": r.world, "slowest": slowest, "value": value}}))
r.close()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_max_time_and_aggregate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, _ = p.communicate(timeout=240)
        assert p.returncode == 0
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["world"] == 2
        assert o["slowest"] == pytest.approx(2.0)                 # max over ranks, not this rank's own time
        assert o["value"] == pytest.approx(2 * 10_000 / 2.0)      # all ranks' bytes over the slowest rank's time
    assert sorted(o["rank"] for o in outs) == [0, 1]


def test_reference_arm_runs_on_rank_zero_only():
    """`--impl reference` under a 2-rank launch: rank 0 prints the line, the other rank exits 0 silently."""
    env1 = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env1, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env0, capture_output=True, text=True, timeout=480)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
