"""bench.py's N > 1 path on the CPU: two gloo ranks (replicas of the batch shard, no data-path collective)
agree on the max-over-ranks time and the whole-job throughput; the reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_share_the_slowest_time(tmp_path):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "tests", "ranks_worker.py"), str(tmp_path)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    r = [json.load(open(tmp_path / ("rank%d.json" % i))) for i in range(2)]
    assert [x["seed"] for x in r] == [0, 1]                 # each rank owns a different shard
    assert r[0]["total_ms"] == r[1]["total_ms"] == 20.0     # the slowest rank's time, on every rank
    # 2 ranks x 5 steps x 1e12 ops in 20 ms -> 500 TOPS for the whole job
    assert abs(r[0]["tops"] - 500.0) < 1e-9 and r[0]["tops"] == r[1]["tops"]


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""
