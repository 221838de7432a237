"""The path does not shard: N GPUs run N independent replicas and only the timing is reduced (maximum over
ranks).  This exercises that reduction and the reference arm's rank rule with two gloo ranks on CPU."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


_WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["TJ_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
mx = bench.max_over_ranks([10.0 + rank, 5.0 - rank], "cpu")
mn = bench.min_over_ranks([7.0 + rank], "cpu")
assert mx == [11.0, 5.0] and mn == [7.0], (mx, mn)
# two replicas of 1000 units each, the slower one took 11 ms
assert abs(bench.aggregate_throughput(1000, 2, mx[0]) - 2000 / 0.011) < 1e-6
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_timing_reduction_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    env = dict(os.environ, TJ_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()), WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "rank 0 ok" in outs[0] and "rank 1 ok" in outs[1]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                          "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                          "--steps", "2", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=120)
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["n_gpus"] == 2


def test_gpus_flag_must_agree_with_the_launcher():
    """`--gpus N` under a launcher that started another number of ranks is an error, not a silent single-GPU run."""
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "1"], env=env,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode != 0 and "--gpus 4" in (out.stderr + out.stdout) and "2 ranks" in (out.stderr + out.stdout)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], env=env, capture_output=True,
                         text=True, timeout=120)
    assert out.returncode != 0 and "2 ranks" in (out.stderr + out.stdout)
