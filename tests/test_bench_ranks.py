"""The multi-rank plumbing of bench.py on CPU (gloo, two ranks): the path has no exchange between
GPUs, so N ranks are N replicas; what the ranks share is the barrier, the max-over-ranks time and the
rule that rank 0 alone prints.  No device work."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


_WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
dist.barrier()
ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
ms_max = bench.max_over_ranks(ms, world, torch.device("cpu"))
val = bench.job_value(1000, 4, ms_max, world)
dist.barrier()
if rank == 0:
    print(json.dumps({"ms_max": ms_max, "value": val}))
dist.destroy_process_group()
"""


def test_max_over_ranks_and_job_value_two_gloo_ranks(tmp_path):
    port = _free_port()
    script = tmp_path / "w.py"
    script.write_text(_WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert outs[1][0].strip() == ""                      # only rank 0 prints
    got = json.loads(outs[0][0].strip())
    assert got["ms_max"] == 15.0
    assert got["value"] == pytest.approx(2 * 1000 * 4 / 15e-3)


def test_reference_arm_runs_on_rank0_only():
    """Under a multi-rank launch the oracle-timing arm runs on rank 0; other ranks exit 0 silently."""
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "c1_single_1024"], env=env, capture_output=True, text=True,
                       timeout=240)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env["RANK"] = "0"
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "c1_single_1024", "--reference-budget", "2"], env=env,
                       capture_output=True, text=True, timeout=240)
    assert p.returncode == 0, p.stderr
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` with no launcher around it starts two ranks; exactly one line comes out and it
    says n_gpus = 2 (here on the oracle-timing arm, which needs no GPU)."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                        "--steps", "1", "--warmup", "0", "--workload", "c1_single_1024", "--reference-budget", "2"],
                       env=env, capture_output=True, text=True, timeout=240)
    assert p.returncode == 0, p.stderr
    lines = [l for l in p.stdout.strip().splitlines() if l.strip()]
    assert len(lines) == 1, lines
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["impl"] == "reference"
