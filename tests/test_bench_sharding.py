"""Host logic of the multi-GPU bench: the path does not shard (replicas only), so N ranks run N
independent verify calls and the job figure is world * steps / (slowest rank's time).  Checked
with two gloo ranks on CPU; no GPU and no library call is involved."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
local_ms = [120.0, 200.0][rank]                      # rank 1 is the slow replica
value, ms_step = bench.aggregate_calls_per_s(local_ms, steps=100, world=world)
slowest = bench.max_over_ranks(float(rank + 1), world)
print(json.dumps(dict(rank=rank, value=value, ms_step=ms_step, slowest=slowest)), flush=True)
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_report_the_slowest_replica():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=str(ROOT))], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for pr in procs:
        out, err = pr.communicate(timeout=180)
        assert pr.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    for o in outs:                                   # both ranks agree on the job figure
        assert abs(o["ms_step"] - 2.0) < 1e-12       # 200 ms / 100 steps: the slow rank decides
        assert abs(o["value"] - 2 * 100 / 0.2) < 1e-6
        assert o["slowest"] == 2.0


def test_plain_python_invocation_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it: the script spawns two ranks, they
    aggregate over gloo (stub step, no GPU), and exactly one JSON line with n_gpus = 2 comes back."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    env.update(DM_BENCH_STUB="1", DM_BENCH_BACKEND="gloo")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--steps", "10", "--warmup", "3"],
                       env=env, capture_output=True, text=True, timeout=180)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2
    assert abs(line["ms_per_step"] - 20.0) < 1e-9          # the slow stub rank: 200 ms over 10 steps
    assert abs(line["value"] - 2 * 10 / 0.2) < 1e-6


def test_single_rank_needs_no_process_group():
    import bench
    value, ms_step = bench.aggregate_calls_per_s(50.0, steps=10, world=1)
    assert ms_step == 5.0 and abs(value - 200.0) < 1e-9


def test_reference_arm_only_rank_zero_works():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
