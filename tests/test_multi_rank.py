"""The benchmark's N > 1 path on CPU: two gloo ranks.

The hot path has no exchange between GPUs (replicas only), so what the ranks share is the
measurement protocol: max-over-ranks times, min-over-ranks health, whole-job rate, and the
reference arm printing from rank 0 only.
"""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2601_09093_b200 import ranks as R
    assert R.rank_env() == (rank, rank, world)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slow one for the first time, rank 0 for the second; rank 1 reports a device error
    times = [10.0 + 5.0 * rank, 3.0 - rank]
    vals, ok = R.max_over_ranks(times, ok=(rank == 0), device="cpu")
    vals2, ok2 = R.max_over_ranks([1.0 + rank], ok=True, device="cpu")
    dist.barrier()
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"vals": vals, "ok": ok, "vals2": vals2, "ok2": ok2,
                   "rate": R.whole_job_rate(64 * 10, world, vals[0] * 1e-3)}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_times_and_min_health(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(world)]
    for g in got:
        assert g["vals"] == [15.0, 3.0]          # the slowest rank's time, per entry
        assert g["ok"] is False                  # one unhealthy rank fails the job
        assert g["vals2"] == [2.0] and g["ok2"] is True
        assert abs(g["rate"] - 2 * 640 / 15e-3) < 1e-6      # weak scaling: all ranks' units over the max time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2601_09093_b200 import ranks as R
    assert R.max_over_ranks([1.5, 2.5], True, "cpu") == ([1.5, 2.5], True)
    assert R.whole_job_rate(64, 1, 0.5) == 128.0


def test_reference_arm_prints_once_under_a_two_rank_launcher():
    """`bench.py --impl reference` under torchrun: rank 0 prints the line, rank 1 exits 0 without work."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "scorer",
           "--gpus", "2", "--steps", "1", "--warmup", "1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
