"""The multi-rank side of bench.py on CPU (gloo, two ranks).  The path shards by independent
replicas only, so there is no data-path collective to test: what the ranks share is the timing
reduction (max over ranks), the whole-job value, and the rule that rank 0 alone prints."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = [3.0, 7.5][rank]                       # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.job_value(1e12, world, ms))
    dist.destroy_process_group()


def test_max_over_ranks_and_job_value_gloo():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        got = dict(out)
    assert got[0] == got[1]                           # every rank sees the slowest rank's time
    ms, value = got[0]
    assert ms == 7.5
    assert value == pytest.approx(2 * 1e12 / 7.5e-3 / 1e12)   # two replicas' work in the slowest rank's time


def test_without_a_process_group_the_value_passes_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, torch.device("cpu")) == 1.25


def test_reference_arm_under_two_ranks_prints_one_line():
    """`bench.py --impl reference` launched as two ranks: rank 0 alone runs and prints."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
           "--config", "1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0
