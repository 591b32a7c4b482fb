"""The multi-rank plumbing of bench.py on CPU: batch sharding over ranks, the max-over-ranks
reduction (gloo, world size 2) and the reference arm's launch contract under torchrun."""
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


def _free_port():
    """A TCP port nobody listens on right now (asked of the kernel, so parallel test runs do not collide)."""
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2601_05149_b200 import synth
    cfg = synth.CONFIGS["C3"]
    rcfg, offset = bench.shard_for_rank(cfg, rank)
    # each rank's own elapsed time; everybody must get the slowest one
    mine = 10.0 + 5.0 * rank
    slowest = bench.reduce_max_ms(dist, mine, torch.device("cpu"))
    offsets = [None] * world
    dist.all_gather_object(offsets, (offset, rcfg.seed, rcfg.B))
    dist.barrier()
    if rank == 0:
        json.dump({"slowest": slowest, "offsets": offsets,
                   "value": bench.whole_job_value(world, cfg.B * cfg.H * cfg.W, 4, slowest)}, open(out, "w"))
    dist.destroy_process_group()


def test_two_ranks_shard_and_reduce(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["slowest"] == 15.0                                 # max over ranks, not rank 0's own 10 ms
    (o0, s0, b0), (o1, s1, b1) = r["offsets"]
    assert (o0, o1) == (0, b0) and b0 == b1 and s0 != s1        # disjoint global image ranges, own data
    assert r["value"] == pytest.approx(2 * 8 * 64 * 64 * 4 / 15e-3)


def test_reference_arm_under_torchrun():
    """Rank 0 alone runs the oracle and prints one JSON line; the other rank exits 0 without work."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "C1"]
    p = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["value"] > 0
    assert j["cpu_baseline"]["kind"] == "oracle" and j["e2e"]["h2d_bytes_per_step"] == 0
