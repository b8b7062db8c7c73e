"""Host-side pieces of bench.py that need no GPU: the reference arm's JSON line and the max-over-ranks timing
reduction used for multi-process runs (two gloo ranks on CPU)."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    res = bench.max_over_ranks([1.0 + rank, 10.0 - rank], dist, "cpu")
    dist.destroy_process_group()
    if rank == 0:
        torch.save(res, out)


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "res.pt")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert torch.load(out) == [2.0, 10.0]


def test_max_over_ranks_without_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 1.0], None, "cpu") == [3.5, 1.0]


def test_reference_arm_prints_the_contract_line():
    # the oracle timed on host cores on the small configuration; rank != 0 prints nothing
    line = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                                    "--steps", "2", "--warmup", "1"], text=True).strip().splitlines()[-1]
    d = json.loads(line)
    assert d["impl"] == "reference" and d["unit"] == "pair*ch/s" and d["value"] > 0 and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                                   "--steps", "1", "--warmup", "0"], text=True, env=env)
    assert out.strip() == ""
