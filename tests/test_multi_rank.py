"""Host-side logic of the N > 1 bench path, on CPU with the gloo backend (world size 2).

The decoding step is batch-1 work with nothing to exchange, so several GPUs run independent replicas;
what the ranks share is only the timing protocol: a barrier on both sides of the timed region and the
MAX over ranks of the measured time.  The reference arm runs on rank 0 alone."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
    got = bench.max_over_ranks(dist, mine, torch.device("cpu"))
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"mine": mine, "max": got}, f)
    dist.destroy_process_group()


def test_max_over_ranks_gloo_world2(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    assert [r["mine"] for r in res] == [10.0, 15.0]
    assert all(r["max"] == 15.0 for r in res)      # every rank reports the slowest replica's time


def test_max_over_ranks_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(None, 3.25, torch.device("cpu")) == 3.25


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    assert r.stdout.strip() == ""


def test_roofline_traffic_is_null_once_the_kernel_source_changed(monkeypatch):
    """`roofline.traffic` comes from one ncu capture of one version of the projection kernel: it is reported only
    while the kernel's source still has the digest recorded with the capture."""
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setattr(bench, "NCU_KERNEL_SOURCE_SHA256_16", "0" * 16)
    assert bench.ncu_traffic(1.0e8) is None
    monkeypatch.undo()
    t = bench.ncu_traffic(1.0e8)
    assert t is None or 1.0e8 <= t <= 1.1e8          # traffic = weight bytes plus the partial sums, no re-reads
