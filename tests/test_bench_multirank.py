"""Host-side logic of the multi-rank benchmark path on CPU (gloo, world size 2): the path has no exchange
step, so ranks are independent replicas and the only cross-rank work is the max-over-ranks of the timings."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]          # rank 1 is slower on the first timing, faster on the second
    dist.barrier()
    red = bench.reduce_max_over_ranks(mine)
    value = bench.whole_job_tokens_per_s(world, 256, 100, red[0])
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"red": red, "value": value}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        d = json.load(open(tmp_path / f"r{r}.json"))
        assert d["red"] == [15.0, 3.0, 7.0]                      # element-wise max, the same on every rank
        assert abs(d["value"] - 2 * 256 * 100 / 15.0e-3) < 1e-6  # all ranks' tokens over the slowest rank's time


def test_single_process_is_identity():
    import bench
    assert bench.reduce_max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_tokens_per_s(1, 256, 10, 2.0) == 256 * 10 / 2.0e-3


def test_reference_arm_runs_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
