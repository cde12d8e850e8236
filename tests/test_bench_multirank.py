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


def _stub_body(out_dir):
    """Stands in for bench.run_cuda on a rank without a GPU: what a rank sees of its surroundings."""
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert dist.is_initialized() and dist.get_world_size() == world and dist.get_rank() == rank
    assert os.environ["LOCAL_RANK"] == str(rank) and os.environ["MASTER_ADDR"] == "127.0.0.1"
    dist.barrier()
    red = bench.reduce_max_over_ranks([100.0 + rank])
    with open(os.path.join(out_dir, f"s{rank}.json"), "w") as f:
        json.dump({"rank": rank, "world": world, "red": red}, f)


def test_gpus_flag_spawns_the_ranks_itself(tmp_path):
    """`python bench.py --gpus N` typed without torchrun starts N ranks: the spawn path driven here with the gloo
    backend, world size 2 and a stubbed per-rank body."""
    import bench
    assert "WORLD_SIZE" not in os.environ
    bench.spawn_ranks(2, _stub_body, (str(tmp_path),), backend="gloo")
    seen = [json.load(open(tmp_path / f"s{r}.json")) for r in range(2)]
    assert [d["rank"] for d in seen] == [0, 1] and all(d["world"] == 2 and d["red"] == [101.0] for d in seen)
    # main() takes that path exactly when --gpus N > 1 is given and no launcher has set WORLD_SIZE
    assert bench.parse_args(["--gpus", "4"]).gpus == 4 and bench.parse_args([]).gpus == 1


def test_timed_regions_repeat_until_enough_has_been_timed(monkeypatch):
    """The K-step region is repeated until at least the minimum has been timed, never fewer than three times."""
    import bench

    class _Ev:
        now = [0.0]

        def __init__(self, enable_timing=True):
            self.t = 0.0

        def record(self):
            self.t = _Ev.now[0]

        def elapsed_time(self, other):
            return other.t - self.t

    monkeypatch.setattr(torch.cuda, "Event", _Ev)

    def step():
        _Ev.now[0] += 2.0                                       # every step "takes" 2 ms

    r = bench.timed_regions(step, 10, lambda: None, min_total_s=0.1)
    assert r == [20.0] * 5                                       # 5 regions of 20 ms reach 100 ms
    r = bench.timed_regions(step, 1000, lambda: None, min_total_s=0.1)
    assert len(r) == 3                                           # one region would do; at least three are taken
    r = bench.timed_regions(step, 10, lambda: None, min_total_s=0.0, max_regions=1)
    assert len(r) == 1
