"""The benchmark's N > 1 path on CPU: the workload shards with no data-path collective
(every rank runs its own batch/head shard), so the only communication is the max-over-ranks
of the device timings.  Two gloo ranks check that reduction and the whole-job aggregate."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [1.0 + rank, 5.0 - rank, 0.25]            # per-rank ms: step, part 0, part 1
    red = bench.max_over_ranks(mine, world, torch.device("cpu"))
    rate = bench.whole_job_rate(2.0e12, world, red[1])  # each rank does 2 TFLOP in red[1] ms
    out.put((rank, red, rate))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, rate in res:
        assert red == [2.0, 5.0, 0.25]                 # element-wise max over the two ranks
        assert abs(rate - 2 * 2.0e12 / 5.0e-3) < 1e-3  # both ranks' work over the slowest time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 1.5], 1, torch.device("cpu")) == [3.0, 1.5]
    assert bench.whole_job_rate(10.0, 1, 2.0) == 5000.0


def _spawned_rank(result_dir):
    # what `python bench.py --gpus 2` starts per rank (bench.spawn_ranks), here with the gloo backend
    sys.path.insert(0, ROOT)
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
    dist.init_process_group("gloo", rank=rank, world_size=world)
    red = bench.max_over_ranks([10.0 * (rank + 1), 1.0], world, torch.device("cpu"))
    with open(os.path.join(result_dir, f"rank{rank}.txt"), "w") as f:
        f.write(repr((world, red)))
    dist.destroy_process_group()


def test_gpus_flag_spawns_its_own_ranks(tmp_path):
    # `--gpus N` without torchrun goes through bench.spawn_ranks: N processes with torchrun's
    # environment that find each other on 127.0.0.1
    sys.path.insert(0, ROOT)
    import bench
    bench.spawn_ranks(2, _spawned_rank, (str(tmp_path),))
    for r in range(2):
        world, red = eval(open(tmp_path / f"rank{r}.txt").read())
        assert world == 2 and red == [20.0, 1.0]
