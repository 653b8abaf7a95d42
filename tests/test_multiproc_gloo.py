"""The N > 1 path of bench.py shards nothing on the data path (independent replicas, no collective): what the ranks
share is the barrier, the max-over-ranks step time and the whole-job aggregation. That host logic is exercised here with
two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                    # rank 1 is the slower replica
    ms = bench.max_over_ranks(ms_local, world, device="cpu")
    value = bench.whole_job_value(flops_per_rank=2.0e12, world=world, ms_total=ms, steps=4)
    dist.barrier()
    out[rank] = (ms, value)
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work():
    world, port = 2, 29731
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            ms, value = out[rank]
            assert ms == 15.0                                         # the slowest rank's time on every rank
            assert abs(value - 2 * 2.0e12 / (15.0e-3 / 4) / 1e12) < 1e-9   # both ranks' FLOPs over that time, TFLOP/s


def _allreduce_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_1901_09290_b200 import harness
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.arange(1000, dtype=torch.float32) * (rank + 1)        # rank r holds (r + 1) * [0, 1, 2, ...]
    harness.allreduce_mean(g, world)
    out[rank] = g.clone()
    dist.destroy_process_group()


def test_two_gloo_ranks_average_the_flat_gradient_buffer():
    """The one exchange of a data-parallel step: every rank ends with the mean of the ranks' gradient buffers."""
    world, port = 2, 29733
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_allreduce_worker, args=(world, port, out), nprocs=world, join=True)
        want = torch.arange(1000, dtype=torch.float32) * 1.5
        for rank in range(world):
            assert torch.equal(out[rank], want)


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1, device="cpu") == 7.5
    assert abs(bench.whole_job_value(1e12, 1, 10.0, 10) - 1.0e12 / 1e-3 / 1e12) < 1e-9


def _spawned_rank(path):
    """What a rank started by bench.spawn_ranks sees: the launcher's environment, and a working rendezvous."""
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    with open(f"{path}.{rank}", "w") as f:
        f.write(f"{world} {t.item()}")
    dist.destroy_process_group()


def test_bench_spawns_the_ranks_itself_when_no_launcher_did(tmp_path):
    """`bench.py --gpus N` without torchrun starts N ranks (one per GPU) instead of silently running one."""
    sys.path.insert(0, ROOT)
    import bench
    path = str(tmp_path / "rank")
    bench.spawn_ranks(2, _spawned_rank, (path,))
    for rank in range(2):
        world, total = open(f"{path}.{rank}").read().split()
        assert int(world) == 2 and float(total) == 3.0


def test_bench_refuses_a_world_size_that_contradicts_gpus():
    import subprocess
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], env=env, capture_output=True, text=True)
    assert r.returncode != 0 and "--gpus 2" in (r.stderr + r.stdout)
