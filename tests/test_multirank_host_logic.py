"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own (fake) replica time; the job time is the
maximum over ranks and the reported value counts every rank's units (weak scaling, no data-path collective)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        job_ms = bench.max_over_ranks(local_ms, world, device="cpu")
        dist.barrier()
        value = bench.aggregate_throughput(1.0e9, world, job_ms)
        with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as fh:
            fh.write(f"{job_ms} {value}\n")
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_time_and_aggregate_value(tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        job_ms, value = map(float, open(tmp_path / f"r{rank}.txt").read().split())
        assert job_ms == 15.0                              # the slowest rank decides, on every rank
        assert value == pytest.approx(2 * 1.0e9 / 15.0e-3)  # both replicas' bytes over that time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.25, 1) == 3.25
    assert bench.aggregate_throughput(2.0e9, 1, 4.0) == pytest.approx(5.0e11)


def test_reference_arm_only_prints_on_rank_zero(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench

    class Args:
        steps, warmup, gpus = 1, 0, 2
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(Args)                              # other ranks leave without work or output
    assert capsys.readouterr().out == ""
