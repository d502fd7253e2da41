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


_RANK_SCRIPT = """
import json, os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
dist.init_process_group("gloo", rank=rank, world_size=world)
job_ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")
dist.barrier()
if rank == 0:
    print(json.dumps({{"n_gpus": world, "ms": job_ms, "value": bench.aggregate_throughput(1.0e9, world, job_ms)}}))
else:
    print("rank", rank, "done")          # must not reach the job's stdout
dist.destroy_process_group()
"""


def test_plain_launch_with_gpus_n_spawns_n_ranks(tmp_path):
    """`bench.py --gpus N` started without torchrun starts the N replicas itself (spawn_ranks): every rank gets the
    rendezvous variables, only rank 0 writes the job's JSON line, the exit code is the worst rank's."""
    import json
    import subprocess
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT.format(root=ROOT))
    driver = ("import sys; sys.path.insert(0, %r); import bench; "
              "sys.exit(bench.spawn_ranks(2, [sys.executable, %r], port=%d))" % (ROOT, str(script), 31500 + os.getpid() % 2000))
    res = subprocess.run([sys.executable, "-c", driver], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1                                   # one JSON line, from rank 0
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["ms"] == 15.0 and out["value"] == pytest.approx(2 * 1.0e9 / 15.0e-3)
    assert "rank 1 done" in res.stderr
    bad = ("import sys; sys.path.insert(0, %r); import bench; "
           "sys.exit(bench.spawn_ranks(2, [sys.executable, '-c', 'import os, sys; sys.exit(int(os.environ[\"RANK\"]) * 3)']))" % ROOT)
    assert subprocess.run([sys.executable, "-c", bad], timeout=120).returncode == 3
