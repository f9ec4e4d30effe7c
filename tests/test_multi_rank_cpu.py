"""The multi-GPU mode of the benchmark is replication: every rank runs the whole path on its own
batch and no collective touches the data. What the ranks do share is the timing rule (the job's step
time is the slowest rank's, the job's throughput is all ranks' work over it). That rule is exercised
here with two CPU processes over gloo."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    ms_local = 10.0 if rank == 0 else 25.0          # rank 1 is the slow one
    ms_per_step, units_per_s = bench.job_throughput(ms_local, steps=5, units_per_step_per_rank=1000.0, world=world, dist=dist)
    dist.barrier()
    out.put((rank, ms_per_step, units_per_s))
    dist.destroy_process_group()


def test_job_throughput_takes_the_slowest_rank_and_sums_the_work():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms_per_step, units_per_s in res:
        assert ms_per_step == pytest.approx(25.0 / 5)               # max over ranks
        assert units_per_s == pytest.approx(2 * 1000.0 / 5e-3)      # both ranks' units over that time


def test_job_throughput_single_rank_needs_no_process_group():
    import bench

    ms_per_step, units_per_s = bench.job_throughput(8.0, steps=4, units_per_step_per_rank=50.0, world=1)
    assert ms_per_step == 2.0 and units_per_s == pytest.approx(50.0 / 2e-3)


def test_gpus_n_starts_n_ranks_and_rank0_prints_one_line(capfd):
    """`bench.py --gpus N` started as a plain program re-launches itself as N ranks: the launcher is run here with a
    CPU stand-in for the timed step (two gloo ranks)."""
    import json

    import bench

    stub = os.path.join(os.path.dirname(os.path.abspath(__file__)), "rank_stub.py")
    rc = bench.spawn_ranks(2, stub, ["--gpus", "2", "--steps", "5"])
    assert rc == 0
    lines = [ln for ln in capfd.readouterr().out.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, "exactly one result line, from rank 0"
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["argv"] == ["--gpus", "2", "--steps", "5"]
    assert line["ms_per_step"] == pytest.approx(25.0 / 5) and line["value"] == pytest.approx(2 * 1000.0 / 5e-3)


def test_recorded_traffic_is_dropped_when_the_kernel_source_changed(tmp_path, monkeypatch):
    import bench

    (tmp_path / "profiles").mkdir()
    src = tmp_path / "k.cu"
    src.write_text("kernel v1")
    (tmp_path / "profiles" / "roofline_traffic.txt").write_text(
        f"launch: gate|up\nsource: k.cu\nsource_sha256: {bench.sha256_of(str(src))}\ndram_bytes_per_launch: 12345\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.recorded_traffic()[0] == 12345
    src.write_text("kernel v2")
    assert bench.recorded_traffic()[0] is None
