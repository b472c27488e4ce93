"""N > 1 is replicas only (no data-path collective): the ranks agree on the step time, which is the slowest
rank's, and the job's value is the sum of the replicas' bytes over that time.  Checked with two gloo ranks."""
import os
import sys

import pytest
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
    mine = [1.5 + rank, 10.0 - rank]          # rank 1 is slower on the first, rank 0 on the second
    agreed = bench.max_over_ranks(mine)
    out.put((rank, agreed, bench.aggregate_value(3.0e9, agreed[0], world)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, agreed, value in got:
        assert agreed == [2.5, 10.0]
        assert value == pytest.approx(2 * 3.0e9 / 2.5e-3 / 1e9)


def test_launcher_starts_replicas(tmp_path):
    """`bench.py --gpus 2` started as one process becomes the launcher: two workers with the ranks, the local ranks
    and the rendezvous address of a torchrun launch; the line reports n_gpus = 2 and the aggregate of both."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    out = tmp_path / "line.json"
    rc = bench.spawn_replicas(2, [str(out)], script=os.path.join(ROOT, "tests", "replica_worker.py"))
    assert rc == 0
    line = json.loads(out.read_text())
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 3.0
    assert line["value"] == pytest.approx(2 * 4.0e9 / 3.0e-3 / 1e9)


def test_timed_blocks_stop_on_time_or_on_the_cap():
    sys.path.insert(0, ROOT)
    import bench

    class Ev:
        def __init__(self, t):
            self.t = t

        def elapsed_time(self, other):
            return other.t - self.t
    calls = []
    run = lambda blk: (calls.append(blk), (Ev(0.0), Ev(300.0)))[1]          # every block takes 300 ms
    assert bench.timed_blocks(run, lambda: None, 20, 1.0, 64) == [300.0] * 4  # 1.2 s >= 1 s after four blocks
    assert bench.timed_blocks(run, lambda: None, 20, 1.0, 2) == [300.0] * 2   # the cap
    assert bench.timed_blocks(run, lambda: None, 20, 0.0, 64) == [300.0]      # no target: one block


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]
    assert bench.aggregate_value(8.0e9, 1.0, 1) == pytest.approx(8000.0)


def test_reference_arm_runs_only_on_rank_zero(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench

    class A:
        workload, gpus, steps, warmup = "cfg0", 2, 1, 0
    monkeypatch.setenv("RANK", "1")
    assert bench.run_reference(A) == 0
    assert capsys.readouterr().out == ""
    monkeypatch.setenv("RANK", "0")
    assert bench.run_reference(A) == 0
    line = capsys.readouterr().out.strip()
    assert '"impl": "reference"' in line and '"kind": "oracle"' in line
