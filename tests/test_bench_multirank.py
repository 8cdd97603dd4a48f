"""The N>1 path of bench.py is N independent replicas: no data-path collective, only the timing
reduction (maximum over ranks) and the whole-job aggregation.  Covered here with 2 gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r measured (10 + r) ms for the step region, (1 + 2r) ms and (5 - r) ms for the stages
    vals = bench.max_over_ranks([10.0 + rank, 1.0 + 2 * rank, 5.0 - rank], torch.device("cpu"), world)
    out.put((rank, vals))
    dist.barrier()
    dist.destroy_process_group()


def test_timing_is_max_over_ranks_and_value_is_whole_job():
    world, port = 2, 29611
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(world):
        assert got[r] == [11.0, 3.0, 5.0]          # every rank sees the slowest rank's time
    sys.path.insert(0, ROOT)
    import bench
    # 2 replicas x 10 steps x 1e12 ops in 11 ms (the slowest rank) -> whole-job TOPS
    assert abs(bench.whole_job_tops(2, 10, 1e12, 11.0) - 2 * 10 / 11e-3) < 1e-9
    assert bench.max_over_ranks([3.0, 4.0], torch.device("cpu"), 1) == [3.0, 4.0]


def test_reference_arm_prints_on_rank0_only(capsys, monkeypatch):
    sys.path.insert(0, ROOT)
    import bench

    class A:
        size, steps, warmup, gpus, no_merge, layout, acc_tile, acc_bits = 256, 1, 0, 2, False, "dgrad", 32, 8

    monkeypatch.setenv("RANK", "1")
    bench.run_reference(A)
    assert capsys.readouterr().out == ""
    monkeypatch.setenv("RANK", "0")
    bench.run_reference(A)
    line = capsys.readouterr().out.strip()
    import json
    d = json.loads(line)
    assert d["impl"] == "reference" and d["e2e"]["h2d_bytes_per_step"] == 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["metric"] == bench.METRIC and d["unit"] == bench.UNIT and d["value"] > 0
