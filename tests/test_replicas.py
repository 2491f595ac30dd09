"""The multi-GPU mode of the benchmark is "replicas only": N independent copies of the
single-GPU path, no data-path collective.  What ranks do share is the timing reduction (max
over ranks) and the whole-job value; both are exercised here with two gloo ranks on CPU."""
import os
import socket
import sys
from pathlib import Path

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [1.0 + rank, 10.0 - rank]                     # rank 1 is slower on the first, faster on the second
    dist.barrier()
    got = bench.max_over_ranks(mine, "cpu")
    out.put((rank, got, bench.whole_job_value(world, 8e9, got[0])))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_throughput():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in results:
        assert got == [2.0, 10.0]                        # max over ranks, identical on every rank
        assert value == pytest.approx(2 * 8e9 / 2.0 / 1e6)


def test_single_process_is_a_no_op():
    import bench
    assert bench.max_over_ranks([3.0, 4.0], "cpu") == [3.0, 4.0]
    assert bench.whole_job_value(1, 1e9, 0.5) == pytest.approx(2000.0)


def test_reference_arm_runs_the_oracle_on_a_bounded_sample(capsys, monkeypatch):
    """`bench.py --impl reference` prints one JSON line from the CPU oracle (tiny sample here)."""
    import json
    import bench
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--steps", "1", "--warmup", "0",
                                      "--ref-coords", "20000", "--workload", "c3"])
    monkeypatch.setenv("RANK", "0")
    bench.main()
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0
