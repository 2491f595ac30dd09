"""The multi-GPU mode of the benchmark is "replicas only": N independent copies of the
single-GPU path, no data-path collective.  What ranks do share is the timing reduction (max
over ranks) and the whole-job value; both are exercised here with two gloo ranks on CPU."""
import os
import socket
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
sys.path.insert(0, str(ROOT / "tests"))


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


def _rank_distributed(rank, world, port, name, d, M, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import fake_kernels as K                      # CPU stand-in for the C ABI (the oracle behind the same calls)
    from paper_2109_12497_b200 import workloads as wl
    w = wl.scaled(name, d, M=M)
    rec, res = bench.bench_distributed(w, steps=2, warmup=1, device="cpu", threads=1, kernels=K, return_out=True)
    out.put((rank, rec, res))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("name,d,M", [("c2", 5003, 4), ("c5", 4099, 2)])
def test_benchmark_times_the_real_exchange_when_there_are_several_processes(name, d, M):
    """With WORLD_SIZE > 1 the benchmark also runs the workload with its workers spread over the
    processes (bench_distributed).  Two gloo ranks on CPU, the C ABI answered by the stand-in: the
    record has both exchange forms with their wire bytes, every rank ends with the single-process
    result of the oracle, and the last step's seed is the one a single process would use."""
    from oracle import uq_oracle as o
    from paper_2109_12497_b200 import workloads as wl
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_distributed, args=(r, world, port, name, d, M, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = wl.scaled(name, d, M=M)
    g = wl.generate(w)[:, : w.d]
    seg = wl.segment_offsets(w)
    seed = w.seed + 1                                      # the second of the two timed steps
    W = o.agree_scale(g, seg, o.NORM_L2 if w.norm == wl.NORM_L2 else o.NORM_LINF)
    if w.quantizer == "multi":
        idx = o.select_scale_multi(g, W, w.scales, seg_off=seg)
        lev = o.encode_multi(g, W, w.scales, idx, seed, w.rng_bits, seg_off=seg)
        want = o.decode(o.aggregate(lev), w.M, W, scales=w.scales, idx=idx, seg_off=seg)
    else:
        lev = o.encode_single(g, W, w.s, seed, w.rng_bits, seg_off=seg)
        want = o.decode(o.aggregate(lev), w.M, W, s=w.s, seg_off=seg)
    lev_bytes = {"i8": 1.0, "i4x2": 0.5}[w.fmt]
    for rank, rec, res in results:
        assert rec["processes"] == world and rec["workers_per_process"] == M // world
        assert set(rec) >= {"gather", "slices"}
        for form in ("gather", "slices"):
            assert rec[form]["ms_per_step"] > 0 and rec[form]["gradient_GBps"] > 0 and rec[form]["status_word"] == 0
        # gather: the other process's level rows (at the padded stride), its packed indices, and the scales
        stride = -(-w.d // 32) * 32
        expect = (world - 1) * (M // world) * int(stride * lev_bytes) + (len(seg) - 1) * 4
        if w.quantizer == "multi":
            expect += (world - 1) * max(16, stride * w.idx_bits // 8)
        assert rec["gather"]["wire_bytes_received_per_process_and_step"] == expect
        # slices: my slice of everybody's rows in, everybody's reconstructed slices in, the index slices both ways
        P = -(-w.d // (world * 128)) * 128
        expect = (world - 1) * ((M // world) * int(P * lev_bytes) + 4 * P) + (len(seg) - 1) * 4
        if w.quantizer == "multi":
            expect += 2 * (world - 1) * (P * w.idx_bits // 8)
        assert rec["slices"]["wire_bytes_received_per_process_and_step"] == expect
        assert np.allclose(res[: w.d], want, rtol=1e-6, atol=0)
