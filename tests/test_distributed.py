"""The distributed step (M workers spread over processes) under gloo on CPU: two and three ranks,
each holding some of the workers, must end with the levels, indices, scales and the reconstructed
average that one process holding all M rows computes.  The C-ABI calls are answered by a CPU
stand-in (tests/fake_kernels.py), so this checks the exchange logic, not the kernels."""
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


def _rank(rank, world, port, name, d, M_local, overrides, exchange, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import fake_kernels as K
    from paper_2109_12497_b200 import workloads as wl
    from paper_2109_12497_b200.distributed import DistributedQuantizer
    w = wl.scaled(name, d, M=world * M_local, **overrides)
    g_all = wl.generate(w)
    fmt = {"i8": K.UQ_FMT_I8, "i4x2": K.UQ_FMT_I4X2, "i2x4": K.UQ_FMT_I2X4}[w.fmt]
    q = DistributedQuantizer(
        M_local, w.d, torch.float32 if w.dtype == wl.F32 else torch.bfloat16, seg_off=wl.segment_offsets(w), s=w.s,
        scales=list(w.scales) if w.quantizer == "multi" else None, fmt=fmt, idx_bits=w.idx_bits,
        norm=K.UQ_NORM_L2 if w.norm == wl.NORM_L2 else K.UQ_NORM_LINF, rng_bits=w.rng_bits, device="cpu", kernels=K,
        exchange=exchange)
    mine = np.zeros((M_local, q.stride), dtype=g_all.dtype)              # rows padded to the quantizer's stride
    mine[:, : g_all.shape[1]] = g_all[rank * M_local: (rank + 1) * M_local]
    t = torch.from_numpy(mine)
    if w.dtype == wl.BF16:
        t = t.view(torch.bfloat16)
    res = q.step(t, seed=w.seed).numpy().copy()
    lev = q.lev_all if q.lev_all is not None else q.lev_local            # all rows, or mine only (slice exchange)
    out.put((rank, res, q.W.numpy().copy(), lev.view(torch.uint8).numpy().copy(),
             None if q.idx is None else q.idx.numpy().copy(), q.wire_bytes_per_step()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,M_local,name,d,overrides,exchange", [
    (2, 1, "c2", 5003, {}, "gather"), (2, 2, "c3", 5003, {}, "gather"), (3, 1, "c5", 4099, {}, "gather"),
    (2, 1, "c4", 3001, {}, "gather"), (2, 3, "c3", 2050, dict(fmt="i2x4", s=1, scales=(1, 16, 256)), "gather"),
    (2, 1, "c2", 5003, {}, "slices"), (3, 2, "c3", 5003, {}, "slices"), (3, 1, "c5", 4099, {}, "slices"),
    (2, 2, "c4", 3001, {}, "slices"), (4, 1, "c3", 300, dict(fmt="i2x4", s=1, scales=(1, 16, 256)), "slices"),
])
def test_ranks_reproduce_the_single_process_result(world, M_local, name, d, overrides, exchange):
    from paper_2109_12497_b200 import workloads as wl
    from parity import run_oracle
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, world, port, name, d, M_local, overrides, exchange, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = wl.scaled(name, d, M=world * M_local, **overrides)
    ref = run_oracle(w, wl.generate(w))
    for rank, res, W, lev_all, idx, wire in results:
        assert np.array_equal(W, ref["W"])
        rows = ref["lev"] if exchange == "gather" else ref["lev"][rank * M_local: (rank + 1) * M_local]
        assert np.array_equal(lev_all[:, : ref["lev"].shape[1]], rows)                 # rows in worker order
        if w.quantizer == "multi":
            assert np.array_equal(idx[: ref["idx"].size], ref["idx"])
        assert np.array_equal(res, ref["out"])
        shift = {"i8": 0, "i4x2": 1, "i2x4": 2}[w.fmt]
        if exchange == "gather":
            assert wire >= (world - 1) * M_local * ((-(-d // 32) * 32) >> shift)       # the level rows dominate
        else:
            assert wire >= (world - 1) * (M_local * (d >> shift) + 4 * d) // world     # a slice of each, from every peer
