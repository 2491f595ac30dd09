"""The pieces the distributed step adds, on one GPU with the real kernels: rows encoded with
their worker's number in the job, the field-wise minimum of packed index rows, and the whole
exchange replayed rank by rank (copies stand in for the collectives) against the oracle's
single-process result."""
import os
import socket

import numpy as np
import pytest
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from paper_2109_12497_b200.pipeline import from_workload
from parity import check_parity, run_gpu, run_oracle, to_device, ulp_distance

pytestmark = pytest.mark.gpu

FMT = {"i8": B.UQ_FMT_I8, "i4x2": B.UQ_FMT_I4X2, "i2x4": B.UQ_FMT_I2X4}


@pytest.mark.parametrize("idx_bits", [1, 2, 4, 8])
@pytest.mark.parametrize("R", [1, 2, 3, 8, 64])
def test_index_min_matches_oracle(idx_bits, R):
    d = 70_016                                      # a multiple of 32 coordinates: whole 8-byte words
    rng = np.random.default_rng(R * 10 + idx_bits)
    raw = rng.integers(0, min(16, 1 << idx_bits), size=(R, d), dtype=np.uint8)
    packed = np.stack([o.pack_index(raw[r], idx_bits) for r in range(R)])
    rows = torch.from_numpy(packed).cuda()
    idx = torch.full((packed.shape[1] + 8,), 0xEE, dtype=torch.uint8, device="cuda")
    B.uq_index_min(rows, idx_bits, idx[: packed.shape[1]])
    want = o.pack_index(o.index_min(raw), idx_bits)
    got = idx.cpu().numpy()
    assert np.array_equal(got[: want.size], want) and (got[packed.shape[1]:] == 0xEE).all()
    B.uq_index_min(rows, idx_bits, rows[0])         # in place into row 0
    assert np.array_equal(rows[0].cpu().numpy(), want)


def test_index_min_argument_checks():
    rows = torch.zeros((2, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.UqError):
        B.uq_index_min(rows, 3, rows[0])
    with pytest.raises(B.UqError):
        B.uq_index_min(rows, 4, rows[0], nbytes=10)                       # not whole 4-byte words


@pytest.mark.parametrize("name,d,M,parts,kw", [
    ("c2", 300_007, 8, [(0, 1), (1, 4), (4, 8)], {}),
    ("c3", 300_007, 8, [(0, 4), (4, 8)], {}),
    ("c5", 200_003, 6, [(0, 1), (1, 2), (2, 3), (3, 4), (4, 5), (5, 6)], {}),
    ("c4", 100_003, 16, [(0, 8), (8, 16)], {}),
    ("c3", 150_001, 4, [(0, 2), (2, 4)], dict(fmt="i2x4", s=1, scales=(1, 16, 256), rng_bits=32)),
])
def test_exchange_replayed_rank_by_rank(name, d, M, parts, kw):
    """Every 'rank' runs the local calls on its own rows; tensor copies play the collectives."""
    w = wl.scaled(name, d, M=M, **kw)
    g_np = wl.generate(w)
    g = to_device(w, g_np)
    seg = wl.segment_offsets(w)
    seg_dev = torch.as_tensor(np.asarray(seg, dtype=np.int64), device="cuda") if len(seg) > 2 else None
    stride, fmt, multi = g.shape[1], FMT[w.fmt], w.quantizer == "multi"
    norm = B.UQ_NORM_L2 if w.norm == wl.NORM_L2 else B.UQ_NORM_LINF
    lays = [B.Layout(b - a, d, stride, g.dtype, seg_dev, worker0=a) for a, b in parts]
    total = B.Layout(M, d, stride, g.dtype, seg_dev)
    nseg = total.nseg
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # max of the norm
    Ws = []
    for (a, b), lay in zip(parts, lays):
        W_r = torch.zeros(nseg, device="cuda")
        ws = torch.empty(max(8, lay.workspace_bytes()), dtype=torch.uint8, device="cuda")
        B.uq_agree_scale(lay, g[a:b], norm, W_r, status, ws)
        Ws.append(W_r)
    W = torch.stack(Ws).max(dim=0).values.contiguous()
    # min of the scale index
    idx = None
    if multi:
        nb = total.index_bytes(w.idx_bits)
        rows = torch.empty((len(parts), nb), dtype=torch.uint8, device="cuda")
        for r, ((a, b), lay) in enumerate(zip(parts, lays)):
            B.uq_select_scale_multi(lay, g[a:b], W, list(w.scales), w.idx_bits, rows[r], status)
        idx = torch.empty(nb, dtype=torch.uint8, device="cuda")
        B.uq_index_min(rows, w.idx_bits, idx)
    # levels of every rank's rows, gathered in worker order, then the fused sum + reconstruction
    lev_all = torch.empty((M, total.level_row_bytes(fmt)), dtype=torch.int8, device="cuda")
    for (a, b), lay in zip(parts, lays):
        if multi:
            B.uq_encode_multi(lay, g[a:b], W, list(w.scales), idx, w.idx_bits, w.seed, w.rng_bits, fmt, lev_all[a:b], status)
        else:
            B.uq_encode_single(lay, g[a:b], W, w.s, w.seed, w.rng_bits, fmt, lev_all[a:b], status)
    out = torch.empty(d, device="cuda")
    B.uq_decode(total, lev_all, B.UQ_SRC_LEVELS, fmt, W, w.s, list(w.scales) if multi else None, idx, w.idx_bits, out)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    one = run_gpu(w, g_np)                      # one process holding all M rows, same kernels
    assert np.array_equal(W.cpu().numpy(), one["W"])
    assert np.array_equal(lev_all.cpu().numpy().view(np.uint8)[:, : (d >> fmt)], one["lev"][:, : (d >> fmt)])
    if multi:
        assert np.array_equal(idx.cpu().numpy()[: d * w.idx_bits // 8], one["idx"][: d * w.idx_bits // 8])
    assert np.array_equal(out.cpu().numpy(), one["out"])
    ref = run_oracle(w, g_np, one["W"])                      # and the oracle, given the same scale bits
    assert ulp_distance(one["W"], run_oracle(w, g_np)["W"]).max() <= 1
    assert np.array_equal(lev_all.cpu().numpy().view(np.uint8)[:, : ref["lev"].shape[1]], ref["lev"])
    assert np.allclose(out.cpu().numpy(), ref["out"], rtol=1e-6, atol=0)


@pytest.mark.parametrize("name,d,M", [("c2", 300_007, 8), ("c3", 200_003, 5), ("c4", 100_003, 16), ("c5", 150_001, 9),
                                      ("c1", 33, 2)])
def test_decode_over_separate_rows(name, d, M):
    """uq_decode_rows: every worker's level row in an allocation of its own (as a peer's row would
    be), handed over as addresses; same sums and values as the one-buffer call."""
    w = wl.scaled(name, d, M=M)
    r = check_parity(w, wl.generate(w))            # the one-buffer result, itself compared with the oracle
    q = r["q"]
    rows = [q.lev[m].clone() for m in reversed(range(M))][::-1]          # allocated in reverse order
    out = torch.full((d + 16,), 7.0, device="cuda")
    S = torch.empty(d, dtype=torch.int32, device="cuda")
    B.uq_decode_rows(q.layout, [t.data_ptr() for t in rows], q.fmt, q.W, q.s, q.scales, q.idx, q.idx_bits,
                     out[8: 8 + d], S)
    got = out.cpu().numpy()
    assert np.array_equal(got[8: 8 + d], r["out"]) and (got[:8] == 7).all() and (got[8 + d:] == 7).all()
    assert np.array_equal(S.cpu().numpy(), r["S"])
    with pytest.raises(B.UqError):
        B.uq_decode_rows(q.layout, [t.data_ptr() + 1 for t in rows], q.fmt, q.W, q.s, q.scales, q.idx, q.idx_bits,
                         out[8: 8 + d])
    with pytest.raises(ValueError):
        B.uq_decode_rows(q.layout, [rows[0].data_ptr()], q.fmt, q.W, q.s, q.scales, q.idx, q.idx_bits, out[8: 8 + d])


@pytest.mark.parametrize("name,d,M,R,kw", [
    ("c2", 300_007, 8, 4, {}), ("c3", 300_007, 6, 3, {}), ("c5", 200_003, 8, 8, {}), ("c4", 100_003, 16, 2, {}),
    ("c3", 1000, 4, 4, dict(fmt="i2x4", s=1, scales=(1, 16, 256), idx_bits=2)), ("c3", 150_001, 4, 2, dict(idx_bits=8)),
    ("c2", 200, 2, 2, dict(scales=None)),
])
def test_slice_exchange_replayed_rank_by_rank(name, d, M, R, kw):
    """The reduce-scatter form of the last exchange with the real kernels: the rows are cut into R
    slices, 'rank' r reconstructs slice r from all M rows with the slice's own layout (segment table
    counted from the slice's start, the matching part of W and of the index; rows handed over in
    (local worker, sender) order as the all-to-all delivers them), and the slices side by side are
    the single-process result."""
    from paper_2109_12497_b200.distributed import SLICE_ALIGN
    kw = {k: v for k, v in kw.items() if v is not None}
    w = wl.scaled(name, d, M=M, **kw)
    g_np = wl.generate(w)
    one = check_parity(w, g_np)                    # the single-process result, itself compared with the oracle
    q = one["q"]
    P = max(1, -(-d // (R * SLICE_ALIGN))) * SLICE_ALIGN
    stride, shift, M_local = R * P, FMT[w.fmt], M // R
    seg = np.asarray(wl.segment_offsets(w), dtype=np.int64)
    sb = P >> shift
    lev = torch.zeros((M, stride >> shift), dtype=torch.int8, device="cuda")        # the rows at the padded stride
    lev[:, : q.lev.shape[1]] = q.lev
    idx = None
    if q.multi:
        idx = torch.zeros(stride * w.idx_bits // 8, dtype=torch.uint8, device="cuda")
        idx[: q.idx.numel()] = q.idx
    out = torch.zeros(R * P, device="cuda")
    for r in range(R):
        c = r * P
        d_r = min(max(d - c, 0), P)
        if d_r == 0:
            continue
        j0 = int(np.searchsorted(seg, c, side="right") - 1)
        j1 = int(np.searchsorted(seg, c + d_r, side="left"))
        sub = np.clip(seg[j0: j1 + 1] - c, 0, d_r)
        lay = B.Layout(M, d_r, P, q.layout.dtype, torch.from_numpy(sub).cuda() if len(sub) > 2 else None)
        # what the all-to-alls deliver to rank r: [local worker][sender][slice bytes]
        recv = lev.view(R, M_local, R, sb)[:, :, r, :].permute(1, 0, 2).contiguous().view(M, sb)
        B.uq_decode(lay, recv, B.UQ_SRC_LEVELS, q.fmt, q.W[j0:j1], q.s, q.scales,
                    None if idx is None else idx[c * w.idx_bits // 8:], q.idx_bits, out[c: c + P])
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy()[:d], one["out"])
    assert (out.cpu().numpy()[d:] == 0).all()


def test_worker_number_is_validated():
    with pytest.raises(B.UqError):
        lay = B.Layout(2, 100, 128, torch.float32, None, worker0=-1)
        g = torch.zeros((2, 128), device="cuda")
        B.uq_encode_single(lay, g, torch.ones(1, device="cuda"), 127, 0, 32, B.UQ_FMT_I8,
                           torch.empty((2, 128), dtype=torch.int8, device="cuda"), None)


def test_distributed_quantizer_on_one_rank_equals_the_pipeline():
    """DistributedQuantizer with the CUDA binding and a one-rank NCCL group."""
    import torch.distributed as dist
    from paper_2109_12497_b200.distributed import DistributedQuantizer
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    try:
        for name in ("c2", "c3"):
            w = wl.scaled(name, 200_003, M=4)
            g_np = wl.generate(w)
            want = check_parity(w, g_np)["out"]    # the pipeline's result, itself compared with the oracle
            q = DistributedQuantizer(
                w.M, w.d, torch.float32, seg_off=wl.segment_offsets(w), s=w.s,
                scales=list(w.scales) if w.quantizer == "multi" else None, fmt=FMT[w.fmt], idx_bits=w.idx_bits,
                norm=B.UQ_NORM_L2, rng_bits=w.rng_bits)
            got = q.step(to_device(w, g_np), w.seed).cpu().numpy()
            assert np.array_equal(got, want) and int(q.status.item()) == 0
            # the same with the level rows in symmetric memory, read where they are
            qp = DistributedQuantizer(
                w.M, w.d, torch.float32, seg_off=wl.segment_offsets(w), s=w.s,
                scales=list(w.scales) if w.quantizer == "multi" else None, fmt=FMT[w.fmt], idx_bits=w.idx_bits,
                norm=B.UQ_NORM_L2, rng_bits=w.rng_bits, pull_levels=True)
            for _ in range(2):
                got = qp.step(to_device(w, g_np), w.seed).cpu().numpy()
                assert np.array_equal(got, want) and int(qp.status.item()) == 0
            # and the reduce-scatter / all-gather form (rows padded to its stride)
            qs = DistributedQuantizer(
                w.M, w.d, torch.float32, seg_off=wl.segment_offsets(w), s=w.s,
                scales=list(w.scales) if w.quantizer == "multi" else None, fmt=FMT[w.fmt], idx_bits=w.idx_bits,
                norm=B.UQ_NORM_L2, rng_bits=w.rng_bits, exchange="slices")
            g_pad = torch.zeros((w.M, qs.stride), device="cuda")
            g_pad[:, : g_np.shape[1]] = to_device(w, g_np)
            got = qs.step(g_pad, w.seed).cpu().numpy()
            assert np.array_equal(got, want) and int(qs.status.item()) == 0
    finally:
        dist.destroy_process_group()
