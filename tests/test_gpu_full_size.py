"""Parity at the full sizes of the five workloads, in the launch configuration the benchmark
times.  c1-c3 are compared in full; c4 and c5 on the complete scale vector plus windows of
coordinates (first, last with the ragged tail, bucket boundaries, random offsets) where every
level, index, sum and reconstructed value is compared with the oracle."""
import dataclasses
import os

import numpy as np
import pytest
import torch

from oracle import uq_oracle as o
from paper_2109_12497_b200 import workloads as wl
from paper_2109_12497_b200.pipeline import from_workload
from parity import FP32_RTOL, check_parity, to_device, ulp_distance

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _oracle_threads():
    o.set_threads(max(1, os.cpu_count() or 1))
    yield
    o.set_threads(1)


@pytest.mark.parametrize("name,rng_bits", [("c1", 16), ("c1", 32), ("c2", 16), ("c2", 32), ("c3", 16)])
def test_full_workload(name, rng_bits):
    w = dataclasses.replace(wl.WORKLOADS[name], rng_bits=rng_bits)
    r = check_parity(w, wl.generate(w))
    lev = r["ref"]["lev_raw"]
    assert np.abs(lev.astype(int)).max() <= w.s
    if name == "c1":                       # max|g| scale: the whole level range is in use
        assert np.abs(lev.astype(int)).max() == 127 and len(np.unique(lev)) > 200


def _windows(w, seg, rng, n_random=6, size=1 << 18):
    d = w.d
    wins = [(0, min(d, size)), (max(0, d - size - 13), d)]
    for e in seg[1:-1][:: max(1, (len(seg) - 2) // 4)]:           # around segment boundaries
        wins.append((max(0, int(e) - size // 2), min(d, int(e) + size // 2)))
    for a in rng.integers(0, max(1, d - size), size=n_random):
        a = int(a) | 1                                            # odd offsets too
        wins.append((a, min(d, a + size)))
    return wins


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_sampled_windows_of_large_workload(name):
    w = wl.WORKLOADS[name]
    g_np = wl.generate(w, threads=max(1, os.cpu_count() or 1))
    seg = wl.segment_offsets(w)
    q = from_workload(w, keep_sums=True)
    g = torch.empty((w.M, w.stride), dtype=torch.float32 if w.dtype == wl.F32 else torch.bfloat16,
                    device="cuda")
    for m in range(w.M):
        g[m].copy_(to_device(w, g_np[m: m + 1])[0])
    q.step(g, w.seed)
    torch.cuda.synchronize()
    assert q.status_bits() == 0
    del g
    W = q.W.cpu().numpy()
    W_ref = o.agree_scale(g_np[:, : w.d], seg, o.NORM_L2)
    assert ulp_distance(W, W_ref).max() <= 1
    rng = np.random.default_rng(17)
    for a, b in _windows(w, seg, rng):
        gw = np.ascontiguousarray(g_np[:, a:b])
        if w.quantizer == "multi":
            idx = o.select_scale_multi(gw, W, w.scales, seg_off=seg, coord0=a)
            lev = o.encode_multi(gw, W, w.scales, idx, w.seed, w.rng_bits, seg_off=seg, coord0=a)
            out = o.decode(o.aggregate(lev), w.M, W, scales=w.scales, idx=idx, seg_off=seg, coord0=a)
            per = 8 // w.idx_bits
            a8, b8 = -(-a // per) * per, b // per * per           # whole index bytes inside the window
            got = q.idx[a8 // per: b8 // per].cpu().numpy()
            assert np.array_equal(got, o.pack_index(idx[a8 - a: b8 - a], w.idx_bits)), (a, b)
        else:
            lev = o.encode_single(gw, W, w.s, w.seed, w.rng_bits, seg_off=seg, coord0=a)
            out = o.decode(o.aggregate(lev), w.M, W, s=w.s, seg_off=seg, coord0=a)
        if w.fmt == "i4x2":
            a2, b2 = a + (a & 1), b - (b & 1)                      # whole bytes inside the window
            got = q.lev[:, a2 // 2: b2 // 2].cpu().numpy().view(np.uint8)
            want = o.pack_levels_i4(_even_stride(lev[:, a2 - a: b2 - a]))
            assert np.array_equal(got, want), (a, b)
        else:
            assert np.array_equal(q.lev[:, a:b].cpu().numpy(), lev), (a, b)
        assert np.array_equal(q.S[a:b].cpu().numpy(), o.aggregate(lev)), (a, b)
        assert np.allclose(q.out[a:b].cpu().numpy(), out, rtol=FP32_RTOL, atol=0), (a, b)
        assert np.abs(lev.astype(int)).max() <= w.s


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_large_workload_in_full(name):
    """The two largest workloads compared with the oracle in full, not on windows: every scale,
    shared index, level, integer sum and reconstructed value (the oracle is fed the GPU's scale
    bits, which may differ from its own by one unit in the last place; see the chain rule in
    parity.py).  One pass of each side; rows are compared one at a time to bound host memory."""
    w = wl.WORKLOADS[name]
    threads = max(1, os.cpu_count() or 1)
    g_np = wl.generate(w, threads=threads)
    seg = wl.segment_offsets(w)
    q = from_workload(w, keep_sums=True)
    g = torch.empty((w.M, w.stride), dtype=torch.float32 if w.dtype == wl.F32 else torch.bfloat16, device="cuda")
    for m in range(w.M):
        g[m].copy_(to_device(w, g_np[m: m + 1])[0])
    q.step(g, w.seed)
    torch.cuda.synchronize()
    assert q.status_bits() == 0
    del g
    W = q.W.cpu().numpy()
    gv = g_np[:, : w.d]
    assert ulp_distance(W, o.agree_scale(gv, seg, o.NORM_L2)).max() <= 1
    if w.quantizer == "multi":
        idx = o.select_scale_multi(gv, W, w.scales, seg_off=seg)
        nb = w.d * w.idx_bits // 8
        assert np.array_equal(q.idx[:nb].cpu().numpy(), o.pack_index(idx, w.idx_bits)[:nb]), "scale indices differ"
        lev = o.encode_multi(gv, W, w.scales, idx, w.seed, w.rng_bits, seg_off=seg)
    else:
        lev = o.encode_single(gv, W, w.s, w.seed, w.rng_bits, seg_off=seg)
    assert np.abs(lev).max() <= w.s
    for m in range(w.M):
        row = q.lev[m].cpu().numpy().view(np.uint8)
        if w.fmt == "i4x2":
            want = o.pack_levels_i4(lev[m: m + 1])[0]
        else:
            want = lev[m].view(np.uint8)
        assert np.array_equal(row[: want.size], want), f"levels of worker {m} differ"
    S = o.aggregate(lev)
    del lev
    assert np.array_equal(q.S[: w.d].cpu().numpy(), S), "integer sums differ"
    if w.quantizer == "multi":
        out = o.decode(S, w.M, W, scales=w.scales, idx=idx, seg_off=seg)
    else:
        out = o.decode(S, w.M, W, s=w.s, seg_off=seg)
    assert np.allclose(q.out[: w.d].cpu().numpy(), out, rtol=FP32_RTOL, atol=0), "reconstruction differs"


def _even_stride(lev):
    """Copy with an even row stride, as the 4-bit packer needs."""
    M, n = lev.shape
    buf = np.zeros((M, n + (n & 1) + 2), dtype=np.int8)
    buf[:, :n] = lev
    return buf[:, :n]


@pytest.mark.parametrize("quantizer", ["single", "multi"])
def test_more_than_2_31_coordinates(quantizer):
    """d = 2^31 + 4099 (bf16, two workers): every index, offset and block number beyond 32 bits.
    The data are drawn on the GPU (seeded) with |v| <= 4 and one planted value of 8, so the L-inf
    scale is 8 by construction; windows around 2^31, 2^32 bytes and the ragged end are compared
    with the oracle coordinate by coordinate."""
    from paper_2109_12497_b200 import binding as B
    from paper_2109_12497_b200.pipeline import Quantizer
    d, M = 2 ** 31 + 4099, 2
    scales = (127, 1016, 8128) if quantizer == "multi" else None
    q = Quantizer(M, d, torch.bfloat16, s=127, scales=scales, fmt=B.UQ_FMT_I8, idx_bits=2 if scales else 0,
                  norm=B.UQ_NORM_LINF, rng_bits=16, keep_sums=True)
    g = torch.empty((M, q.stride), dtype=torch.bfloat16, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(2031)
    chunk = 1 << 28
    for m in range(M):
        for a in range(0, q.stride, chunk):
            n = min(chunk, q.stride - a)
            g[m, a: a + n] = (torch.randn(n, device="cuda", generator=gen) * 0.7).clamp_(-4, 4).to(torch.bfloat16)
    g[:, d:] = 0
    g[1, 2 ** 31 + 5] = -8.0
    q.step(g, 3)
    torch.cuda.synchronize()
    assert q.status_bits() == 0
    W = q.W.cpu().numpy()
    assert W.tolist() == [8.0]
    size = 20_000
    for a in (0, 2 ** 30 - 77, 2 ** 31 - size // 2, 2 ** 31 + 4099 - size, 1_500_000_001):
        b = min(d, a + size)
        gw = g[:, a:b].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        if scales:
            idx = o.select_scale_multi(gw, W, scales, coord0=a)
            lev = o.encode_multi(gw, W, scales, idx, 3, 16, coord0=a)
            out = o.decode(o.aggregate(lev), M, W, scales=scales, idx=idx, coord0=a)
            a4, b4 = -(-a // 4) * 4, b // 4 * 4
            assert np.array_equal(q.idx[a4 // 4: b4 // 4].cpu().numpy(), o.pack_index(idx[a4 - a: b4 - a], 2)), a
        else:
            lev = o.encode_single(gw, W, 127, 3, 16, coord0=a)
            out = o.decode(o.aggregate(lev), M, W, s=127, coord0=a)
        assert np.array_equal(q.lev[:, a:b].cpu().numpy(), lev), a
        assert np.array_equal(q.S[a:b].cpu().numpy(), o.aggregate(lev)), a
        assert np.allclose(q.out[a:b].cpu().numpy(), out, rtol=FP32_RTOL, atol=0), a
    del g, q
    torch.cuda.empty_cache()
