"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2109_12497_b200 import binding as B
from paper_2109_12497_b200 import workloads as wl
from oracle import uq_oracle as o
from parity import check_parity, run_gpu, run_oracle, to_device

pytestmark = pytest.mark.gpu

# sizes: below one unit, around unit / tile boundaries, several tiles with a ragged tail
SIZES = [1, 2, 3, 7, 8, 9, 15, 16, 17, 31, 33, 255, 4095, 4097, 8191, 8193, 20011, 70001]


@pytest.mark.parametrize("d", SIZES)
@pytest.mark.parametrize("name", ["c1", "c4"])
def test_one_segment_sizes(name, d):
    w = wl.scaled(name, d, M=3)
    check_parity(w, wl.generate(w))


@pytest.mark.parametrize("d", [161 * 8, 20011, 300007])
@pytest.mark.parametrize("name", ["c2", "c3", "c5"])
@pytest.mark.parametrize("rng_bits", [32, 16])
def test_segmented_workloads_small(name, d, rng_bits):
    w = wl.scaled(name, d, rng_bits=rng_bits)
    r = check_parity(w, wl.generate(w))
    lev = r["ref"]["lev_raw"]
    assert np.abs(lev.astype(int)).max() <= w.s


@pytest.mark.parametrize("name,d,M,kw", [
    ("c2", 2_100_003, 8, {}), ("c2", 2_100_003, 8, dict(rng_bits=16)), ("c3", 2_100_003, 8, {}),
    ("c4", 1_060_013, 16, {}), ("c4", 1_060_013, 16, dict(rng_bits=16)), ("c5", 1_060_013, 16, {}), ("c5", 2_100_003, 8, dict(rng_bits=32, idx_bits=8)),
    ("c3", 2_100_003, 8, dict(dtype=wl.BF16, fmt="i4x2", s=7, scales=(7, 112, 1792))),
    ("c2", 2_100_003, 8, dict(fmt="i2x4", s=1, scales=(1,))),
    ("c2", 2_100_003, 8, dict(fmt="i6p", s=31, scales=(31,))),
    ("c5", 1_060_013, 16, dict(fmt="i6p", s=31, scales=tuple(31 * 8 ** k for k in range(8)))),
    ("c3", 2_100_003, 8, dict(dtype=wl.BF16, fmt="i2x4", s=1, scales=(1, 16, 256))),
])
def test_mid_size_workloads(name, d, M, kw):
    """A few million coordinates per worker: hundreds of tiles per kernel, a ragged last tile and
    rows crossed by segment boundaries, in every wire format."""
    w = wl.scaled(name, d, M=M, **kw)
    check_parity(w, wl.generate(w))


@pytest.mark.parametrize("norm", [wl.NORM_L2, wl.NORM_LINF])
@pytest.mark.parametrize("fmt,s", [("i8", 127), ("i8", 1), ("i8", 5), ("i4x2", 7), ("i4x2", 1), ("i2x4", 1), ("i6p", 31), ("i6p", 9)])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
def test_single_scale_variants(norm, fmt, s, dtype):
    w = wl.scaled("c2", 50021, M=4, norm=norm, fmt=fmt, s=s, scales=(s,), dtype=dtype)
    check_parity(w, wl.generate(w))


@pytest.mark.parametrize("idx_bits,N", [(1, 2), (2, 2), (2, 4), (4, 3), (4, 8), (4, 16), (8, 5), (8, 16)])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("fmt,s,ratio", [("i8", 127, 8), ("i4x2", 7, 16), ("i8", 31, 2), ("i2x4", 1, 4), ("i6p", 31, 16)])
def test_multi_scale_variants(idx_bits, N, dtype, fmt, s, ratio):
    if s * ratio ** (N - 1) >= 2 ** 31:
        pytest.skip("scale does not fit int32")
    scales = tuple(s * ratio ** k for k in range(N))
    w = wl.scaled("c3", 40009, M=5, idx_bits=idx_bits, scales=scales, s=s, fmt=fmt, dtype=dtype)
    r = check_parity(w, wl.generate(w))
    assert len(np.unique(r["ref"]["idx_raw"])) >= 2          # more than one scale is in use


@pytest.mark.parametrize("bits,fmt", [((8, 12), "i8"), ((6, 10), "i8"), ((6, 10), "i6p"), ((4, 8), "i4x2"), ((2, 6), "i2x4")])
@pytest.mark.parametrize("dtype", [wl.F32, wl.BF16])
@pytest.mark.parametrize("idx_bits", [1, 2])
def test_two_scale_pairs_of_the_experiments(bits, fmt, dtype, idx_bits):
    """The two-scale compressors of the paper's experiments, named by the bit widths of their two
    scales: a scale of r bits has s = 2^(r-1) - 1 levels.  The levels travel in the narrowest
    supported format that holds the smaller scale, the choice of scale in a 1-bit (or 2-bit) field."""
    scales = tuple(2 ** (r - 1) - 1 for r in bits)
    w = wl.scaled("c3", 120_011, M=8, idx_bits=idx_bits, scales=scales, s=scales[0], fmt=fmt, dtype=dtype)
    r = check_parity(w, wl.generate(w))
    assert set(np.unique(r["ref"]["idx_raw"]).tolist()) == {0, 1}
    assert np.abs(r["ref"]["lev_raw"].astype(int)).max() <= scales[0]


@pytest.mark.parametrize("M", [1, 2, 7, 8, 9, 16, 17, 33, 64])
def test_worker_counts(M):
    for name in ("c1", "c4", "c3"):
        w = wl.scaled(name, 9001, M=M)
        check_parity(w, wl.generate(w))


@pytest.mark.parametrize("M", [1, 3, 8, 15, 63, 64])
@pytest.mark.parametrize("d", [5, 31, 33, 8191, 70001])
def test_two_bit_levels(M, d):
    """Levels -1, 0, 1 at four per byte: every worker count up to the byte-lane limit of the
    aggregation, sizes around the 32-coordinate unit, and the format limit s = 1."""
    w = wl.scaled("c1", d, M=M, fmt="i2x4", s=1, scales=(1,))
    r = check_parity(w, wl.generate(w))
    assert set(np.unique(r["ref"]["lev_raw"]).tolist()) <= {-1, 0, 1}
    from paper_2109_12497_b200.pipeline import from_workload
    bad = from_workload(dataclasses.replace(w, s=2, scales=(2,)))             # the format takes s = 1 only
    with pytest.raises(B.UqError):
        bad.encode(to_device(w, wl.generate(w)), 0)


@pytest.mark.parametrize("M", [1, 3, 16, 17, 33, 64])
@pytest.mark.parametrize("d", [5, 31, 33, 8191, 70001])
def test_six_bit_levels(M, d):
    """Levels -31..31 in two planes: worker counts across the flush of the nibble lanes (16) up
    to the limit, sizes around the 32-coordinate unit, and the format limit s <= 31."""
    w = wl.scaled("c1", d, M=M, fmt="i6p", s=31, scales=(31,))
    r = check_parity(w, wl.generate(w))
    assert np.abs(r["ref"]["lev_raw"].astype(int)).max() == 31        # max|g| scale: the top level is in use
    from paper_2109_12497_b200.pipeline import from_workload
    bad = from_workload(dataclasses.replace(w, s=32, scales=(32,)))
    with pytest.raises(B.UqError):
        bad.encode(to_device(w, wl.generate(w)), 0)


def test_seed_changes_the_draws_only():
    w = wl.scaled("c1", 30000, M=2)
    g = wl.generate(w)
    a = check_parity(w, g, seed=0)
    b = check_parity(w, g, seed=(1 << 40) + 12345)
    la, lb = a["lev"].view(np.int8)[:, : w.d].astype(int), b["lev"].view(np.int8)[:, : w.d].astype(int)
    assert (la != lb).mean() > 0.2 and np.abs(la - lb).max() <= 1


def test_full_level_range_and_saturation():
    """Values at, just below and (with a caller-supplied scale) above W: levels reach +-s and
    never leave [-s, s]."""
    w = wl.scaled("c1", 4096, M=2)
    g = wl.generate(w)
    g[0, 5] = np.abs(g).max() * 3
    r = check_parity(w, g)
    lev = r["lev"].view(np.int8)
    assert lev[0, 5] == 127 and np.abs(lev.astype(int)).max() == 127
    # a scale smaller than the data: the clamp saturates instead of overflowing int8
    q = r["q"]
    gd = to_device(w, g)
    q.W.fill_(float(np.abs(g).max()) / 50)
    q.encode(gd, 0)
    torch.cuda.synchronize()
    lev = q.lev.cpu().numpy()
    ref = run_oracle(w, g, q.W.cpu().numpy())["lev_raw"]
    assert np.array_equal(lev[:, : w.d], ref) and np.abs(lev.astype(int)).max() == 127


def test_zero_and_empty_inputs():
    w = wl.scaled("c3", 5000, M=3)
    g = np.zeros((w.M, w.stride), dtype=np.float32)
    r = check_parity(w, g)
    assert not r["W"].any() and not r["S"].any() and not r["out"].any()
    assert (r["ref"]["idx_raw"] == len(w.scales) - 1).all()
    # segments that are empty or all zero next to ordinary ones
    w = dataclasses.replace(wl.scaled("c2", 6000, M=3), segments="one")
    g = wl.generate(w)
    g[:, 1000:2000] = 0
    seg = np.array([0, 0, 1000, 2000, 2000, 4097, 6000], dtype=np.int64)
    from paper_2109_12497_b200.pipeline import Quantizer
    from oracle import uq_oracle as o
    q = Quantizer(w.M, w.d, seg_off=seg, s=127, keep_sums=True)
    out = q.step(torch.from_numpy(g).cuda(), 3).cpu().numpy()
    W = o.agree_scale(g[:, : w.d], seg)
    assert np.array_equal(q.W.cpu().numpy(), W) and W[0] == 0 and W[2] == 0 and W[3] == 0
    lev = o.encode_single(g[:, : w.d], W, 127, 3, seg_off=seg)
    assert np.array_equal(q.lev.cpu().numpy()[:, : w.d], lev)
    assert np.allclose(out, o.decode(o.aggregate(lev), w.M, W, s=127, seg_off=seg), rtol=1e-6, atol=0)
    assert q.status_bits() == 0
    # d = 0 launches nothing and succeeds
    q0 = Quantizer(2, 0)
    q0.step(torch.zeros((2, 0), dtype=torch.float32, device="cuda"))
    assert q0.status_bits() == 0


def test_aggregate_and_decode_entry_points_agree_with_the_fused_kernel():
    for name in ("c2", "c4", "c5"):
        w = wl.scaled(name, 33333)
        r = check_parity(w, wl.generate(w))
        q = r["q"]
        S = torch.empty(w.d, dtype=torch.int32, device="cuda")
        B.uq_aggregate(q.layout, q.lev, q.fmt, S)
        out = torch.empty(w.d, dtype=torch.float32, device="cuda")
        B.uq_decode(q.layout, S, B.UQ_SRC_SUMS, q.fmt, q.W, q.s, q.scales, q.idx, q.idx_bits, out)
        torch.cuda.synchronize()
        assert np.array_equal(S.cpu().numpy(), r["S"])
        assert np.array_equal(out.cpu().numpy(), r["out"])


def test_outputs_stay_inside_their_buffers():
    """Canaries around out / S / idx survive; level padding may be written but stays small."""
    w = wl.scaled("c3", 10007, M=3)
    g = wl.generate(w)
    q = run_gpu(w, g)["q"]
    pad = 64
    out = torch.full((w.d + 2 * pad,), 7.0, dtype=torch.float32, device="cuda")
    S = torch.full((w.d + 2 * pad,), 7, dtype=torch.int32, device="cuda")
    # slices keep 16-byte alignment (pad is a multiple of 4 elements)
    B.uq_decode(q.layout, q.lev, B.UQ_SRC_LEVELS, q.fmt, q.W, q.s, q.scales, q.idx, q.idx_bits,
                out[pad: pad + w.d], S[pad: pad + w.d])
    torch.cuda.synchronize()
    for t in (out, S):
        t = t.cpu().numpy()
        assert (t[:pad] == 7).all() and (t[pad + w.d:] == 7).all()
    nbytes = q.layout.index_bytes(w.idx_bits)
    idx = torch.full((nbytes + 32,), 0xAB, dtype=torch.uint8, device="cuda")
    B.uq_select_scale_multi(q.layout, to_device(w, g), q.W, q.scales, q.idx_bits, idx[16: 16 + nbytes], None)
    torch.cuda.synchronize()
    idx = idx.cpu().numpy()
    assert (idx[:16] == 0xAB).all() and (idx[16 + nbytes:] == 0xAB).all()


def test_status_word_reports_bad_data_without_trapping():
    w = wl.scaled("c2", 20000, M=2)
    g = wl.generate(w)
    for bad in (np.nan, np.inf, -np.inf):
        for norm in (wl.NORM_L2, wl.NORM_LINF):
            ww = dataclasses.replace(w, norm=norm)
            gg = g.copy(); gg[1, 12345] = bad
            r = run_gpu(ww, gg)
            assert r["status"] & B.UQ_STATUS_NONFINITE
            assert np.abs(r["lev"].view(np.int8).astype(int)).max() <= 127
    # a segment table that does not end at d / is not monotone
    from paper_2109_12497_b200.pipeline import Quantizer
    for seg in ([0, 100, 50, 20000], [0, 100, 19000], [5, 100, 20000]):
        q = Quantizer(2, 20000, seg_off=np.array(seg))
        q.step(torch.from_numpy(g).cuda())
        assert q.status_bits() & B.UQ_STATUS_BAD_SEGMENTS
    # a scale so small that s / W overflows
    q = Quantizer(2, 20000)
    q.W.fill_(1e-44)
    q.encode(torch.from_numpy(g).cuda(), 0)
    assert q.status_bits() & B.UQ_STATUS_SCALE_OVERFLOW


def test_reproducible_bit_for_bit():
    w = wl.scaled("c5", 200003)
    g = wl.generate(w)
    a, b = run_gpu(w, g), run_gpu(w, g)
    for k in ("W", "S", "out"):
        assert np.array_equal(a[k], b[k])
    assert np.array_equal(a["lev"][:, : w.d], b["lev"][:, : w.d])          # padding is not data
    nb = w.d * w.idx_bits // 8
    assert np.array_equal(a["idx"][:nb], b["idx"][:nb])


@pytest.mark.parametrize("name,kw", [("c2", {}), ("c2", dict(rng_bits=16)), ("c3", {}), ("c5", {}),
                                      ("c4", {}), ("c3", dict(fmt="i2x4", s=1, scales=(1, 16, 256)))])
def test_gradient_handed_over_in_pieces(name, kw):
    """The encoders on pieces of the gradient (layout.coord0 = start of the piece, seg_off counted
    from the piece's start, pointers moved to the piece) write the levels of the one-piece call."""
    import ctypes as C
    d = 250_000
    w = wl.scaled(name, d, M=4, **kw)
    g_np = wl.generate(w)
    one = run_gpu(w, g_np)
    q = one["q"]
    g = to_device(w, g_np)
    seg = np.asarray(wl.segment_offsets(w), dtype=np.int64)
    eb = 4 if w.dtype == wl.F32 else 2
    fmt_shift = {"i8": 0, "i4x2": 1, "i2x4": 2}[w.fmt]
    lev = torch.zeros_like(q.lev)
    cuts = [0, 256, 16384 + 512, 100_096, d]
    lib = B.lib()
    for a, b in zip(cuts[:-1], cuts[1:]):
        j0 = int(np.searchsorted(seg, a, side="right") - 1)
        j1 = int(np.searchsorted(seg, b, side="left"))                     # segments j0 .. j1-1 overlap [a, b)
        sub = np.clip(seg[j0: j1 + 1] - a, 0, b - a)
        sub_dev = torch.from_numpy(sub).cuda() if len(sub) > 2 else None
        lay = B.uq_layout(b - a, q.stride, None if sub_dev is None else sub_dev.data_ptr(), w.M, len(sub) - 1,
                          B.UQ_F32 if w.dtype == wl.F32 else B.UQ_BF16, 0, a)
        gp, lp, Wp = g.data_ptr() + a * eb, lev.data_ptr() + (a >> fmt_shift), q.W.data_ptr() + 4 * j0
        if q.multi:
            sc = (C.c_int32 * len(q.scales))(*q.scales)
            rc = lib.uq_encode_multi(C.byref(lay), gp, Wp, sc, len(q.scales), q.idx.data_ptr() + a * q.idx_bits // 8,
                                     q.idx_bits, w.seed, w.rng_bits, q.fmt, lp, q.status.data_ptr(), None)
        else:
            rc = lib.uq_encode_single(C.byref(lay), gp, Wp, q.s, w.seed, w.rng_bits, q.fmt, lp, q.status.data_ptr(), None)
        assert rc == 0
    torch.cuda.synchronize()
    nb = d >> fmt_shift
    assert np.array_equal(lev.cpu().numpy().view(np.uint8)[:, :nb], one["lev"][:, :nb])
    assert q.status_bits() == 0


@pytest.mark.parametrize("rng_bits", [16, 32])
def test_block_counter_wraps_inside_a_tile(rng_bits):
    """A piece that starts just below the coordinate where the low word of the Philox block
    number wraps (2^35 for 16-bit draws, 2^34 for 32-bit draws): levels match the oracle's."""
    import ctypes as C
    wrap = 2 ** 35 if rng_bits == 16 else 2 ** 34
    coord0, d, M = wrap - 40_000, 100_003, 3
    w = wl.scaled("c1", d, M=M, rng_bits=rng_bits, norm=wl.NORM_L2)
    g_np = wl.generate(w)
    g = to_device(w, g_np)
    stride = g.shape[1]
    W = torch.from_numpy(o.agree_scale(g_np[:, :d], None, o.NORM_L2)).cuda()
    lev = torch.zeros((M, stride), dtype=torch.int8, device="cuda")
    lay = B.uq_layout(d, stride, None, M, 1, B.UQ_F32, 0, coord0)
    rc = B.lib().uq_encode_single(C.byref(lay), g.data_ptr(), W.data_ptr(), 127, 5, rng_bits, B.UQ_FMT_I8, lev.data_ptr(),
                                  None, None)
    assert rc == 0
    want = o.encode_single(g_np[:, :d], W.cpu().numpy(), 127, 5, rng_bits, coord0=coord0)
    assert np.array_equal(lev.cpu().numpy()[:, :d], want)
    # the draws really moved: the same data at coord0 = 0 gives other levels
    assert not np.array_equal(o.encode_single(g_np[:, :d], W.cpu().numpy(), 127, 5, rng_bits), want)


def test_step_right_after_an_asynchronous_copy():
    """Inputs arriving by an asynchronous copy from pinned host memory on the same stream, the
    step enqueued right behind it and the result read back asynchronously: the kernels (which may
    be scheduled while their predecessor drains) still see the complete copy, step after step."""
    w = wl.scaled("c3", 1_000_003, M=4)
    g_np = wl.generate(w)
    ref = run_oracle(w, g_np)
    from paper_2109_12497_b200.pipeline import from_workload
    q = from_workload(w, keep_sums=True)
    host = torch.from_numpy(g_np).pin_memory()
    g = torch.zeros_like(host, device="cuda")
    out_host = torch.empty(w.d, dtype=torch.float32).pin_memory()
    junk = torch.from_numpy(np.full_like(g_np, 3.0)).pin_memory()
    for k in range(3):
        g.copy_(junk, non_blocking=True)                       # what a stale read would see
        g.copy_(host, non_blocking=True)
        out = q.step(g, w.seed)
        out_host.copy_(out, non_blocking=True)
        torch.cuda.synchronize()
        assert np.array_equal(q.S.cpu().numpy()[: w.d], ref["S"]), k
        assert np.allclose(out_host.numpy(), ref["out"], rtol=1e-6, atol=0), k
    # the same behind kernels that know nothing of the library's launch attribute
    src = host.cuda()
    for k in range(3):
        g.fill_(3.0)
        g.copy_(src)
        g.mul_(1.0)
        out = q.step(g, w.seed)
        got = out.clone()                                      # a framework kernel right behind the step
        torch.cuda.synchronize()
        assert np.array_equal(q.S.cpu().numpy()[: w.d], ref["S"]), k
        assert np.allclose(got.cpu().numpy(), ref["out"], rtol=1e-6, atol=0), k


def _random_workload(rng):
    name = ["c1", "c2", "c3", "c4", "c5"][rng.integers(5)]
    d = int([rng.integers(1, 300), rng.integers(300, 40_000), rng.integers(40_000, 400_000)][rng.integers(3)])
    M = int([1, 2, 3, 5, 8, 13, 16, 17, 31, 64][rng.integers(10)])
    if d * M > 6_000_000:
        M = max(1, 6_000_000 // d)
    fmt, smax = [("i8", 127), ("i6p", 31), ("i4x2", 7), ("i2x4", 1)][rng.integers(4)]
    s = int(rng.integers(1, smax + 1))
    kw = dict(fmt=fmt, s=s, scales=(s,), dtype=[wl.F32, wl.BF16][rng.integers(2)], rng_bits=[16, 32][rng.integers(2)],
              norm=[wl.NORM_L2, wl.NORM_LINF][rng.integers(2)], seed=int(rng.integers(0, 2**62)))
    if wl.WORKLOADS[name].quantizer == "multi":
        idx_bits = int([1, 2, 4, 8][rng.integers(4)])
        N = int(rng.integers(1, min(16, 1 << idx_bits) + 1))
        ratio = int([2, 3, 8, 16][rng.integers(4)])
        scales = [s]
        while len(scales) < N and scales[-1] * ratio < 2**31:
            scales.append(scales[-1] * ratio)
        kw.update(idx_bits=idx_bits, scales=tuple(scales))
    return wl.scaled(name, d, M=M, **kw)


@pytest.mark.parametrize("case", range(48))
def test_randomized_configurations(case):
    """Seeded random draws over every argument of the path (workload recipe, d, M, element type,
    wire format, level count, scale set, index width, norm, draw width, seed)."""
    w = _random_workload(np.random.default_rng(9000 + case))
    check_parity(w, wl.generate(w))


@pytest.mark.parametrize("d", [1, 9, 2047, 2049, 8191, 8193, 70001])
@pytest.mark.parametrize("name", ["c3", "c5"])
def test_multi_scale_without_a_segment_table(name, d):
    """The multi-scale path on one segment (no table at all) with a ragged last tile."""
    w = wl.scaled(name, d, M=3, segments="one")
    assert len(wl.segment_offsets(w)) == 2
    check_parity(w, wl.generate(w))


@pytest.mark.parametrize("name", ["c2", "c3"])
def test_back_to_back_steps_do_not_interfere(name):
    """A hundred steps enqueued without a host synchronization in between (the launches let a
    kernel's blocks be scheduled while the kernel before it drains): every step must leave exactly
    the sums and values of the first one."""
    w = wl.scaled(name, 1_500_007, M=8)
    g = to_device(w, wl.generate(w))
    from paper_2109_12497_b200.pipeline import from_workload
    q = from_workload(w, keep_sums=True)
    q.step(g, w.seed)
    torch.cuda.synchronize()
    S0, out0, lev0 = q.S.clone(), q.out.clone(), q.lev.clone()
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for k in range(100):
        q.lev.fill_(0x55)                                    # stale levels would change the sums
        q.step(g, w.seed)
        bad += (q.S != S0).sum() + (q.out != out0).sum() + (q.lev[:, : w.d] != lev0[:, : w.d]).sum()
    torch.cuda.synchronize()
    assert int(bad.item()) == 0


@pytest.mark.parametrize("name,kw", [("c2", dict(rng_bits=16)), ("c2", dict(rng_bits=32)), ("c3", dict(rng_bits=16)),
                                      ("c3", dict(rng_bits=32)), ("c5", {}), ("c5", dict(rng_bits=32)), ("c4", {}),
                                      ("c4", dict(rng_bits=16))])
@pytest.mark.parametrize("power", [100, 112, -80, -100])
def test_gradients_of_extreme_magnitude(name, kw, power):
    """Gradients scaled by 2^power.  Beyond W = s * 2^100 the factor s / W is too small for the
    encoder's saturating form of the clamp with 16-bit draws (its division by 256 would no longer be
    exact), and below W = s * 2^-100 it is too large for the fixed-point form with 32-bit draws
    (times 2^23 it could overflow): the kernel must take its plain path for such tiles.  A
    power-of-two scaling changes no level (the oracle says so too), so the levels are also compared
    with those of the unscaled gradients."""
    w = wl.scaled(name, 150_001, M=4 if name != "c4" else 16, **kw)
    g = wl.generate(w)
    if w.dtype == wl.BF16:
        f = wl.bf16_bits_to_f32(g) * np.float32(2.0 ** power)
        big = wl.f32_to_bf16_bits(f)
    else:
        big = g * np.float32(2.0 ** power)
    assert np.isfinite(big.astype(np.float32) if w.dtype == wl.F32 else wl.bf16_bits_to_f32(big)).all()
    r = check_parity(w, big)
    if abs(power) <= 100 or w.dtype == wl.F32:
        base = check_parity(w, g)
        if power > 0:                                       # nothing underflows on the way up
            nb = base["ref"]["lev"].shape[1]
            assert np.array_equal(r["lev"][:, :nb], base["lev"][:, :nb])


@pytest.mark.parametrize("multi", [False, True])
@pytest.mark.parametrize("rng_bits", [16, 32])
def test_draws_at_the_edges_of_the_threshold(multi, rng_bits):
    """Scaled magnitudes x that sit on and next to the points where the draw threshold rint(p * 2^b)
    changes or carries: just below an integer (p rounds up to 1: every draw rounds up), just above
    one, exact ties between two thresholds, the clamp at the largest level.  W = 127 under the
    L-infinity norm with s = 127 makes the factor s / W exactly 1, so x = |v|."""
    ulp = lambda x: np.spacing(np.float32(x))
    xs = []
    for k in [0, 1, 2, 3, 63, 64, 126]:
        base = np.float32(k)
        for t in [1.0, 0.5, 0.25, 2.0 ** -15, 2.0 ** -16, 2.0 ** -17, 2.0 ** -22, 2.0 ** -23, 2.0 ** -24, 2.0 ** -25, 2.0 ** -30]:
            for sgn in (1.0, -1.0):
                x = np.float32(base + np.float32(0.5) + np.float32(sgn * t * 0.5))
                xs += [x, np.float32(x - ulp(x)), np.float32(x + ulp(x))]
                x = np.float32(base + np.float32(1.0 if sgn < 0 else 0.0) + np.float32(sgn * t))
                xs += [x, np.float32(x - ulp(x)) if x > 0 else x, np.float32(x + ulp(x))]
    xs = np.array([x for x in xs if 0.0 <= x <= 127.0], dtype=np.float32)
    xs = np.concatenate([xs, -xs, np.float32([127.0, -127.0, 126.99999, 0.0, -0.0, 1e-38, 1e-44, 0.99999994, 0.49999997])])
    reps = 40                                                # the same value under many different draws
    d = xs.size * reps
    if multi:
        w = wl.scaled("c3", d, M=3, rng_bits=rng_bits, norm=wl.NORM_LINF)
        w = dataclasses.replace(w, segments="one")
    else:
        w = wl.scaled("c1", d, M=3, rng_bits=rng_bits, norm=wl.NORM_LINF)
    g = np.zeros((w.M, w.stride), dtype=np.float32)
    rng = np.random.default_rng(5)
    for m in range(w.M):
        g[m, :d] = np.tile(xs, reps)[rng.permutation(d)] if m else np.tile(xs, reps)
    assert np.abs(g).max() == np.float32(127.0)
    for seed in (0, 1, 0xFFFF_FFFF_FFFF):
        r = check_parity(w, g, seed=seed)
        assert r["W"][0] == np.float32(127.0)


@pytest.mark.parametrize("name,kw", [("c5", {}), ("c2", dict(rng_bits=16)), ("c3", {})])
def test_step_replayed_from_a_cuda_graph(name, kw):
    """The step a user gets (uq_step without the integer sums; for c5's recipe two kernels, the second
    one with its shared-memory limit raised on first use) captured once in a CUDA graph, after a call
    outside the capture, and replayed on new gradients: every replay must match the oracle."""
    from paper_2109_12497_b200.pipeline import from_workload
    w = wl.scaled(name, 300_007, M=8, **kw)
    g_np = wl.generate(w)
    q = from_workload(w, one_kernel=False)
    g = to_device(w, g_np)
    q.step(g, w.seed)                                   # set-up call, outside any capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            q.step(g, w.seed)
    torch.cuda.current_stream().wait_stream(side)
    for trial in range(2):
        g_new = np.roll(g_np, 17 * (trial + 1), axis=1).copy()
        g_new[:, w.d:] = 0
        g.copy_(to_device(w, g_new))
        q.out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert q.status_bits() == 0
        ref = run_oracle(w, g_new, q.W.cpu().numpy())        # downstream of the GPU's scale bits
        assert np.abs(q.W.cpu().numpy().view(np.int32).astype(np.int64) - ref["W"].view(np.int32)).max() <= 1
        nb = ref["lev"].shape[1]
        assert np.array_equal(q.lev.cpu().numpy().view(np.uint8)[:, :nb], ref["lev"])
        assert np.allclose(q.out.cpu().numpy()[: w.d], ref["out"], rtol=1e-6, atol=0)
