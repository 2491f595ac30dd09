"""Pins for the oracle's multi-scale quantizer Q_{s_}, scale sharing and R_{s_}
(Section "QSGDMaxNormMultiScale Quantization", Algorithm 2, Lemma 2)."""
import json
from fractions import Fraction

import numpy as np
import pytest

from oracle import uq_oracle as o
from paper_2109_12497_b200 import workloads as wl
from exact_model import own_scale_index, q_single, reconstruct


@pytest.fixture(scope="module")
def examples(golden_dir):
    return json.loads((golden_dir / "worked_examples.json").read_text())


@pytest.mark.parametrize("rng_bits", [32, 16])
def test_worked_example_multi(examples, rng_bits):
    ex = examples["C_multi"]
    g = np.array(ex["g"], dtype=np.float32)
    W = np.array([ex["W"]], dtype=np.float32)
    scales = ex["scales"]
    idx, own = o.select_scale_multi(g, W, scales, return_own=True)
    assert own.tolist() == ex["own"] and idx.tolist() == ex["shared"]
    b = 23 if rng_bits == 32 else 16
    h = np.full(g.shape, int(ex["u"] * (1 << b)), dtype=np.uint32)
    lev = o.encode_multi(g, W, scales, idx, seed=0, rng_bits=rng_bits, h_inject=h)
    assert lev.tolist() == ex["zeta"]
    S = o.aggregate(lev)
    assert S.tolist() == ex["S"]
    assert o.decode(S, 2, W, scales=scales, idx=idx).tolist() == ex["g_hat"]
    # the fixture follows from the definitions in exact arithmetic
    Wq, u = Fraction(ex["W"]), Fraction(int(ex["u"] * (1 << b)), 1 << b)
    own_x = [[own_scale_index(Fraction(v), Wq, scales) for v in row] for row in ex["g"]]
    assert own_x == ex["own"]
    shared = [min(c) for c in zip(*own_x)]
    assert shared == ex["shared"]
    zeta_x = [[q_single(Fraction(v), Wq, scales[k], u) for v, k in zip(row, shared)] for row in ex["g"]]
    assert zeta_x == ex["zeta"]
    assert [float(reconstruct(sum(c), Wq, scales[k], 2)) for c, k in zip(zip(*zeta_x), shared)] == ex["g_hat"]


def test_one_scale_is_the_single_scale_quantizer():
    w = wl.scaled("c2", 3000, M=4)
    g = wl.generate(w)[:, :w.d]
    seg = wl.segment_offsets(w)
    W = o.agree_scale(g, seg)
    idx = o.select_scale_multi(g, W, [127], seg_off=seg)
    assert not idx.any()
    for rng_bits in (32, 16):
        a = o.encode_multi(g, W, [127], idx, seed=4, rng_bits=rng_bits, seg_off=seg)
        b = o.encode_single(g, W, 127, seed=4, rng_bits=rng_bits, seg_off=seg)
        assert np.array_equal(a, b)
    S = o.aggregate(a)
    assert np.array_equal(o.decode(S, w.M, W, scales=[127], idx=idx, seg_off=seg),
                          o.decode(S, w.M, W, s=127, seg_off=seg))


@pytest.mark.parametrize("name,scales", [("c3", wl.WORKLOADS["c3"].scales),
                                         ("c5", wl.WORKLOADS["c5"].scales),
                                         ("c3", (7, 7 * 16))])         # a two-scale (4, 8)-bit pair
def test_selection_properties(name, scales):
    w = wl.scaled(name, 6000, M=5)
    g = wl.generate(w)[:, :w.d]
    gf = g if g.dtype == np.float32 else wl.bf16_bits_to_f32(g)
    seg = wl.segment_offsets(w)
    W = o.agree_scale(g, seg)
    idx, own = o.select_scale_multi(g, W, scales, seg_off=seg, return_own=True)
    N, s_hat = len(scales), scales[0]
    # scale sharing: the shared index is the minimum of the workers' own indices
    assert np.array_equal(idx, own.min(0))
    assert idx.max() <= N - 1 and len(np.unique(idx)) > 1
    # the own index is the largest scale that satisfies the paper's inequality (exact check)
    Wc = np.repeat(W, np.diff(seg))
    for m in range(w.M):
        for i in range(0, w.d, 37):
            if Wc[i] == 0:
                continue
            want = own_scale_index(Fraction(float(gf[m, i])), Fraction(float(Wc[i])), list(scales))
            got = int(own[m, i])
            if want != got:      # only a binary32 rounding of |v| s / W at the boundary may differ
                v, Wj = Fraction(float(gf[m, i])), Fraction(float(Wc[i]))
                edge = [abs(abs(v) * s / Wj - s_hat) for s in scales]
                assert min(edge) <= Fraction(s_hat, 1 << 22), (m, i)
    # zero coordinates take the largest scale; the index never grows with |v|
    assert (own[gf == 0] == N - 1).all()
    for j in range(len(seg) - 1):
        a = np.abs(gf[0, seg[j]:seg[j + 1]]); k = own[0, seg[j]:seg[j + 1]]
        order = np.argsort(a, kind="stable")
        assert (np.diff(k[order].astype(int)) <= 0).all()
    # levels fit the bits of the smallest scale, and wherever a worker's level is below s_hat
    # it equals the single-scale quantizer run at the chosen scale with the same draw
    lev = o.encode_multi(g, W, scales, idx, seed=9, seg_off=seg)
    assert np.abs(lev.astype(int)).max() <= s_hat
    for k in range(N):
        if scales[k] > 127:
            continue
        ref = o.encode_single(g, W, scales[k], seed=9, seg_off=seg)
        sel = (idx == k)[None, :] & (np.abs(ref.astype(int)) <= s_hat)
        assert np.array_equal(lev[sel], ref[sel])


@pytest.mark.parametrize("rng_bits", [32, 16])
def test_monte_carlo_unbiased_and_lemma2_bound(rng_bits):
    """Lemma 2: E[Q_{s_}(v)] = v and E||Q - v||^2 <= (1 + min(n/s_hat^2, sqrt(n)/s_hat)) W^2."""
    n, scales, trials = 40, [3, 12, 48], 10_000
    rng = np.random.default_rng(8)
    g = (rng.standard_normal((2, n)) * np.logspace(-3, 0, n)).astype(np.float32)
    W = o.agree_scale(g)
    idx = o.select_scale_multi(g, W, scales)
    assert len(np.unique(idx)) == 3
    s_star = np.array(scales, dtype=np.float64)[idx]
    x = np.abs(g.astype(np.float64)) * s_star / float(W[0])
    p = x - np.floor(x)
    acc = np.zeros((2, n)); err2 = np.zeros(2)
    for seed in range(trials):
        lev = o.encode_multi(g, W, scales, idx, seed=seed, rng_bits=rng_bits).astype(np.float64)
        acc += lev
        err2 += ((float(W[0]) * lev / s_star - g) ** 2).sum(1)
    tol = 5 * np.sqrt(p * (1 - p) / trials) + 1e-4
    assert (np.abs(acc / trials - np.sign(g) * x) <= tol).all()
    closed = ((float(W[0]) / s_star) ** 2 * p * (1 - p)).sum(1)
    assert (np.abs(err2 / trials - closed) <= 0.05 * closed).all()
    s_hat = scales[0]
    assert (err2 / trials <= (1 + min(n / s_hat ** 2, np.sqrt(n) / s_hat)) * float(W[0]) ** 2).all()
    # finer scales can only reduce the error of the smallest-scale quantizer
    coarse = ((float(W[0]) / s_hat) ** 2 * ((np.abs(g) * s_hat / float(W[0])) % 1) *
              (1 - (np.abs(g) * s_hat / float(W[0])) % 1)).sum(1)
    assert (closed <= coarse + 1e-12).all()


def test_decode_commutes_with_the_sum_multi():
    w = wl.scaled("c5", 5000, M=8)
    g = wl.generate(w)[:, :w.d]
    seg = wl.segment_offsets(w)
    scales = list(w.scales)
    W = o.agree_scale(g, seg)
    idx = o.select_scale_multi(g, W, scales, seg_off=seg)
    lev = o.encode_multi(g, W, scales, idx, seed=0, seg_off=seg)
    S = o.aggregate(lev)
    tot = o.decode(S, w.M, W, scales=scales, idx=idx, seg_off=seg, f64=True)
    per = np.mean([o.decode(lev[m].astype(np.int32), 1, W, scales=scales, idx=idx, seg_off=seg, f64=True)
                   for m in range(w.M)], axis=0)
    assert np.allclose(tot, per, rtol=1e-12, atol=1e-12 * float(W.max()) / 127)
    f32 = o.decode(S, w.M, W, scales=scales, idx=idx, seg_off=seg)
    assert np.allclose(f32, tot, rtol=1e-6, atol=0)
    # the decoded mean tracks the true mean within the quantization step of each coordinate
    gf = wl.bf16_bits_to_f32(g).astype(np.float64)
    step = np.repeat(W, np.diff(seg)) / np.array(scales, dtype=np.float64)[idx]
    assert (np.abs(tot - gf.mean(0)) <= step + 1e-12).all()


def test_index_packing_layout():
    idx = np.array([0, 1, 2, 3, 3, 2, 1], dtype=np.uint8)
    assert o.pack_index(idx, 2).tolist() == [0b11100100, 0b00011011]
    assert o.pack_index(idx, 4).tolist() == [0x10, 0x32, 0x23, 0x01]
    assert o.pack_index(idx, 8).tolist() == idx.tolist()
    # 1-bit indices (two scales): coordinate i is bit i % 8 of byte i / 8
    bits = np.array([1, 0, 0, 1, 1, 1, 0, 1, 1, 0, 1], dtype=np.uint8)
    assert o.pack_index(bits, 1).tolist() == [0b10111001, 0b00000101]


def test_workers_split_over_processes_give_the_same_result():
    """A job whose M workers are spread over R processes: every process quantizes its own rows
    with its first worker's number, the shared index is the minimum of the per-process minima.
    Both must equal the one-process result (the draws are keyed by the worker's number in the
    job, and a minimum of minima is the minimum)."""
    w = wl.scaled("c3", 3001, M=6)
    g = wl.generate(w)[:, : w.d]
    seg = wl.segment_offsets(w)
    W = o.agree_scale(g, seg, o.NORM_L2)
    idx = o.select_scale_multi(g, W, w.scales, seg_off=seg)
    lev = o.encode_multi(g, W, w.scales, idx, 11, 16, seg_off=seg)
    lev1 = o.encode_single(g, W, 127, 11, 32, seg_off=seg)
    parts = [(0, 2), (2, 3), (3, 6)]
    # the scale: a maximum of per-process maxima
    W_parts = np.stack([o.agree_scale(g[a:b], seg, o.NORM_L2) for a, b in parts])
    assert np.array_equal(W_parts.max(axis=0), W)
    rows = np.stack([o.select_scale_multi(g[a:b], W, w.scales, seg_off=seg) for a, b in parts])
    assert np.array_equal(o.index_min(rows), idx) and np.array_equal(rows.min(axis=0), idx)
    for a, b in parts:
        assert np.array_equal(o.encode_multi(g[a:b], W, w.scales, idx, 11, 16, seg_off=seg, worker0=a), lev[a:b])
        assert np.array_equal(o.encode_single(g[a:b], W, 127, 11, 32, seg_off=seg, worker0=a), lev1[a:b])
    # and the worker number matters: the wrong one gives other draws
    assert not np.array_equal(o.encode_single(g[2:3], W, 127, 11, 32, seg_off=seg, worker0=0), lev1[2:3])
