"""Pins for the oracle's single-scale quantizer Q_s and reconstruction R_s
(Section "QSGDMaxNorm Quantization", Algorithm 1, Lemma 1 and its proof)."""
import json
from fractions import Fraction
from math import floor

import numpy as np
import pytest

from oracle import uq_oracle as o
from paper_2109_12497_b200 import workloads as wl
import exact_model as em
from exact_model import level_and_p, q_single, reconstruct


def _h(u, rng_bits):
    """The integer draw that represents the uniform u in [0, 1)."""
    return int(u * (1 << (23 if rng_bits == 32 else 16)))


@pytest.fixture(scope="module")
def examples(golden_dir):
    return json.loads((golden_dir / "worked_examples.json").read_text())


@pytest.mark.parametrize("rng_bits", [32, 16])
def test_worked_example_single(examples, rng_bits):
    ex = examples["A_single"]
    v = np.array([ex["v"]], dtype=np.float32)
    W = np.array([ex["W"]], dtype=np.float32)
    for case in ex["cases"]:
        h = np.full(v.shape, _h(case["u"], rng_bits), dtype=np.uint32)
        zeta = o.encode_single(v, W, ex["s"], seed=0, rng_bits=rng_bits, h_inject=h)
        assert zeta[0].tolist() == case["zeta"]
        # the fixture itself follows from the definitions in exact arithmetic
        want = [q_single(Fraction(x), Fraction(ex["W"]), ex["s"], Fraction(case["u"])) for x in ex["v"]]
        assert want == case["zeta"]
    last = np.array(ex["cases"][-1]["zeta"], dtype=np.int32)
    assert o.decode(last, 1, W, s=ex["s"]).tolist() == ex["decode_last_M1"]
    # E||Q - v||^2 = (W/s)^2 sum_i p_i (1 - p_i)   (variance identity in the proof of Lemma 1)
    ps = [level_and_p(Fraction(x), Fraction(1), ex["s"])[1] for x in ex["v"]]
    assert float(sum(p * (1 - p) for p in ps) / ex["s"] ** 2) == ex["expected_sq_error"]


def test_worked_example_exact_recovery(examples):
    ex = examples["B_exact_recovery"]
    g = np.array(ex["g"], dtype=np.float32)
    W = o.agree_scale(g)
    assert W.tolist() == [ex["W_l2"]]
    for seed in range(20):
        for rng_bits in (32, 16):
            lev = o.encode_single(g, W, ex["s"], seed=seed, rng_bits=rng_bits)
            assert np.array_equal(lev, g.astype(np.int8))       # p = 0 everywhere
            S = o.aggregate(lev)
            assert S.tolist() == ex["S"]
            assert o.decode(S, 2, W, s=ex["s"]).tolist() == ex["g_hat"]
    assert ex["g_hat"] == (g.sum(0) / 2).tolist()


@pytest.mark.parametrize("rng_bits", [32, 16])
def test_brute_force_against_exact_rationals(rng_bits):
    """Random dyadic inputs: the oracle's binary32 path must reproduce the exact-arithmetic
    definition for every injected draw (round up iff u < p)."""
    rng = np.random.default_rng(5)
    b = 23 if rng_bits == 32 else 16
    for s in (1, 3, 7, 64, 127):
        W = Fraction(1, 4)
        v = rng.integers(-256, 257, size=(2, 64)) / 1024.0      # multiples of 2^-10 in [-1/4, 1/4]
        v[0, :3] = [0.25, -0.25, 0.0]
        h = rng.integers(0, 1 << b, size=v.shape).astype(np.uint32)
        h[1, :4] = [0, (1 << b) - 1, 1 << (b - 1), 1]
        lev = o.encode_single(v.astype(np.float32), np.array([0.25], np.float32), s, 0,
                              rng_bits=rng_bits, h_inject=h)
        for m in range(2):
            for i in range(64):
                want = q_single(Fraction(v[m, i]), W, s, Fraction(int(h[m, i]), 1 << b))
                assert lev[m, i] == want, (s, m, i)


def test_exact_grid_inputs_have_no_randomness():
    """v = W t / s with integer t has p = 0: the level is t for every seed."""
    s = 127
    t = np.arange(-127, 128, dtype=np.float32)
    g = (t / 64.0)[None, :]                      # W = 127/64  =>  s / W = 64 exactly
    W = o.agree_scale(g, norm=o.NORM_LINF)
    assert W[0] == np.float32(127 / 64)
    for seed in (0, 1, 99):
        for rng_bits in (32, 16):
            assert np.array_equal(o.encode_single(g, W, s, seed, rng_bits)[0], t.astype(np.int8))


@pytest.mark.parametrize("s", [1, 7, 127])
def test_level_range_on_adversarial_inputs(s):
    W = np.float32(0.37)
    up = np.nextafter(W, np.float32(1))
    tiny = np.float32(1e-45)
    v = np.array([[W, -W, up, -up, 0.0, -0.0, tiny, -tiny, np.float32(1.17e-38), W * 0.999999]],
                 dtype=np.float32)
    for seed in range(50):
        lev = o.encode_single(v, np.array([W]), s, seed)
        assert np.abs(lev.astype(int)).max() <= s
        assert lev[0, 0] == s and lev[0, 1] == -s and lev[0, 2] == s and lev[0, 3] == -s
        assert lev[0, 4] == 0 and lev[0, 5] == 0                  # sign(0) = 0, Q(0) = 0
    # a caller-supplied scale smaller than the data: a = |v| / W > 1 has no level below s, the
    # level saturates at s (and never wraps around in int8)
    big = np.array([[2 * W, -3 * W, 1.5 * W, W / 2]], dtype=np.float32)
    for seed in range(5):
        lev = o.encode_single(big, np.array([W]), s, seed)
        assert lev[0, :3].tolist() == [s, -s, s] and abs(int(lev[0, 3])) <= s
    # an all-zero vector has W = 0 and quantizes to zero
    z = np.zeros((2, 16), dtype=np.float32)
    Wz = o.agree_scale(z)
    assert Wz[0] == 0 and not o.encode_single(z, Wz, s, 3).any()
    assert not o.decode(np.zeros(16, np.int32), 2, Wz, s=s).any()


def test_symmetry_equivariance_and_locality():
    w = wl.scaled("c1", 2048, M=2)
    g = wl.generate(w)[:, :w.d]
    W = o.agree_scale(g, norm=o.NORM_LINF)
    base = o.encode_single(g, W, 127, seed=11)
    # Q(-v) = -Q(v) with the same draws
    assert np.array_equal(o.encode_single(-g, W, 127, seed=11), -base)
    # scaling v and W by a power of two changes nothing
    assert np.array_equal(o.encode_single(g * 8, W * 8, 127, seed=11), base)
    # zeta_i depends on (v_i, W, seed, m, i) only: other coordinates and the segmentation
    # (with equal scales) do not matter
    g2 = g.copy(); g2[:, 1000:] = 0
    assert np.array_equal(o.encode_single(g2, W, 127, seed=11)[:, :1000], base[:, :1000])
    seg = [0, 100, 100, 777, 2048]
    assert np.array_equal(o.encode_single(g, np.repeat(W, 4), 127, 11, seg_off=seg), base)
    # a window of coordinates gives the same levels as the whole vector
    win = o.encode_single(np.ascontiguousarray(g[:, 500:900]), W, 127, 11, coord0=500)
    assert np.array_equal(win, base[:, 500:900])
    # different workers draw from different streams
    same = np.stack([g[0], g[0]])
    lv = o.encode_single(same, W, 127, seed=11)
    assert (lv[0] != lv[1]).mean() > 0.2
    assert (np.abs(lv[0].astype(int) - lv[1]) <= 1).all()


@pytest.mark.parametrize("rng_bits", [32, 16])
@pytest.mark.parametrize("norm", [o.NORM_L2, o.NORM_LINF])
def test_monte_carlo_unbiased_and_variance(rng_bits, norm):
    """Lemma 1: E[Q_s(v)] = v; proof of Lemma 1: Var xi_i = p (1 - p) / s^2, so
    E||Q - v||^2 = (W/s)^2 sum p_i (1 - p_i), which Lemma 1 bounds by
    (1 + min(n/s^2, sqrt(n)/s)) W^2 when W is the L2 norm."""
    n, s, trials = 48, 5, 10_000
    rng = np.random.default_rng(3)
    v = rng.standard_normal((1, n)).astype(np.float32)
    v[0, :4] = [0.0, 1e-3, -2.5, 0.5]
    W = o.agree_scale(v, norm=norm)
    x = np.abs(v[0].astype(np.float64)) * s / float(W[0])
    p = x - np.floor(x)
    acc = np.zeros(n); err2 = 0.0
    for seed in range(trials):
        lev = o.encode_single(v, W, s, seed=seed, rng_bits=rng_bits)[0].astype(np.float64)
        acc += lev
        q = float(W[0]) * lev / s
        err2 += ((q - v[0]) ** 2).sum()
    mean = acc / trials
    tol = 5 * np.sqrt(p * (1 - p) / trials) + 1e-4
    assert (np.abs(mean - np.sign(v[0]) * x) <= tol).all()
    closed = (float(W[0]) / s) ** 2 * (p * (1 - p)).sum()
    assert abs(err2 / trials - closed) <= 0.05 * closed
    if norm == o.NORM_L2:
        assert err2 / trials <= (1 + min(n / s ** 2, np.sqrt(n) / s)) * float(W[0]) ** 2
    assert err2 / trials <= n * float(W[0]) ** 2 / (4 * s ** 2) * 1.05


def test_one_long_vector_of_equal_values_rounds_up_with_frequency_p():
    """Independence across coordinates: n copies of one value round up about p n times."""
    n, s = 200_000, 127
    for rng_bits in (32, 16):
        for frac in (0.1, 0.5, 0.9):
            g = np.full((1, n), (3 + frac) / 64.0, dtype=np.float32)
            g[0, 0] = 127 / 64.0                         # sets W (L-infinity) so that s / W = 64
            W = o.agree_scale(g, norm=o.NORM_LINF)
            lev = o.encode_single(g, W, s, seed=2, rng_bits=rng_bits)[0, 1:].astype(int)
            assert set(np.unique(lev)) <= {3, 4}
            assert abs((lev == 4).mean() - frac) < 5 * np.sqrt(frac * (1 - frac) / n)


def test_decode_commutes_with_the_sum():
    """All-reduce compatibility: reconstructing the summed levels equals the mean of the
    per-worker reconstructions (remark after Algorithm 1)."""
    w = wl.scaled("c2", 4001, M=8)
    g = wl.generate(w)[:, :w.d]
    seg = wl.segment_offsets(w)
    W = o.agree_scale(g, seg)
    lev = o.encode_single(g, W, 127, seed=0, seg_off=seg)
    S = o.aggregate(lev)
    assert np.array_equal(S, lev.astype(np.int64).sum(0))
    tot = o.decode(S, w.M, W, s=127, seg_off=seg, f64=True)
    per = np.mean([o.decode(lev[m].astype(np.int32), 1, W, s=127, seg_off=seg, f64=True)
                   for m in range(w.M)], axis=0)
    # (terms of opposite sign cancel in the mean, so the absolute floor is set by one level)
    assert np.allclose(tot, per, rtol=1e-12, atol=1e-12 * float(W.max()) / 127)
    f32 = o.decode(S, w.M, W, s=127, seg_off=seg)
    assert np.allclose(f32, tot, rtol=1e-6, atol=0)                     # the stated fp32 bar
    # and the reconstruction is the exact-arithmetic R_s up to binary32 rounding
    for i in (0, 17, 4000):
        j = np.searchsorted(seg, i, side="right") - 1
        want = reconstruct(int(S[i]), Fraction(float(W[j])), 127, w.M)
        assert abs(Fraction(float(f32[i])) - want) <= abs(want) * Fraction(1, 1 << 22)


def test_int4_packing_layout():
    lev = np.array([[-7, 7, 0, -1, 3], [1, 2, 3, 4, 5]], dtype=np.int8)
    padded = np.zeros((2, 32), dtype=np.int8); padded[:, :5] = lev
    packed = o.pack_levels_i4(padded[:, :5])
    assert packed.shape == (2, 3)
    assert packed[0].tolist() == [0x79, 0xF0, 0x03] and packed[1].tolist() == [0x21, 0x43, 0x05]


def test_int2_packing_layout():
    """Four two's-complement 2-bit fields per byte, the lowest coordinate in the lowest bits."""
    lev = np.array([[-1, 1, 0, -1, 1], [0, 0, 1, 1, -1]], dtype=np.int8)
    padded = np.zeros((2, 32), dtype=np.int8); padded[:, :5] = lev
    packed = o.pack_levels_i2(padded[:, :5])
    assert packed.shape == (2, 2)
    # row 0: fields 11 01 00 11 -> 0b11000111, then 01;   row 1: 00 00 01 01 -> 0b01010000, then 11
    assert packed[0].tolist() == [0b11000111, 0b01] and packed[1].tolist() == [0b01010000, 0b11]
    # unpacking with sign extension gives the levels back
    for m in range(2):
        bits = np.repeat(packed[m], 4) >> np.tile(np.arange(4) * 2, 2) & 3
        assert (((bits ^ 2) - 2)[:5] == lev[m]).all()


def test_int6_planar_packing_layout():
    """Two planes per row: nibbles of bits 0..3, then 2-bit fields of bits 4..5 at byte stride/2."""
    lev = np.array([[-31, 31, 0, -1, 17, -16]], dtype=np.int8)
    buf = np.zeros((1, 32), dtype=np.int8); buf[:, :6] = lev
    packed = o.pack_levels_i6p(buf[:, :6], 32)
    assert packed.shape == (1, 32)                   # 16 + 8 = 24 bytes, rounded up to 16
    # 6-bit codes: -31 = 100001, 31 = 011111, 0, -1 = 111111, 17 = 010001, -16 = 110000
    assert packed[0, :3].tolist() == [0xF1, 0xF0, 0x01]                       # nibbles 1 F | 0 F | 1 0
    assert packed[0, 16:18].tolist() == [0b11_00_01_10, 0b11_01]             # fields 10 01 00 11 | 01 11
    assert not packed[0, 3:16].any() and not packed[0, 18:].any()
    # reading the planes back: 16 * signed(2-bit field) + nibble
    nib = np.repeat(packed[0, :16], 2) >> np.tile([0, 4], 16) & 15
    cr = np.repeat(packed[0, 16:24], 4) >> np.tile([0, 2, 4, 6], 8) & 3
    assert ((16 * ((cr ^ 2) - 2) + nib)[:6] == lev[0]).all()


@pytest.mark.parametrize("b,rng_bits", [(16, 16), (23, 32)])
def test_draw_threshold_is_the_nearest_multiple_ties_to_even(b, rng_bits):
    """Reading of "with probability p" for a b-bit draw: round up iff h < rint(p * 2^b), ties to
    even.  Draws are injected on both sides of the threshold; the expected levels come from the
    exact-rational model, which a ceiling, a floor or round-half-up each fail on one of the cases:
      two values of p for which p * 2^b has a fraction above and below one half, so the nearest
        multiple is the ceiling for one and the floor for the other;
      p * 2^b = k + 1/2 exactly with k even and with k odd: the tie goes to the even neighbour.
    W = 1 and s a power of two keep x = |v| * (s / W) exact, so the model sees the oracle's p."""
    s, W = 4, np.float32(1.0)
    f32 = lambda x: Fraction(float(np.float32(x)))
    ulp = Fraction(1, 2 ** (b + 1))                                     # half a step of the draw
    half = Fraction(1, 2)
    # x = 1.3, 1.7 (nearest binary32): p * 2^16 has fraction 0.8.. / 0.2..; for 23 bits the fraction
    # bits must lie below 2^-23, so x < 1/2: x = 1/4 + 5 * 2^-25 and 1/4 + 7 * 2^-25 (fractions 1/4, 3/4)
    vs = [np.float32(0.325), np.float32(-0.425)] if b == 16 else \
         [np.float32(float((Fraction(1, 4) + Fraction(5, 2 ** 25)) / s)), np.float32(float(-(Fraction(1, 4) + Fraction(7, 2 ** 25)) / s))]
    vs += [
          np.float32(float((half + 5 * ulp) / s)), np.float32(float(-(half + 7 * ulp) / s)),   # ties: p * 2^b = k + 1/2, k even / odd
          np.float32(float(-(half + 9 * ulp) / s)), np.float32(float((half + 3 * ulp) / s))]   # k even / odd
    assert len(vs) == 6
    for v in vs:
        assert Fraction(float(v)) * s == f32(float(v) * s)                # x is exact in binary32
        l, p = em.level_and_p(Fraction(float(v)), Fraction(1), s)
        P = em.rint_half_even(p * 2 ** b)
        assert 0 < P < 2 ** b
        for h in (P - 1, P, 0, 2 ** b - 1):
            g = np.array([[v]], dtype=np.float32)
            got = int(o.encode_single(g, np.array([W]), s, 0, rng_bits, h_inject=np.array([[h]], dtype=np.uint32))[0, 0])
            want = em.q_single_draw(Fraction(float(v)), Fraction(1), s, h, b)
            assert got == want, (float(v), h, got, want)
        # the two draws around the threshold really straddle it
        assert em.q_single_draw(Fraction(float(v)), Fraction(1), s, P - 1, b) != em.q_single_draw(Fraction(float(v)), Fraction(1), s, P, b)
    for v, k_par in zip(vs[2:], (0, 1, 0, 1)):                         # the ties really are ties, of both parities
        pb = em.level_and_p(Fraction(float(v)), Fraction(1), s)[1] * 2 ** b
        assert pb % 1 == half and floor(pb) % 2 == k_par
        assert em.rint_half_even(pb) == floor(pb) + k_par
    # and the rounding direction differs between the cases, so neither ceiling nor floor fits all
    fr = [(em.level_and_p(Fraction(float(v)), Fraction(1), s)[1] * 2 ** b) % 1 for v in vs[:2]]
    assert fr[0] > Fraction(1, 2) > fr[1] or fr[1] > Fraction(1, 2) > fr[0]
