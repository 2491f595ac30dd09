"""Pins for the oracle's shared scale (Algorithm 1, line "MaxAllReduce Norm")."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import uq_oracle as o
from paper_2109_12497_b200 import workloads as wl


def test_l2_closed_forms():
    g = np.zeros((2, 8), dtype=np.float32)
    g[0, :2] = [3, -4]          # norm 5
    g[1, 2:5] = [1, -2, 2]      # norm 3
    assert o.agree_scale(g, norm=o.NORM_L2)[0] == np.float32(5.0)
    assert o.agree_scale(g, norm=o.NORM_LINF)[0] == np.float32(4.0)
    for k, c in [(4, 0.75), (9, -1.5), (16, 2.0 ** -70), (1 << 20, 3.0)]:
        g = np.full((1, k), c, dtype=np.float32)
        assert o.agree_scale(g)[0] == np.float32(abs(c) * math.isqrt(k))


def test_max_is_over_workers_and_per_segment():
    # worker 1 has the larger norm in segment 0, worker 0 in segment 1
    g = np.array([[1, 0, 0, 6, 8, 0], [0, 3, 4, 0, 0, 1]], dtype=np.float32)
    seg = [0, 3, 6]
    assert list(o.agree_scale(g, seg, o.NORM_L2)) == [5.0, 10.0]
    assert list(o.agree_scale(g, seg, o.NORM_LINF)) == [4.0, 8.0]
    # an empty segment and an all-zero segment have scale 0
    g = np.array([[0, 0, 2, 0]], dtype=np.float32)
    assert list(o.agree_scale(g, [0, 2, 2, 4], o.NORM_L2)) == [0.0, 0.0, 2.0]


def test_l2_against_exact_rational_sum():
    """Every float is a dyadic rational, so the sum of squares is exact in Fractions; the oracle's
    W must be the binary32 nearest to the square root of the largest worker's exact sum."""
    w = wl.scaled("c2", 3001, M=3)
    g = wl.generate(w)[:, :w.d]
    seg = wl.segment_offsets(w)
    W = o.agree_scale(g, seg)
    for j in range(len(seg) - 1):
        sums = [sum(Fraction(float(x)) ** 2 for x in g[m, seg[j]:seg[j + 1]]) for m in range(w.M)]
        best = max(sums)
        got = Fraction(float(W[j]))
        lo = Fraction(float(np.nextafter(W[j], np.float32(0))))
        hi = Fraction(float(np.nextafter(W[j], np.float32(np.inf))))
        # nearest: W^2 side conditions with the midpoints to the neighbouring floats
        assert ((got + lo) / 2) ** 2 <= best <= ((got + hi) / 2) ** 2


def test_linf_is_bruteforce_max_and_bf16_is_widened_exactly():
    w = wl.scaled("c5", 4099, M=4)
    g = wl.generate(w)[:, :w.d]
    seg = wl.segment_offsets(w)
    f = wl.bf16_bits_to_f32(g)
    W = o.agree_scale(g, seg, o.NORM_LINF)
    for j in range(len(seg) - 1):
        assert W[j] == np.abs(f[:, seg[j]:seg[j + 1]]).max()
    # the bf16 path gives the same L2 scale as the same values stored as float32
    assert np.array_equal(o.agree_scale(g, seg), o.agree_scale(np.ascontiguousarray(f), seg))


def test_scale_bounds_every_coordinate():
    """|v_i| / W <= 1 for both norms: what the definition of xi_i needs (a in [0, 1])."""
    w = wl.scaled("c4", 5003, M=5)
    g = wl.generate(w)[:, :w.d]
    for norm in (o.NORM_L2, o.NORM_LINF):
        W = o.agree_scale(g, None, norm)[0]
        assert np.abs(g).max() <= W
