"""Pins for the oracle's GlobalRandK functions (Sections "GlobalRandKMaxNorm Compression" and
"GlobalRandKMaxNormMultiScale Compression"): the shared choice of K distinct coordinates is a
prefix of a permutation, uniform in the statistical sense, and gather / scatter / sparse update
agree with numpy indexing and exact arithmetic."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle.uq_oracle as o


@pytest.mark.parametrize("d", [1, 2, 3, 4, 5, 7, 8, 9, 31, 32, 33, 1000, 4097, 65537])
def test_full_selection_is_a_permutation(d):
    for seed in (0, 1, 2**63 + 12345):
        sel = o.randk_indices(d, d, seed)
        assert sorted(sel.tolist()) == list(range(d))


def test_selection_is_a_prefix_and_distinct_at_large_d():
    for d in (25_557_032, 2**35 + 7, 2**40):
        sel = o.randk_indices(d, 10_000, 42)
        assert sel.min() >= 0 and sel.max() < d and len(np.unique(sel)) == 10_000
        assert np.array_equal(o.randk_indices(d, 100, 42), sel[:100])
        assert not np.array_equal(o.randk_indices(d, 100, 43), sel[:100])
        # spread over the whole range, not clustered: every tenth of [0, d) gets its share
        counts = np.bincount((sel.astype(np.float64) / d * 10).astype(int), minlength=10)
        assert counts.min() > 850 and counts.max() < 1150


@pytest.mark.parametrize("d,n", [(3, 12_000), (4, 24_000), (5, 36_000), (6, 72_000)])
def test_every_ordering_of_a_tiny_domain_is_equally_likely(d, n):
    """'Uniformly' pinned at the strongest level that can be enumerated: over many seeds all d!
    orderings of d coordinates appear equally often (chi-square, d! - 1 degrees of freedom)."""
    counts = {}
    for seed in range(n):
        key = tuple(o.randk_indices(d, d, seed).tolist())
        counts[key] = counts.get(key, 0) + 1
    f = math.factorial(d)
    assert len(counts) == f
    chi2 = sum((c - n / f) ** 2 / (n / f) for c in counts.values())
    assert chi2 < (f - 1) + 5 * math.sqrt(2 * (f - 1))    # five standard deviations above the mean


@pytest.mark.parametrize("d,K", [(64, 8), (100, 10), (37, 5)])
def test_inclusion_and_pair_frequencies_are_uniform(d, K):
    n = 20_000
    incl = np.zeros(d)
    first_two = np.zeros((d, d))
    for seed in range(n):
        sel = o.randk_indices(d, K, seed + 1000)
        incl[sel] += 1
        first_two[sel[0], sel[1]] += 1
    # each coordinate is kept with probability K/d
    e = n * K / d
    chi2 = ((incl - e) ** 2 / (e * (1 - K / d))).sum()
    assert chi2 < d + 6 * np.sqrt(2 * d)
    # the first two choices are uniform over the d(d-1) ordered pairs
    assert np.trace(first_two) == 0
    pairs = first_two[~np.eye(d, dtype=bool)]
    ep = n / (d * (d - 1))
    chi2p = ((pairs - ep) ** 2 / ep).sum()
    dof = d * (d - 1) - 1
    assert chi2p < dof + 6 * np.sqrt(2 * dof)


def test_gather_scatter_update_against_numpy_indexing():
    rng = np.random.default_rng(5)
    d, M, K = 1000, 3, 77
    sel = o.randk_indices(d, K, 9)
    for dtype in (np.float32, np.uint16):
        g = rng.standard_normal((M, 1024)).astype(np.float32)
        g = g if dtype == np.float32 else (g.view(np.uint32) >> 16).astype(np.uint16)
        gk = o.randk_gather(g[:, :d], sel)
        assert gk.shape == (M, K) and np.array_equal(gk, g[:, sel])
        assert gk.base is not None and (gk.base[:, K:] == 0).all()          # the row padding is zero
    vals = rng.standard_normal(K).astype(np.float32)
    out = np.full(d, 7.0, dtype=np.float32)
    want = out.copy(); want[sel] = vals
    assert np.array_equal(o.randk_scatter(sel, vals, out), want)
    want[sel] = 0
    assert np.array_equal(o.randk_scatter(sel, None, out), want)
    # sparse update: exact rationals on dyadic inputs, binary32 rounding after each operation
    theta = (rng.integers(-2**10, 2**10, d) / 2.0**7).astype(np.float32)
    v = (rng.integers(-2**8, 2**8, K) / 2.0**9).astype(np.float32)
    got = o.randk_update(sel, v, theta, 0.25)
    for t in (0, 1, K - 1):
        i = sel[t]
        assert Fraction(float(got[i])) == Fraction(float(theta[i])) - Fraction(1, 4) * Fraction(float(v[t]))
    mask = np.ones(d, bool); mask[sel] = False
    assert np.array_equal(got[mask], theta[mask])
    lr = np.float32(0.1)
    got = o.randk_update(sel, vals, theta, 0.1)
    want = theta.copy(); want[sel] = theta[sel] - (lr * vals).astype(np.float32)
    assert np.array_equal(got, want)
