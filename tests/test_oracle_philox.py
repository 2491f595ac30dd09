"""Pins for the oracle's random draws."""
import numpy as np
import pytest

from oracle import uq_oracle as o


def _kat(golden_dir):
    rows = []
    for line in (golden_dir / "philox4x32_10_kat.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert list(o.philox4x32_10(ctr, key)) == want


def test_philox_is_a_bijection_of_the_counter_sample():
    # distinct counters under one key never collide (the block function is a permutation)
    key = [7, 9]
    outs = {tuple(o.philox4x32_10([c, 0, 0, 0], key)) for c in range(4096)}
    assert len(outs) == 4096


@pytest.mark.parametrize("rng_bits,width,per_block", [(32, 23, 4), (16, 16, 8)])
def test_draw_layout(rng_bits, width, per_block):
    """Coordinate i of worker m reads block i // per_block of the stream keyed by the seed with
    counter (block, m): consecutive coordinates walk through the block's four words."""
    seed, m = 0x1234_5678_9ABC_DEF0, 5
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for i in [0, 1, 2, 3, 4, 7, 8, 9, 1023, (1 << 34) + 5]:
        blk = i // per_block
        words = o.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, m, 0], key)
        if rng_bits == 32:
            want = int(words[i % 4]) >> 9
        else:
            w = int(words[(i % 8) // 2])
            want = (w >> 16) if i % 2 else (w & 0xFFFF)
        got = o.draw(seed, m, i, rng_bits)
        assert got == want and 0 <= got < (1 << width)


@pytest.mark.parametrize("rng_bits,width", [(32, 23), (16, 16)])
def test_draws_are_uniform_and_differ_by_worker_and_seed(rng_bits, width):
    n = 1 << 16
    h0 = np.array([o.draw(0, 0, i, rng_bits) for i in range(n)], dtype=np.float64) / (1 << width)
    h1 = np.array([o.draw(0, 1, i, rng_bits) for i in range(n)], dtype=np.float64) / (1 << width)
    h2 = np.array([o.draw(1, 0, i, rng_bits) for i in range(n)], dtype=np.float64) / (1 << width)
    for h in (h0, h1, h2):
        assert abs(h.mean() - 0.5) < 5 * np.sqrt(1 / 12 / n)
        counts, _ = np.histogram(h, bins=64, range=(0, 1))
        chi2 = ((counts - n / 64) ** 2 / (n / 64)).sum()
        assert chi2 < 63 + 6 * np.sqrt(2 * 63)
    for a, b in ((h0, h1), (h0, h2), (h1, h2)):
        assert abs(np.corrcoef(a, b)[0, 1]) < 5 / np.sqrt(n)
    # neighbouring coordinates are uncorrelated too
    assert abs(np.corrcoef(h0[:-1], h0[1:])[0, 1]) < 5 / np.sqrt(n)
