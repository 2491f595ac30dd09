"""The paper's definitions in exact rational arithmetic (test helper, no floating point).

Independent of the oracle's C code: used to brute-force small cases whose inputs are dyadic
rationals, where binary32 represents every intermediate exactly and both must agree.
"""
from fractions import Fraction
from math import floor


def sign(v):
    return (v > 0) - (v < 0)


def level_and_p(v: Fraction, W: Fraction, s: int):
    """l and p(a, s) = a s - l for a = |v| / W  (definition of xi_i); a = 1 gives (s, 0)."""
    a = abs(v) / W
    assert 0 <= a <= 1
    l = floor(a * s)
    return l, a * s - l


def q_single(v: Fraction, W: Fraction, s: int, u: Fraction) -> int:
    """zeta_i = sign(v) * s * xi_i with xi_i = (l+1)/s iff u < p."""
    l, p = level_and_p(v, W, s)
    return sign(v) * (l + (1 if u < p else 0))


def own_scale_index(v: Fraction, W: Fraction, scales) -> int:
    """Index of the largest s in the set with s <= (W / |v|) * min_j s_j (any s if v = 0)."""
    s_hat = min(scales)
    ok = [k for k, s in enumerate(scales) if v == 0 or s <= (W / abs(v)) * s_hat]
    return max(ok, key=lambda k: scales[k])


def reconstruct(S: int, W: Fraction, s: int, M: int) -> Fraction:
    """R applied to the averaged levels: W * (S / M) / s."""
    return W * Fraction(S, M) / s


def rint_half_even(x: Fraction) -> int:
    """The integer nearest to x, a tie going to the even one (IEEE round-to-nearest-even)."""
    f = floor(x)
    r = x - f
    if r > Fraction(1, 2) or (r == Fraction(1, 2) and f % 2 == 1):
        return f + 1
    return f


def q_single_draw(v: Fraction, W: Fraction, s: int, h: int, b: int) -> int:
    """The reading of "with probability p" for a b-bit draw h, uniform on [0, 2^b): round up iff
    h < rint(p * 2^b), i.e. with the multiple of 2^-b nearest to p (ties to even)."""
    l, p = level_and_p(v, W, s)
    return sign(v) * (l + (1 if h < rint_half_even(p * 2 ** b) else 0))
