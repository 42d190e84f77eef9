"""Exact rational arithmetic with explicit IEEE-754 binary32 rounding.

Used to pin the C oracle by brute force on tiny inputs: every operation is
carried out on ``fractions.Fraction`` values (no rounding at all) and then
rounded once, to nearest with ties to even, onto the binary32 grid including
subnormals.  Nothing here calls libm, numpy arithmetic or the oracle.
"""
from fractions import Fraction

import numpy as np

_EMIN = -126          # exponent of the smallest normal binary32
_PREC = 24            # significand bits including the hidden one
_MAX = Fraction((1 << 24) - 1) * Fraction(2) ** (127 - 23)


def to_fraction(x) -> Fraction:
    """Exact value of a finite numpy/Python float."""
    return Fraction(float(x))


def round_binary32(x: Fraction) -> Fraction:
    """Nearest binary32 value to ``x`` (ties to even); ``x`` must not overflow."""
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    a = -x if x < 0 else x
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    e = max(e, _EMIN)
    quantum = Fraction(2) ** (e - (_PREC - 1))
    q = a / quantum
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    r = n * quantum
    if r > _MAX:
        raise OverflowError("binary32 overflow")
    return sign * r


def as_f32(x: Fraction) -> np.float32:
    """A Fraction already on the binary32 grid as numpy.float32 (exact)."""
    f = np.float32(float(x))
    assert Fraction(float(f)) == x
    return f


def add32(a: Fraction, b: Fraction) -> Fraction:
    return round_binary32(a + b)


def div32(a: Fraction, b: Fraction) -> Fraction:
    return round_binary32(a / b)


def fma32(a: Fraction, b: Fraction, c: Fraction) -> Fraction:
    return round_binary32(a * b + c)


def pairwise_sum32(values):
    """Pairwise (tree) sum with binary32 rounding, formulated as a binary
    counter: a new leaf is merged with the pending partial sums of equal span
    (left operand = the older partial); what is pending at the end is folded
    from the youngest to the oldest.  For c leaves this builds
    tree(first h) + tree(rest), h the largest power of two below c."""
    pending = {}                      # level -> partial sum over 2**level leaves
    for leaf in values:
        carry, level = leaf, 0
        while level in pending:
            carry = add32(pending.pop(level), carry)
            level += 1
        pending[level] = carry
    levels = sorted(pending)
    total = pending[levels[0]]
    for level in levels[1:]:
        total = add32(pending[level], total)
    return total


def grouped_update_exact32(p, v, g, groups, lrs, mu, wd, tree=False):
    """One element of the grouped update with every step rounded to binary32.

    p, v: Fractions; g: list of Fractions per worker; groups: list of lists of
    worker ids in schedule order; lrs: one Fraction per group; mu, wd: Fractions.
    Returns (p, v, [p after each group]).
    """
    trail = []
    for k, members in enumerate(groups):
        if tree:
            s = pairwise_sum32([g[w] for w in members])
        else:
            s = g[members[0]]
            for w in members[1:]:
                s = add32(s, g[w])
        gbar = div32(s, Fraction(len(members)))
        d = fma32(wd, p, gbar)
        v = fma32(mu, v, d)
        p = fma32(-lrs[k], v, p)
        trail.append(p)
    return p, v, trail


def grouped_update_real(p, v, g, groups, lrs, mu, wd):
    """The same recurrence over the rationals, never rounded."""
    for k, members in enumerate(groups):
        gbar = sum((g[w] for w in members), Fraction(0)) / len(members)
        d = gbar + wd * p
        v = mu * v + d
        p = p - lrs[k] * v
    return p, v
