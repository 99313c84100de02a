"""Second, independent statement of HCCS in pure Python (unbounded ints).

TEST INFRASTRUCTURE, not part of the product.  It exists to cross-check the C
oracle by brute force on tiny rows: the two were written separately from the
paper's Section III and share nothing but the paper.  Here the row is treated
the way the equations are printed -- as whole-row list expressions -- rather
than as Algorithm 1's loops, and floor(log2 Z) comes from ``int.bit_length``.
"""
from __future__ import annotations

from fractions import Fraction

T_INT16 = 32767
T_INT8 = 255
R_INV_SHIFT = 15


def scores(x, B, S, D, valid=None):
    """(m, delta, s) over the valid positions: Eq. 2 and Eq. 3."""
    idx = [j for j in range(len(x)) if valid is None or valid[j]]
    if not idx:
        return None, {}, {}
    m = max(int(x[j]) for j in idx)
    delta = {j: min(m - int(x[j]), D) for j in idx}
    s = {j: B - S * delta[j] for j in idx}
    return m, delta, s


def reciprocal(Z, u16, clb):
    """Eq. 6 (T = 32767), Eq. 8 (255 * 2^R) or their leading-bit form Eq. 9."""
    numer = T_INT16 if u16 else T_INT8 * 2 ** R_INV_SHIFT
    if clb:
        k = Z.bit_length() - 1          # floor(log2 Z)
        return numer // 2 ** k
    return numer // Z


def hccs_row(x, theta, u16=False, clb=False, out_shift=0, valid=None):
    """Scaled integer probabilities of one row (list of Python ints)."""
    B, S, D = (int(t) for t in theta)
    _, _, s = scores(x, B, S, D, valid)
    out = [0] * len(x)
    if not s:
        return out
    Z = sum(s.values())
    rho = reciprocal(Z, u16, clb)
    for j, sj in s.items():
        if u16:
            out[j] = sj * rho
        else:
            q = (sj * rho) // 2 ** (R_INV_SHIFT + out_shift)
            out[j] = min(q, T_INT8) if clb else q
    return out


def exact_probabilities(x, theta, valid=None):
    """p_i = s_i / Z of Eq. 5 as exact fractions (what the integer outputs approximate)."""
    B, S, D = (int(t) for t in theta)
    _, _, s = scores(x, B, S, D, valid)
    Z = sum(s.values())
    return [Fraction(s[j], Z) if j in s else Fraction(0) for j in range(len(x))]
