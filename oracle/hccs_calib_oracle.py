"""Oracle of the offline calibration objective (paper Section "Offline Calibration", Eq. 10).

TEST INFRASTRUCTURE, not part of the product.  Plain numpy/fp64, straight from the definition:
for a candidate theta = (B, S, Dmax) and a set of rows of one head,

    objective(theta) = mean over rows of KL( softmax(alpha * x) || q ),
    q_j = p_j / sum_k p_k,  p = the int16-path HCCS output of the row (Eq. 6, Eq. 7),

evaluated candidate by candidate and row by row with the C oracle's own row function.  The paper
leaves open how the integer outputs become a distribution and which logit scale enters the
softmax; the readings here are: renormalise the integer row to sum one, and softmax of alpha * x.
"""
from __future__ import annotations

import numpy as np

from . import hccs_oracle as orc


def candidates(n: int, grid):
    """(B, S, D) triples of a bounded grid inside the admissible band for row length n, in
    lexicographic (D, S, B) order.  grid = (D_lo, D_hi, D_step, S_lo, S_hi, S_step, B_step):
    B runs from S*D + ceil(256/n) upwards in steps of B_step while B <= floor(32767/n)."""
    D_lo, D_hi, D_step, S_lo, S_hi, S_step, B_step = grid
    f, bmax = -(-256 // n), 32767 // n
    out = []
    for D in range(max(D_lo, 1), min(D_hi, 127) + 1, D_step):
        for S in range(max(S_lo, 0), min(S_hi, 127) + 1, S_step):
            B = S * D + f
            while B <= bmax:
                out.append((B, S, D))
                B += B_step
    return out


def objective(rows, theta, alpha: float) -> float:
    """Mean KL(softmax(alpha*x) || renormalised int16 HCCS) over the rows (int8 [R, n])."""
    rows = np.asarray(rows, dtype=np.int8)
    total = 0.0
    for x in rows:
        p, _, _ = orc.row(x, theta, orc.MODE_U16)
        q = p.astype(np.float64) / float(p.sum())
        z = alpha * x.astype(np.float64)
        z -= z.max()
        sm = np.exp(z)
        sm /= sm.sum()
        nz = sm > 0
        total += float(np.sum(sm[nz] * (np.log(sm[nz]) - np.log(q[nz]))))
    return total / rows.shape[0]


def calibrate(rows, n_design: int, grid, alpha: float):
    """Grid scan: (best theta, best objective, all objectives in candidate order)."""
    cands = candidates(n_design, grid)
    vals = np.array([objective(rows, c, alpha) for c in cands])
    k = int(np.argmin(vals))            # first minimum = lexicographically smallest (D, S, B)
    return cands[k], float(vals[k]), vals
