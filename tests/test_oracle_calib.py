"""Pins for the calibration-objective oracle (Eq. 10): closed forms and identities that do not
come from the oracle's own code."""
import math
from fractions import Fraction

import numpy as np

from oracle import hccs_calib_oracle as cal
from oracle import hccs_oracle as orc


def test_uniform_surrogate_closed_form():
    """S = 0 makes HCCS uniform: KL(softmax || uniform) = log n - H(softmax), any B, D."""
    rng = np.random.default_rng(0)
    n = 64
    rows = rng.integers(-40, 40, size=(5, n)).astype(np.int8)
    alpha = 1 / 16
    want = 0.0
    for x in rows:
        z = alpha * x.astype(np.float64)
        sm = np.exp(z - z.max()); sm /= sm.sum()
        want += math.log(n) + float(np.sum(sm * np.log(sm)))
    want /= len(rows)
    for theta in ((511, 0, 1), (100, 0, 77)):
        assert abs(cal.objective(rows, theta, alpha) - want) < 1e-12


def test_objective_depends_only_on_scores_over_their_sum():
    """With renormalisation the reciprocal cancels: q_j = s_j / Z exactly (checked with fractions),
    so the objective equals -H - sum sm_j log s_j + log Z."""
    rng = np.random.default_rng(1)
    n, theta, alpha = 32, (700, 9, 40), 1 / 8
    assert orc.check_params(*theta, n) == 0
    x = rng.integers(-60, 60, size=n).astype(np.int8)
    p, Z, rho = orc.row(x, theta, orc.MODE_U16)
    m = int(x.max())
    s = [theta[0] - theta[1] * min(m - int(v), theta[2]) for v in x]
    assert Z == sum(s) and all(Fraction(int(pj), int(p.sum())) == Fraction(sj, Z) for pj, sj in zip(p, s))
    z = alpha * x.astype(np.float64); sm = np.exp(z - z.max()); sm /= sm.sum()
    want = float(np.sum(sm * np.log(sm)) - np.sum(sm * np.log(np.array(s, dtype=np.float64))) + math.log(Z))
    assert abs(cal.objective(x[None, :], theta, alpha) - want) < 1e-12
    assert cal.objective(x[None, :], theta, alpha) >= 0.0          # KL is non-negative


def test_candidates_stay_in_band_and_order():
    for n in (16, 64, 128, 512):
        c = cal.candidates(n, (4, 127, 9, 0, 127, 5, 7))
        assert c and all(orc.check_params(B, S, D, n) == 0 for B, S, D in c)
        assert [(D, S, B) for B, S, D in c] == sorted((D, S, B) for B, S, D in c)


def test_calibrate_picks_the_minimum():
    rng = np.random.default_rng(2)
    rows = np.clip(np.rint(rng.normal(0, 20, size=(6, 64))), -128, 127).astype(np.int8)
    grid = (8, 120, 28, 1, 9, 4, 120)
    best, val, vals = cal.calibrate(rows, 64, grid, 1 / 16)
    cands = cal.candidates(64, grid)
    assert val == vals.min() and best == cands[int(np.argmin(vals))]
    assert abs(cal.objective(rows, best, 1 / 16) - val) < 1e-15
