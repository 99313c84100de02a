"""Fidelity of HCCS against an exact fp64 exp-softmax on the synthetic workloads (a report, not a
gate).  TEST INFRASTRUCTURE: uses only the CPU oracle and the seeded input generators.

    python -m oracle.fidelity_report            # prints a markdown table

The paper states its calibration objective on raw int8 logits without a dequantisation scale
(Eq. 10), so the softmax is taken of alpha*x for a few alpha.  Reported per workload, mode and
alpha, over a seeded sample of rows: the mean and maximum over rows of max_j |p_j/T - softmax_j|,
and the mean KL(softmax || q) with q the HCCS row renormalised to sum one (zero bins floored at
1e-12).  theta is drawn uniformly from the admissible band, not calibrated, so these numbers say
how far an uncalibrated surrogate is from softmax, not what the paper's calibrated heads reach.
"""
from __future__ import annotations

import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

from oracle import hccs_oracle as orc                      # noqa: E402
from paper_2604_02292_b200 import workloads                # noqa: E402

ALPHAS = (1 / 32, 1 / 16, 1 / 8)
MODES = (("u8/div", 0, 255.0), ("u16/div", orc.MODE_U16, 32767.0), ("u8/CLB", orc.MODE_CLB, 255.0))


def softmax64(x, valid):
    z = np.where(valid, x, -np.inf)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def report(max_rows: int = 4096, seed: int = 0):
    rng = np.random.default_rng(seed)
    lines = ["| workload | mode | alpha | mean max-abs | worst max-abs | mean KL |", "|---|---|---|---|---|---|"]
    for c, batch in ((1, None), (2, 16), (3, 2), (4, 1)):
        wl = workloads.make_config(c, batch=batch)
        Bt, H, Lq, Lk = wl.shape
        causal = bool(wl.flags & workloads.FLAG_CAUSAL)
        for name, mode, T in MODES:
            m = mode | (orc.MODE_CAUSAL if causal else 0)
            p = orc.forward(wl.logits, wl.theta, m, threads=os.cpu_count() or 1).reshape(-1, Lk).astype(np.float64)
            x = wl.logits.reshape(-1, Lk).astype(np.float64)
            qi = np.tile(np.arange(Lq), Bt * H)
            pick = rng.choice(x.shape[0], size=min(max_rows, x.shape[0]), replace=False)
            valid = (np.arange(Lk)[None, :] <= qi[pick, None] + (Lk - Lq)) if causal else np.ones((pick.size, Lk), bool)
            for alpha in ALPHAS:
                sm = softmax64(alpha * x[pick], valid)
                ph = p[pick]
                err = np.abs(ph / T - sm).max(axis=1)
                q = np.where(valid, np.maximum(ph, 1e-12), 0.0)
                q = q / q.sum(axis=1, keepdims=True)
                with np.errstate(divide="ignore", invalid="ignore"):
                    kl = np.where(sm > 0, sm * (np.log(sm) - np.log(np.where(q > 0, q, 1.0))), 0.0).sum(axis=1)
                lines.append(f"| {wl.name} {list(wl.shape)} | {name} | 1/{round(1 / alpha)} | {err.mean():.4f} | "
                             f"{err.max():.4f} | {kl.mean():.3f} |")
    return "\n".join(lines)


if __name__ == "__main__":
    print(report())
