"""Calibrate theta per head on synthetic logits with hccs_calibrate (grid scan, Eq. 10) and report
how close the calibrated HCCS is to an fp64 softmax -- next to the uncalibrated, uniformly drawn
theta of the workload.  Needs a GPU.

    python tests/calibration_report.py [--alpha 0.0625]

A report script, kept with the test infrastructure (it holds softmax / KL arithmetic of its own, which has
no place in the library package).

Per workload: 64 batch entries are the calibration set (as in the paper's Section "Calibration");
the report is taken on the following 16 entries.  Columns: mean over rows of max_j |p_j/T - sm_j|
and of KL(sm || q) for the int16 output path, q = row renormalised to one.
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def _fidelity(p, x, alpha, valid=None):
    p = p.astype(np.float64)
    z = alpha * x.astype(np.float64)
    if valid is not None:
        z = np.where(valid, z, -np.inf)
    z -= z.max(axis=-1, keepdims=True)
    sm = np.exp(z)
    sm /= sm.sum(axis=-1, keepdims=True)
    q = p / np.maximum(p.sum(axis=-1, keepdims=True), 1.0)
    with np.errstate(divide="ignore", invalid="ignore"):
        kl = np.where((sm > 0) & (q > 0), sm * (np.log(sm) - np.log(np.where(q > 0, q, 1.0))), 0.0).sum(axis=-1)
    return float(np.abs(p / 32767.0 - sm).max(axis=-1).mean()), float(kl.mean())


def main():
    import torch
    import paper_2604_02292_b200 as pkg
    ap = argparse.ArgumentParser()
    ap.add_argument("--alpha", type=float, default=1 / 16)
    args = ap.parse_args()
    ctx = pkg.Context(0)
    print("| workload | theta | mean max-abs (u16/div) | mean KL |")
    print("|---|---|---|---|")
    for c, batch in ((2, 80), (4, 80)):
        wl = pkg.workloads.make_config(c, batch=batch)
        Bt, H, Lq, Lk = wl.shape
        x = torch.from_numpy(wl.logits).cuda()
        grid = (2, 127, 1, 0, 127, 1, 1)
        theta_cal, kl_cal = pkg.hccs_calibrate(x[:64].contiguous(), args.alpha, grid)
        test = wl.logits[64:]
        for name, theta in (("uniform in band", wl.theta), ("calibrated", theta_cal)):
            ctx.hccs_params_upload(theta, Lk)
            p = torch.empty(test.shape, dtype=torch.uint16, device="cuda")
            ctx.hccs_forward(x[64:].contiguous(), p, pkg.HCCS_OUT_U16)
            torch.cuda.synchronize()
            err, kl = _fidelity(p.cpu().numpy().reshape(-1, Lk), test.reshape(-1, Lk), args.alpha)
            print(f"| {wl.name} [{Lk} keys], alpha = {args.alpha:g} | {name} | {err:.4f} | {kl:.3f} |")
        print(f"| | calibrated theta per head: {theta_cal.tolist()}; objective on the calibration set "
              f"{np.round(kl_cal, 3).tolist()} | | |")
    ctx.close()


if __name__ == "__main__":
    main()
