"""GPU parity of hccs_calibrate against the calibration oracle (fp64 on both sides)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-9      # fp64 sums in a different order: relative 1e-13 would do; the objective is O(1)


@pytest.mark.parametrize("c,batch,grid,alpha", [
    (1, None, (8, 120, 28, 0, 9, 3, 100), 1 / 16),
    (3, 1, (4, 127, 41, 1, 3, 1, 60), 1 / 32),
    (2, 2, (20, 20, 1, 2, 2, 1, 1), 1 / 8),          # one (D, S) pair, every B of the band
])
def test_grid_scan_matches_oracle(hccs, c, batch, grid, alpha):
    import torch
    from oracle import hccs_calib_oracle as cal
    wl = hccs.workloads.make_config(c, batch=batch)
    Bt, H, Lq, Lk = wl.shape
    x = torch.from_numpy(wl.logits).cuda()
    theta, kl = hccs.hccs_calibrate(x, alpha, grid)
    for h in range(H):
        rows = wl.logits[:, h].reshape(-1, Lk)
        best, val, vals = cal.calibrate(rows, Lk, grid, alpha)
        assert abs(kl[h] - val) <= TOL, (h, kl[h], val)
        got = tuple(int(v) for v in theta[h])
        # the chosen theta is a minimiser (ties within rounding may pick another one)
        assert abs(cal.objective(rows, got, alpha) - val) <= TOL, (h, got, best)
        cands = cal.candidates(Lk, grid)
        assert got in cands
        if np.sum(np.abs(vals - val) <= 10 * TOL) == 1:
            assert got == best


def test_calibrated_theta_beats_the_band_corner(hccs):
    """A fine scan on Gaussian logits must do at least as well as any single candidate, and the
    result must be usable as a parameter table."""
    import torch
    wl = hccs.workloads.make_config(2, batch=64)                  # 64 batch samples, as in the paper
    x = torch.from_numpy(wl.logits).cuda()
    grid = (4, 127, 1, 0, 127, 1, 1)
    theta, kl = hccs.hccs_calibrate(x, 1 / 16, grid)
    assert (kl > 0).all() and (kl < 1.0).all()
    st, bad = hccs.hccs_params_check(theta, 64)
    assert st == hccs.HCCS_OK
    coarse, kl_coarse = hccs.hccs_calibrate(x, 1 / 16, (4, 127, 30, 0, 127, 30, 50))
    assert (kl <= kl_coarse + 1e-12).all()


def test_grid_without_candidates(hccs):
    import torch
    x = torch.zeros((1, 2, 4, 64), dtype=torch.int8, device="cuda")
    with pytest.raises(hccs.HccsError) as ei:
        hccs.hccs_calibrate(x, 0.1, (127, 127, 1, 100, 127, 1, 1))   # S*D far above the band
    assert ei.value.status == hccs.HCCS_ERR_CONSTRAINT
