"""GPU parity at the full benchmark sizes (configs 2-4), every element against the oracle,
in the launch configuration the benchmark times."""
import numpy as np
import pytest

from gpu_util import assert_same, oracle_mode

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("c", [2, 3, 4])
def test_full_size_config(hccs, oracle, c):
    import torch
    wl = hccs.workloads.make_config(c)
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    x = torch.from_numpy(wl.logits).cuda()
    for extra in (0, hccs.HCCS_RECIP_CLB, hccs.HCCS_OUT_U16):
        flags = wl.flags | extra
        p = torch.empty(wl.logits.shape, dtype=torch.uint16 if flags & 1 else torch.uint8, device="cuda")
        ctx.hccs_forward(x, p, flags)
        torch.cuda.synchronize()
        want = oracle.forward(wl.logits, wl.theta, oracle_mode(oracle, flags), threads=8)
        assert_same(p.cpu().numpy(), want, f"config{c} flags={flags}")
        del p
    assert ctx.hccs_device_status() == 0
    ctx.close()
