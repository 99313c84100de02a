"""Device-side waits give up after a limit, report it in the status word and leave the GPU usable.

No test here makes a GPU hang, trap or fault: the wait that runs out is a wait on a barrier that is
never completed, taken with a short limit through the same wait routines the TMA-staged kernels
use (hccs_debug_wait_timeout); the kernel returns by itself and the host reads the status word.
Also covered: launches of one context that overlap on the GPU (two streams) through the long-row
kernel, which keeps no per-launch state on the device.
"""
import ctypes

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode,bit", [(0, 1), (1, 2)])
def test_a_wait_that_runs_out_sets_the_status_word(hccs, mode, bit):
    import torch
    ctx = hccs.Context(0)
    assert ctx.hccs_device_status() == 0
    ctx.hccs_debug_wait_timeout(mode, 100_000)
    word = ctypes.c_uint32(0)
    st = hccs.raw().hccs_device_status(ctx._h, ctypes.byref(word), None)
    assert st == hccs.HCCS_ERR_DEVICE_TIMEOUT
    assert word.value == bit
    assert ctx.hccs_device_status() == 0, "reading the status word clears it"
    # the context is as usable as before
    wl = hccs.workloads.make_rows(31, (1, 2, 16, 64))
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    x = torch.from_numpy(wl.logits).cuda()
    p = torch.empty(wl.logits.shape, dtype=torch.uint8, device="cuda")
    ctx.hccs_forward(x, p, 0)
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0
    ctx.close()


def test_probe_arguments_are_checked(hccs):
    ctx = hccs.Context(0)
    for mode, limit in ((2, 1000), (-1, 1000), (0, 0), (0, 10_000_001)):
        with pytest.raises(hccs.HccsError) as ei:
            ctx.hccs_debug_wait_timeout(mode, limit)
        assert ei.value.status == hccs.HCCS_ERR_INVALID_ARG
    ctx.close()


@pytest.mark.parametrize("flags", [0, 4])
def test_overlapping_launches_of_one_context(hccs, oracle, flags):
    """Two hccs_forward calls of one context on two streams, both through the long-row kernel
    (16384 keys), each checked against the oracle: the launches share nothing but the table."""
    import torch
    from gpu_util import oracle_mode
    wl_a = hccs.workloads.make_rows(41, (1, 2, 150, 16384), kind="gauss")
    rng = np.random.default_rng(42)
    xb = rng.integers(-128, 128, size=wl_a.logits.shape, dtype=np.int8)
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(wl_a.theta, wl_a.n_design)
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    xa_d, xb_d = torch.from_numpy(wl_a.logits).cuda(), torch.from_numpy(xb).cuda()
    pa = torch.full(xa_d.shape, 0x5A, dtype=torch.uint8, device="cuda")
    pb = torch.full(xa_d.shape, 0x5A, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    for _ in range(3):                      # several rounds, so that the two grids do meet
        ctx.hccs_forward(xa_d, pa, flags, stream=s1)
        ctx.hccs_forward(xb_d, pb, flags, stream=s2)
    torch.cuda.synchronize()
    mode = oracle_mode(oracle, flags)
    assert np.array_equal(pa.cpu().numpy(), oracle.forward(wl_a.logits, wl_a.theta, mode, threads=8))
    assert np.array_equal(pb.cpu().numpy(), oracle.forward(xb, wl_a.theta, mode, threads=8))
    assert ctx.hccs_device_status() == 0
    ctx.close()
