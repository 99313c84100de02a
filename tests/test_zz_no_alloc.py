"""The allocation-free entry point (hccs_forward_static_scratch).

Some users of this library run where device memory may not be allocated: inside an allocator
callback, in a serving process that gave all device memory away at start-up, or in a loop whose
latency budget has no room for a call that may synchronise the device.  For them the library offers
one call that keeps its working memory (parameter table, status word) in a fixed array inside the
library image.  This test calls it several times in a row through the C ABI -- the array is shared
between calls and keeps the previous call's contents, so a call must not be disturbed by the one
before it -- and compares each result bit for bit with the CPU oracle and with the regular entry
point (integer outputs: the tolerance is zero).  It also checks the property the call exists for:
the device memory in use does not change across calls.
The file sorts last so that a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest

from gpu_util import oracle_mode

pytestmark = pytest.mark.gpu


def _run_both(hccs, oracle, ctx, wl, flags):
    import torch
    x = torch.from_numpy(wl.logits).cuda()
    odt = torch.uint16 if flags & hccs.HCCS_OUT_U16 else torch.uint8
    regular = torch.empty(wl.logits.shape, dtype=odt, device="cuda")
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    ctx.hccs_forward(x, regular, flags)
    got = torch.full(wl.logits.shape, 0x5A, dtype=odt, device="cuda")
    word = hccs.hccs_forward_static_scratch(wl.theta, wl.n_design, x, got, flags, check_timeout=True)
    torch.cuda.synchronize()
    assert word == 0
    want = oracle.forward(wl.logits, wl.theta, oracle_mode(oracle, flags), threads=8)
    assert np.array_equal(got.cpu().numpy(), want), (wl.name, flags, "against the oracle")
    assert torch.equal(got.view(torch.uint8), regular.view(torch.uint8)), (wl.name, flags, "against hccs_forward")


def test_calls_in_a_row_match_the_oracle_and_hccs_forward(hccs, oracle):
    ctx = hccs.Context(0)
    # first call: long causal rows, several heads; second call: another table, another shape,
    # fewer heads -- stale table entries and the status word of the first call must not leak
    first = hccs.workloads.make_rows(901, (2, 5, 70, 4096), kind="gauss")
    second = hccs.workloads.make_rows(902, (3, 2, 33, 512), kind="laplace")
    _run_both(hccs, oracle, ctx, first, hccs.HCCS_CAUSAL)
    _run_both(hccs, oracle, ctx, second, 0)
    # and once more with the other output type and the leading-bit reciprocal
    _run_both(hccs, oracle, ctx, first, hccs.HCCS_OUT_U16 | hccs.HCCS_RECIP_CLB)
    _run_both(hccs, oracle, ctx, second, hccs.HCCS_RECIP_CLB)
    ctx.close()


def test_device_memory_in_use_does_not_change(hccs, oracle):
    """Free device memory (driver's count) and torch's own count are the same before and after the
    second and the third call; the first call on a device may still load the kernel image."""
    import torch
    wl = hccs.workloads.make_rows(903, (2, 3, 40, 1024), kind="gauss")
    x = torch.from_numpy(wl.logits).cuda()
    got = torch.empty(wl.logits.shape, dtype=torch.uint8, device="cuda")
    hccs.hccs_forward_static_scratch(wl.theta, wl.n_design, x, got, 0, check_timeout=True)     # first call
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0 = torch.cuda.memory_allocated()
    for _ in range(2):
        got.fill_(0x5A)
        word = hccs.hccs_forward_static_scratch(wl.theta, wl.n_design, x, got, 0, check_timeout=True)
        torch.cuda.synchronize()
        assert word == 0
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, "free device memory changed across an allocation-free call"
        assert torch.cuda.memory_allocated() == alloc0
    want = oracle.forward(wl.logits, wl.theta, 0, threads=8)
    assert np.array_equal(got.cpu().numpy(), want)


def test_limits_are_reported(hccs):
    import torch
    x = torch.zeros((1, 300, 1, 64), dtype=torch.int8, device="cuda")
    p = torch.zeros((1, 300, 1, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(hccs.HccsError) as ei:              # more heads than the fixed table holds
        hccs.hccs_forward_static_scratch([(300, 3, 85)] * 300, 64, x, p)
    assert ei.value.status == hccs.HCCS_ERR_UNSUPPORTED
    x = torch.zeros((1, 2, 4, 40), dtype=torch.int8, device="cuda")
    p = torch.zeros((1, 2, 4, 40), dtype=torch.uint8, device="cuda")
    with pytest.raises(hccs.HccsError) as ei:              # row length not a multiple of 16
        hccs.hccs_forward_static_scratch([(300, 3, 85)] * 2, 64, x, p)
    assert ei.value.status == hccs.HCCS_ERR_UNSUPPORTED
    with pytest.raises(hccs.HccsError) as ei:              # inadmissible table
        hccs.hccs_forward_static_scratch([(200, 3, 85)] * 2, 64, x, p)
    assert ei.value.status == hccs.HCCS_ERR_CONSTRAINT
