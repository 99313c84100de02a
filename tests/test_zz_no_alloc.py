"""The allocation-free entry point (hccs_forward_static_scratch) against hccs_forward.

Some users of this library run where device memory may not be allocated: inside an allocator
callback, in a serving process that gave all device memory away at start-up, or in a loop whose
latency budget has no room for a call that may synchronise the device.  For them the library offers one call that keeps its working memory (parameter
table, row counter, status word) in a fixed array inside the library image.  This test calls it
twice in a row through the C ABI -- the array is shared between calls and keeps the previous
call's contents, so the second call must not be disturbed by the first -- and compares each
result bit for bit with the regular entry point (integer outputs: the tolerance is zero).
The file sorts last so that a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _run_both(hccs, ctx, wl, flags):
    import torch
    x = torch.from_numpy(wl.logits).cuda()
    odt = torch.uint16 if flags & hccs.HCCS_OUT_U16 else torch.uint8
    want = torch.empty(wl.logits.shape, dtype=odt, device="cuda")
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    ctx.hccs_forward(x, want, flags)
    got = torch.full(wl.logits.shape, 0x5A, dtype=odt, device="cuda")
    word = hccs.hccs_forward_static_scratch(wl.theta, wl.n_design, x, got, flags, check_timeout=True)
    torch.cuda.synchronize()
    assert word == 0
    assert torch.equal(got.view(torch.uint8), want.view(torch.uint8)), (wl.name, flags)


def test_two_calls_in_a_row_match_hccs_forward(hccs):
    ctx = hccs.Context(0)
    # first call: long causal rows, several heads; second call: another table, another shape,
    # fewer heads -- stale table entries, counter and status of the first call must not leak
    first = hccs.workloads.make_rows(901, (2, 5, 70, 4096), kind="gauss")
    second = hccs.workloads.make_rows(902, (3, 2, 33, 512), kind="laplace")
    _run_both(hccs, ctx, first, hccs.HCCS_CAUSAL)
    _run_both(hccs, ctx, second, 0)
    # and once more with the other output type and the leading-bit reciprocal
    _run_both(hccs, ctx, first, hccs.HCCS_OUT_U16 | hccs.HCCS_RECIP_CLB)
    ctx.close()


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
