"""Helpers for the GPU parity tests: move numpy inputs to the device, call the C ABI through the
binding, bring the result back, and guard the output buffer with canary bytes."""
import numpy as np

CANARY = 0xA5
PAD = 256


def oracle_mode(orc, flags):
    """Library flags -> the oracle's own mode bits."""
    import paper_2604_02292_b200 as pkg
    m = 0
    if flags & pkg.HCCS_OUT_U16:
        m |= orc.MODE_U16
    if flags & pkg.HCCS_RECIP_CLB:
        m |= orc.MODE_CLB
    if flags & pkg.HCCS_CAUSAL:
        m |= orc.MODE_CAUSAL
    return m


def forward_np(ctx, x, flags=0, misalign=0, inplace=False, out_misalign=None):
    """hccs_forward on a numpy int8 [B,H,Lq,Lk] array; returns the numpy result.

    The output lives inside a larger byte buffer filled with a canary value, `misalign` bytes off
    a 256-byte boundary (also applied to the input; `out_misalign` sets the output's offset in bytes on
    its own); bytes around it must come back untouched."""
    import torch
    import paper_2604_02292_b200 as pkg
    x = np.ascontiguousarray(x, dtype=np.int8)
    u16 = bool(flags & pkg.HCCS_OUT_U16)
    osz = 2 if u16 else 1
    n = x.size
    dev = torch.device("cuda", ctx.device)
    xin_buf = torch.full((n + 2 * PAD,), 0x11, dtype=torch.uint8, device=dev)
    xin = xin_buf[PAD + misalign: PAD + misalign + n].view(torch.int8)
    xin.copy_(torch.from_numpy(x.reshape(-1)))
    xin = xin.view(x.shape)
    if inplace:
        assert not u16
        ctx.hccs_forward(xin, xin.view(torch.uint8), flags)
        torch.cuda.synchronize()
        out = xin.view(torch.uint8).cpu().numpy()
        guard = xin_buf.cpu().numpy()
        assert (guard[:PAD + misalign] == 0x11).all() and (guard[PAD + misalign + n:] == 0x11).all()
        return out
    obuf = torch.full((n * osz + 2 * PAD,), CANARY, dtype=torch.uint8, device=dev)
    off = PAD + (misalign * osz if out_misalign is None else out_misalign)
    oview = obuf[off: off + n * osz]
    probs = (oview.view(torch.uint16) if u16 else oview).view(x.shape)
    ctx.hccs_forward(xin, probs, flags)
    torch.cuda.synchronize()
    host = obuf.cpu().numpy()
    assert (host[:off] == CANARY).all(), "bytes before the output were overwritten"
    assert (host[off + n * osz:] == CANARY).all(), "bytes after the output were overwritten"
    assert (xin.cpu().numpy() == x).all(), "the input was modified"
    res = host[off: off + n * osz]
    return (res.view(np.uint16) if u16 else res).reshape(x.shape).copy()


def assert_same(got, want, what=""):
    if got.shape != want.shape or not (got == want).all():
        bad = np.argwhere(got != want)
        first = tuple(bad[0])
        raise AssertionError(f"{what}: {len(bad)} mismatches of {got.size}; first at {first}: "
                             f"gpu={got[first]} oracle={want[first]}")
