"""Seeded random sweeps over the public entry points against the oracle, bit for bit: shapes, modes, masks,
alignments, design lengths and output shifts drawn together, so that combinations no hand-written case
names go through every dispatch path of the library."""
import numpy as np
import pytest

from gpu_util import assert_same, forward_np, oracle_mode

pytestmark = pytest.mark.gpu

ROW_LENGTHS = [1, 5, 16, 31, 32, 48, 64, 77, 96, 100, 128, 144, 160, 200, 256, 272, 320, 500, 512, 640, 768,
               1000, 1024, 1040, 1536, 2048, 2100, 3072, 4096, 4112, 6144, 8192, 9000]


@pytest.mark.parametrize("seed", range(40))
def test_random_forward_calls(hccs, oracle, seed):
    import torch
    rng = np.random.default_rng(90_000 + seed)
    Lk = int(rng.choice(ROW_LENGTHS))
    Lq = int(rng.integers(1, 70))
    H = int(rng.integers(1, 6))
    Bt = int(rng.integers(1, 5))
    while Bt * H * Lq * Lk > (1 << 22):
        Lq = max(1, Lq // 2)
    flags = int(rng.integers(0, 8))
    out_shift = int(rng.choice([0, 0, 0, 1, 2, 3, 6]))
    n_design = Lk if rng.random() < 0.6 else int(min(32767, Lk + rng.integers(1, 200)))
    kind = str(rng.choice(["gauss", "laplace", "uniform", "extreme", "const"]))
    wl = hccs.workloads.make_rows(91_000 + seed, (Bt, H, Lq, Lk), n_design=n_design, kind=kind)
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(wl.theta, wl.n_design, out_shift)
    mode = oracle_mode(oracle, flags)
    what = f"seed={seed} shape={wl.shape} n_design={n_design} flags={flags} os={out_shift} kind={kind}"
    if rng.random() < 0.35:
        # per-batch key lengths through hccs_forward_keylen
        key_len = rng.integers(-2, Lk + 3, size=Bt).astype(np.int32)
        x = torch.from_numpy(wl.logits).cuda()
        odt = torch.uint16 if flags & 1 else torch.uint8
        p = torch.full(wl.logits.shape, 0x5A, dtype=odt, device="cuda")
        ctx.hccs_forward_keylen(x, p, torch.from_numpy(key_len).cuda(), flags)
        torch.cuda.synchronize()
        want = oracle.forward(wl.logits, wl.theta, mode, out_shift, threads=4, key_len=np.clip(key_len, 0, Lk))
        assert_same(p.cpu().numpy(), want, what + f" key_len={key_len.tolist()}")
    else:
        misalign = int(rng.choice([0, 0, 1, 4, 16, 32, 48]))
        inplace = bool(rng.random() < 0.2) and not (flags & 1)
        got = forward_np(ctx, wl.logits, flags, misalign=misalign, inplace=inplace)
        want = oracle.forward(wl.logits, wl.theta, mode, out_shift, threads=4)
        assert_same(got, want, what + f" misalign={misalign} inplace={inplace}")
    assert ctx.hccs_device_status() == 0
    ctx.close()


@pytest.mark.parametrize("seed", range(24))
def test_random_fused_calls(hccs, oracle, seed):
    import torch
    rng = np.random.default_rng(95_000 + seed)
    d = int(rng.choice([64, 128]))
    L = int(rng.choice([1, 17, 100, 128, 129, 300, 512, 513, 700, 1000, 1024]))
    H = int(rng.integers(1, 4))
    Bt = int(rng.integers(1, 4))
    flags = int(rng.choice([0, 2, 4, 6]))
    sh = int(rng.choice([12, 20, 20, 24, 26]))
    out_shift = int(rng.choice([0, 0, 1, 2, 4]))
    lo, hi = (-128, 128) if rng.random() < 0.5 else (-64, 64)
    Q, K, V = (rng.integers(lo, hi, size=(Bt, H, L, d), dtype=np.int8) for _ in range(3))
    theta = hccs.workloads.sample_theta(rng, H, 1024)
    # multipliers that keep the logits spread over the int8 range for this shift and head dimension
    mult = np.maximum(1, (rng.integers(768, 3841, size=H) * 64 // d * 2.0 ** (sh - 20)).astype(np.int64))
    mult = np.minimum(mult, min(8191, 2 ** (sh - 1) - 1)).astype(np.int32)
    key_len = rng.integers(0, L + 1, size=Bt).astype(np.int32) if rng.random() < 0.4 else None
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(theta, 1024, out_shift)
    dQ, dK, dV = (torch.from_numpy(a).cuda() for a in (Q, K, V))
    O = torch.full(Q.shape, 0x7EADBEEF, dtype=torch.int32, device="cuda")
    what = f"seed={seed} shape={(Bt, H, L, d)} flags={flags} sh={sh} os={out_shift} mult={mult.tolist()} key_len={None if key_len is None else key_len.tolist()}"
    try:
        if key_len is None:
            ctx.hccs_attention_fused(dQ, dK, dV, O, mult, sh, flags)
        else:
            ctx.hccs_attention_fused_keylen(dQ, dK, dV, O, torch.from_numpy(key_len).cuda(), mult, sh, flags)
    except hccs.HccsError as e:
        # the only refusal these draws can meet: a multiplier too large for the single-multiply flow of this shift
        assert e.status == hccs.HCCS_ERR_UNSUPPORTED, what
        ctx.close()
        return
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0, what
    want = oracle.attention(Q, K, V, mult, sh, theta, oracle_mode(oracle, flags), out_shift, threads=8, key_len=key_len)
    assert_same(O.cpu().numpy(), want, what)
    ctx.close()
