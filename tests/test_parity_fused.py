"""GPU parity of hccs_attention_fused (int8 Q.K^T -> requantise -> HCCS -> P.V, int32 out) against
the oracle's naive triple loops, bit for bit."""
import numpy as np
import pytest

from gpu_util import assert_same, oracle_mode

pytestmark = pytest.mark.gpu


def _run(hccs, Q, K, V, theta, mult, sh, n_design, flags=0, out_shift=0):
    import torch
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(theta, n_design, out_shift)
    dQ, dK, dV = (torch.from_numpy(a).cuda() for a in (Q, K, V))
    O = torch.full(Q.shape, 0x7EADBEEF, dtype=torch.int32, device="cuda")
    ctx.hccs_attention_fused(dQ, dK, dV, O, mult, sh, flags)
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0, "a bounded device-side wait gave up"
    out = O.cpu().numpy()
    ctx.close()
    return out


def _rand_qkv(rng, shape, lo=-64, hi=64):
    return tuple(rng.integers(lo, hi, size=shape, dtype=np.int8) for _ in range(3))


@pytest.mark.parametrize("L", [1, 37, 128, 200, 256, 640, 1000, 1024])
@pytest.mark.parametrize("flags", [0, 2, 4, 6])
def test_small_heads(hccs, oracle, L, flags):
    rng = np.random.default_rng(1000 + L + flags)
    Bt, H, d = 1, 3, 64
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d))
    theta = hccs.workloads.sample_theta(rng, H, L)
    mult = rng.integers(768, 3841, size=H).astype(np.int32)
    got = _run(hccs, Q, K, V, theta, mult, 20, L, flags)
    want = oracle.attention(Q, K, V, mult, 20, theta, oracle_mode(oracle, flags), threads=8)
    assert_same(got, want, f"fused L={L} flags={flags}")


@pytest.mark.parametrize("L", [1, 100, 128, 384, 500, 512])
@pytest.mark.parametrize("flags", [0, 4, 6])
def test_head_dimension_128(hccs, oracle, L, flags):
    """d = 128 (two 64-byte column halves per Q, K and V tile, 128 output columns), up to 512 keys,
    full-range int8 operands: |acc| reaches 2^21."""
    rng = np.random.default_rng(4000 + L + flags)
    Bt, H, d = 2, 2, 128
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d), -128, 128)
    theta = hccs.workloads.sample_theta(rng, H, 512)
    mult = rng.integers(400, 1500, size=H).astype(np.int32)
    got = _run(hccs, Q, K, V, theta, mult, 20, 512, flags)
    want = oracle.attention(Q, K, V, mult, 20, theta, oracle_mode(oracle, flags), threads=8)
    assert_same(got, want, f"fused d=128 L={L} flags={flags}")


@pytest.mark.parametrize("L", [513, 640, 1000, 1024])
@pytest.mark.parametrize("flags", [0, 4, 6])
def test_head_dimension_128_beyond_512_keys(hccs, oracle, L, flags):
    """d = 128 with more than 512 keys: K and V stream through a ring of four slots (K twice, for the two
    rounds of the first contraction, then V).  More tiles than SMs, so that the ring runs across tiles."""
    rng = np.random.default_rng(4200 + L + flags)
    Bt, H, d = 7, 3, 128
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d), -128, 128)
    theta = hccs.workloads.sample_theta(rng, H, 1024)
    mult = rng.integers(150, 700, size=H).astype(np.int32)
    got = _run(hccs, Q, K, V, theta, mult, 20, 1024, flags)
    want = oracle.attention(Q, K, V, mult, 20, theta, oracle_mode(oracle, flags), threads=8)
    assert_same(got, want, f"fused d=128 L={L} flags={flags}")


def test_head_dimension_128_ring_key_lengths_and_wide_shift(hccs, oracle):
    """The ring with per-batch key lengths (tiles use different numbers of key blocks, also zero keys) and
    with the single-round requantisation flow of shifts above 24."""
    import torch
    rng = np.random.default_rng(4300)
    Bt, H, L, d = 6, 2, 900, 128
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d))
    theta = hccs.workloads.sample_theta(rng, H, 1024)
    mult = rng.integers(300, 900, size=H).astype(np.int32)
    key_len = np.array([900, 0, 1, 513, 129, 640], dtype=np.int32)
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(theta, 1024)
    dQ, dK, dV = (torch.from_numpy(a).cuda() for a in (Q, K, V))
    for flags in (0, 4):
        O = torch.full(Q.shape, 0x7EADBEEF, dtype=torch.int32, device="cuda")
        ctx.hccs_attention_fused_keylen(dQ, dK, dV, O, torch.from_numpy(key_len).cuda(), mult, 20, flags)
        torch.cuda.synchronize()
        assert ctx.hccs_device_status() == 0
        want = oracle.attention(Q, K, V, mult, 20, theta, oracle_mode(oracle, flags), threads=8, key_len=key_len)
        assert_same(O.cpu().numpy(), want, f"ring with key lengths, flags={flags}")
    mult_wide = (mult.astype(np.int64) * 64).astype(np.int32) // 8         # shift 26: the 64-bit flow
    O = torch.full(Q.shape, 0x7EADBEEF, dtype=torch.int32, device="cuda")
    ctx.hccs_attention_fused(dQ, dK, dV, O, mult_wide, 26, 0)
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0
    want = oracle.attention(Q, K, V, mult_wide, 26, theta, 0, threads=8)
    assert_same(O.cpu().numpy(), want, "ring, shift 26")
    ctx.close()


def test_head_dimension_128_many_tiles_and_wide_shift(hccs, oracle):
    """More tiles than SMs (persistent CTAs take several), and the 64-bit requantisation flow."""
    rng = np.random.default_rng(4100)
    Bt, H, L, d = 10, 5, 512, 128
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d))
    theta = hccs.workloads.sample_theta(rng, H, L)
    for sh, lo, hi in ((21, 768, 3841), (28, 4096, 8192)):
        mult = rng.integers(lo, hi, size=H).astype(np.int32)
        got = _run(hccs, Q, K, V, theta, mult, sh, L)
        want = oracle.attention(Q, K, V, mult, sh, theta, 0, threads=16)
        assert_same(got, want, f"fused d=128 sh={sh}")


def test_full_range_int8_and_saturating_requant(hccs, oracle):
    """Operands over all of int8 (|acc| up to 2^20) with multipliers that drive the logits into
    the int8 clamp; also OUT_SHIFT = 1 and a table designed for more keys than the call uses."""
    rng = np.random.default_rng(5)
    Bt, H, L, d = 2, 2, 256, 64
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d), -128, 128)
    theta = hccs.workloads.sample_theta(rng, H, 512)
    mult = np.array([8191, 37], dtype=np.int32)
    for sh, out_shift in ((20, 0), (16, 1), (31, 0)):
        if mult.max() >= 2 ** (sh - 1):
            continue
        got = _run(hccs, Q, K, V, theta, mult, sh, 512, 0, out_shift)
        want = oracle.attention(Q, K, V, mult, sh, theta, 0, out_shift, threads=8)
        assert_same(got, want, f"fused full-range sh={sh} os={out_shift}")


@pytest.mark.parametrize("sh,mults", [(24, [0, 1, 8191]), (14, [8191, 100, 3]), (8, [127, 1, 64]),
                                      (2, [1, 0, 1]), (25, [8191, 0, 1])])
@pytest.mark.parametrize("flags", [0, 4])
def test_requantisation_corner_cases(hccs, oracle, sh, mults, flags):
    """Multipliers 0 and 1, the largest multiplier each shift admits, tiny and large shifts (both
    requantisation flows of the kernel), on a ragged length with full-range int8 operands."""
    rng = np.random.default_rng(77 + sh + flags)
    Bt, H, L, d = 2, 3, 200, 64
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d), -128, 128)
    theta = hccs.workloads.sample_theta(rng, H, L)
    mult = np.array(mults, dtype=np.int32)
    got = _run(hccs, Q, K, V, theta, mult, sh, L, flags)
    want = oracle.attention(Q, K, V, mult, sh, theta, oracle_mode(oracle, flags), threads=8)
    assert_same(got, want, f"fused requant sh={sh} mult={mults} flags={flags}")


def test_config5_every_head_slice(hccs, oracle):
    """The benchmark's fused workload at full size: every one of the 384 (batch, head) slices is
    recomputed by the oracle (about 40 core-seconds, spread over the host cores)."""
    import os
    wl = hccs.workloads.make_config(5)
    got = _run(hccs, wl.Q, wl.K, wl.V, wl.theta, wl.requant_mult, wl.requant_shift, wl.n_design)
    want = oracle.attention(wl.Q, wl.K, wl.V, wl.requant_mult, wl.requant_shift, wl.theta,
                            threads=os.cpu_count() or 1)
    assert_same(got, want, "config5, all head slices")


def test_unsupported_shapes_are_refused(hccs):
    import torch
    ctx = hccs.Context(0)
    ctx.hccs_params_upload([(31, 1, 20)] * 2, 1024)
    for L, d in ((128, 32), (2048, 64), (1040, 64), (1040, 128), (128, 96)):
        q = torch.zeros((1, 2, L, d), dtype=torch.int8, device="cuda")
        o = torch.zeros((1, 2, L, d), dtype=torch.int32, device="cuda")
        with pytest.raises(hccs.HccsError) as ei:
            ctx.hccs_attention_fused(q, q, q, o, [1000, 1000], 20, 0)
        assert ei.value.status in (hccs.HCCS_ERR_UNSUPPORTED, hccs.HCCS_ERR_CONSTRAINT)
    q = torch.zeros((1, 2, 128, 64), dtype=torch.int8, device="cuda")
    o = torch.zeros((1, 2, 128, 64), dtype=torch.int32, device="cuda")
    with pytest.raises(hccs.HccsError) as ei:
        ctx.hccs_attention_fused(q, q, q, o, [1000, 1000], 20, hccs.HCCS_OUT_U16)
    assert ei.value.status == hccs.HCCS_ERR_UNSUPPORTED
    ctx.close()


@pytest.mark.parametrize("d", [64, 128])
def test_fp32_dequantised_output(hccs, oracle, d):
    """O_f32 = float(int32 O) * scale_h: within 1e-6 relative of the exact product (fp64 from the oracle)."""
    import torch
    rng = np.random.default_rng(9)
    Bt, H, L = 1, 3, 384
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d), -128, 128)
    theta = hccs.workloads.sample_theta(rng, H, L)
    mult = rng.integers(768, 3841, size=H).astype(np.int32) // (d // 64)
    scale = np.array([0.03125 / 255, 1.7e-3, 0.4], dtype=np.float32)
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(theta, L)
    dQ, dK, dV = (torch.from_numpy(a).cuda() for a in (Q, K, V))
    O = torch.empty(Q.shape, dtype=torch.float32, device="cuda")
    ctx.hccs_attention_fused_f32(dQ, dK, dV, O, scale, mult, 20, 0)
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0
    want = oracle.attention(Q, K, V, mult, 20, theta, 0, threads=8).astype(np.float64) * \
        scale.astype(np.float64).reshape(1, H, 1, 1)
    got = O.cpu().numpy().astype(np.float64)
    err = np.abs(got - want)
    assert (err <= 1e-6 * np.abs(want)).all(), float((err / np.maximum(np.abs(want), 1e-300)).max())
    assert np.abs(want).max() > 0
    ctx.close()


@pytest.mark.parametrize("d,L", [(64, 1024), (64, 300), (128, 512)])
@pytest.mark.parametrize("flags,sh", [(0, 20), (4, 20), (0, 27), (6, 26)])
def test_key_length_mask(hccs, oracle, d, L, flags, sh):
    """hccs_attention_fused_keylen: per-batch key lengths (0, 1, a block edge, ragged, L and beyond L),
    alone and with the causal rule."""
    import torch
    rng = np.random.default_rng(6000 + d + L + flags + sh)
    Bt, H = 7, 2
    Q, K, V = _rand_qkv(rng, (Bt, H, L, d), -128, 128)
    theta = hccs.workloads.sample_theta(rng, H, L)
    mult = rng.integers(300, 1200, size=H).astype(np.int32) * (6 if sh > 24 else 1)
    key_len = np.array([0, 1, 128, min(L, 257), L - 1, L, L + 50], dtype=np.int32)
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(theta, L)
    dQ, dK, dV = (torch.from_numpy(a).cuda() for a in (Q, K, V))
    O = torch.full(Q.shape, 0x7EADBEEF, dtype=torch.int32, device="cuda")
    ctx.hccs_attention_fused_keylen(dQ, dK, dV, O, torch.from_numpy(key_len).cuda(), mult, sh, flags)
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0
    want = oracle.attention(Q, K, V, mult, sh, theta, oracle_mode(oracle, flags), threads=16, key_len=key_len)
    assert_same(O.cpu().numpy(), want, f"fused key_len d={d} L={L} flags={flags} sh={sh}")
    ctx.close()


@pytest.mark.parametrize("shape,flags", [((2, 3, 333, 64), 0), ((2, 3, 333, 64), 4), ((1, 2, 1024, 64), 2),
                                         ((1, 2, 200, 128), 0), ((2, 2, 512, 128), 6)])
def test_int8_output(hccs, oracle, shape, flags):
    """hccs_attention_fused_i8: the int32 result requantised per head, bit for bit against the oracle's
    output requantisation of the oracle's attention; multipliers chosen so that both clamps are hit."""
    import torch
    rng = np.random.default_rng(5000 + shape[2] + flags)
    Bt, H, L, d = shape
    Q, K, V = _rand_qkv(rng, shape, -128, 128)
    n_design = max(L, 512)
    theta = hccs.workloads.sample_theta(rng, H, n_design)
    mult = (rng.integers(768, 3841, size=H) * 64 // d).astype(np.int32)
    out_mult = rng.integers(100, 8192, size=H).astype(np.int32)
    out_mult[0] = 8191
    acc = oracle.attention(Q, K, V, mult, 20, theta, oracle_mode(oracle, flags), threads=8)
    # a shift that puts the largest accumulator of head 0 near 300: both clamps and the middle are reached
    out_sh = int(min(31, max(1, np.floor(np.log2(max(int(np.abs(acc[:, 0]).max()), 1) * 8191 / 300.0)))))
    ctx = hccs.Context(0)
    ctx.hccs_params_upload(theta, n_design)
    dQ, dK, dV = (torch.from_numpy(a).cuda() for a in (Q, K, V))
    O = torch.full(shape, 0x5A, dtype=torch.int8, device="cuda")
    ctx.hccs_attention_fused_i8(dQ, dK, dV, O, out_mult, out_sh, mult, 20, flags)
    torch.cuda.synchronize()
    assert ctx.hccs_device_status() == 0
    want = oracle.requant_output(acc, out_mult, out_sh)
    if np.abs(acc[:, 0]).max() > 300:       # (1024 keys of full-range logits give all-zero uint8 probabilities)
        assert (want == 127).any() and (want == -128).any() and (np.abs(want.astype(np.int32)) < 100).any()
    assert_same(O.cpu().numpy(), want, f"fused int8 output {shape} flags={flags}")
    # bad arguments are refused before anything is launched
    for om, osh in ((out_mult, 0), (out_mult, 32), (np.full(H, 8192, np.int32), 10), (np.full(H, -1, np.int32), 10)):
        with pytest.raises(hccs.HccsError) as ei:
            ctx.hccs_attention_fused_i8(dQ, dK, dV, O, om, osh, mult, 20, flags)
        assert ei.value.status == hccs.HCCS_ERR_INVALID_ARG
    ctx.close()
