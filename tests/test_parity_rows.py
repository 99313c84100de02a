"""GPU parity: hccs_forward (through the C ABI) against the CPU oracle, bit for bit."""
import numpy as np
import pytest

from gpu_util import assert_same, forward_np, oracle_mode

pytestmark = pytest.mark.gpu

ALL_FLAGS = list(range(8))     # {u8,u16} x {div,clb} x {plain,causal}


@pytest.fixture(scope="module")
def ctx(hccs):
    c = hccs.Context(0)
    yield c
    c.close()


def _check(ctx, orc, wl, flags, out_shift=0, misalign=0, inplace=False, threads=8, out_misalign=None):
    ctx.hccs_params_upload(wl.theta, wl.n_design, out_shift)
    got = forward_np(ctx, wl.logits, flags, misalign=misalign, inplace=inplace, out_misalign=out_misalign)
    want = orc.forward(wl.logits, wl.theta, oracle_mode(orc, flags), out_shift, threads=threads)
    assert_same(got, want, f"{wl.name} shape={wl.shape} flags={flags} os={out_shift} mis={misalign}")
    assert ctx.hccs_device_status() == 0


@pytest.mark.parametrize("flags", ALL_FLAGS)
def test_config1_all_modes(ctx, oracle, hccs, flags):
    wl = hccs.workloads.make_config(1)
    _check(ctx, oracle, wl, flags)


@pytest.mark.parametrize("c,batch", [(2, 33), (3, 5), (4, 2)])
@pytest.mark.parametrize("flags", ALL_FLAGS)
def test_reduced_configs_all_modes(ctx, oracle, hccs, c, batch, flags):
    wl = hccs.workloads.make_config(c, batch=batch)
    _check(ctx, oracle, wl, flags)


# row lengths around every dispatch boundary: lane-group sizes, two chunks per lane, the
# CTA-per-row kernel, ragged tails and lengths that are no multiple of 16
LENGTHS = [1, 2, 3, 15, 16, 17, 31, 32, 33, 48, 64, 80, 96, 100, 112, 128, 144, 256, 257, 272, 384,
           496, 512, 528, 1000, 1008, 1024, 1040, 2048, 2064, 2304, 4096, 4112, 5000, 8192, 16384, 32752]


@pytest.mark.parametrize("Lk", LENGTHS)
def test_row_lengths(ctx, oracle, hccs, Lk):
    for kind, flags, shape in (("gauss", 0, (2, 3, 7, Lk)), ("uniform", 1, (1, 5, 4, Lk)),
                               ("laplace", 2, (3, 2, 5, Lk)), ("extreme", 3, (1, 1, 9, Lk)),
                               ("const", 0, (1, 2, 3, Lk))):
        wl = hccs.workloads.make_rows(1000 + Lk, shape, kind=kind)
        _check(ctx, oracle, wl, flags)


# the register-resident kernel's shapes with three, five or seven chunks per lane (and 4096 keys)
@pytest.mark.parametrize("Lk", [96, 160, 192, 224, 320, 384, 448, 640, 768, 896, 1280, 1536, 1792, 2560,
                                3072, 3584, 4096,
                                # 16-byte chunks: multiples of 16 whose odd part is 3 ... 15
                                48, 80, 112, 144, 176, 208, 240, 288, 352, 416, 480, 576, 960, 1152, 2304,
                                3328, 4608, 7680,
                                # padded lane groups: the other multiples of 16 up to 4096
                                272, 304, 336, 528, 544, 1008, 1040, 1104, 2064, 2192, 4080,
                                4128, 5024, 6144, 8160, 8192])
@pytest.mark.parametrize("flags", ALL_FLAGS)
def test_odd_chunk_counts(ctx, oracle, hccs, Lk, flags):
    Lq = 70 if flags & 4 else 37                       # several warps, a ragged last warp, causal rows of every length class
    wl = hccs.workloads.make_rows(7000 + Lk + flags, (2, 3, Lq, Lk), kind="gauss")
    _check(ctx, oracle, wl, flags)
    if flags & 4:                                      # square causal heads as well: every chunk-skipping case
        wl = hccs.workloads.make_rows(7100 + Lk, (1, 2, min(Lk, 512), Lk), kind="laplace")
        _check(ctx, oracle, wl, flags)


@pytest.mark.parametrize("Lq,Lk", [(1, 64), (5, 64), (64, 5), (100, 128), (128, 100), (33, 512),
                                   (40, 1024), (7, 2048), (3, 1), (130, 144), (2100, 2048), (300, 4096),
                                   (4100, 4112)])
def test_causal_alignment(ctx, oracle, hccs, Lq, Lk):
    for flags in (4, 5, 6, 7):
        wl = hccs.workloads.make_rows(50 + Lq + Lk, (2, 3, Lq, Lk), kind="gauss")
        _check(ctx, oracle, wl, flags)


def test_shorter_rows_than_designed(ctx, oracle, hccs):
    for Lk in (16, 48, 64, 100):
        wl = hccs.workloads.make_rows(7, (2, 4, 9, Lk), n_design=128, kind="gauss")
        for flags in (0, 1, 2, 3, 4):
            _check(ctx, oracle, wl, flags)


@pytest.mark.parametrize("out_shift", [0, 1, 2, 3, 5, 8])
def test_out_shift(ctx, oracle, hccs, out_shift):
    for Lk in (16, 64, 100, 128, 272, 2048, 4112):
        wl = hccs.workloads.make_rows(3, (2, 3, 8, Lk), kind="gauss")
        for flags in (0, 2, 4):
            _check(ctx, oracle, wl, flags, out_shift=out_shift)


@pytest.mark.parametrize("misalign", [1, 4, 8, 15, 16, 48])
def test_unaligned_pointers(ctx, oracle, hccs, misalign):
    for Lk in (64, 128, 2048, 4096):
        wl = hccs.workloads.make_rows(9, (1, 2, 6, Lk), kind="gauss")
        for flags in (0, 1, 4):
            _check(ctx, oracle, wl, flags, misalign=misalign)


@pytest.mark.parametrize("Lk", [16, 32, 48, 64, 96, 128, 160, 272, 512, 1008, 1024, 2048, 3584, 4096])
def test_sixteen_byte_aligned_tensors(ctx, oracle, hccs, Lk):
    """Tensors that start on a 16-byte but not on a 32-byte boundary stay in the register-resident kernel
    (16-byte chunks, padded lane groups), in every mode."""
    wl = hccs.workloads.make_rows(11000 + Lk, (2, 3, 37, Lk), kind="gauss")
    for flags in ALL_FLAGS:
        _check(ctx, oracle, wl, flags, misalign=16, out_misalign=16)
        _check(ctx, oracle, wl, flags, misalign=32, out_misalign=48)


def test_in_place(ctx, oracle, hccs):
    for Lk in (64, 100, 512, 1024, 4096):
        wl = hccs.workloads.make_rows(21, (2, 2, 10, Lk), kind="gauss")
        for flags in (0, 2, 4):
            _check(ctx, oracle, wl, flags, inplace=True)


@pytest.mark.parametrize("shape,flags", [((400, 4, 64, 64), 0), ((400, 4, 64, 64), 2), ((50, 8, 128, 128), 4),
                                         ((2, 12, 512, 512), 0), ((800, 4, 64, 32), 0), ((3000, 4, 64, 64), 0)])
def test_chain_of_dependent_launches(ctx, oracle, hccs, shape, flags):
    """X -> A -> B -> C, three launches back to back on one stream with no synchronisation, each reading as
    int8 logits the bytes the previous one wrote.  With programmatic dependent launch a kernel's prologue --
    and its L2 prefetch of the input -- runs while the previous kernel still writes that input (the grids
    here are mostly smaller than one wave, so that both kernels are resident together); A, B and C hold
    other bytes beforehand, so a load that did not wait for the previous kernel shows."""
    import torch
    wl = hccs.workloads.make_rows(77, shape, kind="gauss")
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    mode = oracle_mode(oracle, flags)
    want, stages = wl.logits, []
    for _ in range(3):
        want = oracle.forward(want.view(np.int8), wl.theta, mode, threads=16).view(np.int8)
        stages.append(want)
    dev = torch.device("cuda", ctx.device)
    x = torch.from_numpy(wl.logits).to(dev)
    bufs = [torch.empty(shape, dtype=torch.int8, device=dev) for _ in range(3)]
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234)
    for rep in range(12):
        for t in bufs:
            t.view(torch.uint8).copy_(torch.randint(0, 256, shape, dtype=torch.uint8, device=dev, generator=gen))
        torch.cuda.synchronize()
        src = x
        for t in bufs:
            ctx.hccs_forward(src, t.view(torch.uint8), flags)
            src = t
        torch.cuda.synchronize()
        for k, t in enumerate(bufs):
            assert_same(t.cpu().numpy().view(np.uint8), stages[k].view(np.uint8),
                        f"chain stage {k + 1} shape={shape} flags={flags} repeat={rep}")
    assert ctx.hccs_device_status() == 0


def test_many_heads_and_odd_head_count(ctx, oracle, hccs):
    wl = hccs.workloads.make_rows(5, (3, 67, 3, 64), kind="gauss")
    _check(ctx, oracle, wl, 0)
    wl = hccs.workloads.make_rows(6, (2, 200, 2, 32), kind="laplace")
    _check(ctx, oracle, wl, 1)


def test_every_row_sum_is_reached(ctx, oracle, hccs):
    """The reciprocal is the one scalar step per row and is computed without an integer divide,
    so every row sum Z in 1..32767 is driven through it, in the byte kernel and in the fast one."""
    W = hccs.workloads.Workload
    # (a) one key per row, table designed for one key: Z = B for every B in 256..32767
    Bs = np.arange(256, 32768, dtype=np.int32)
    theta = np.stack([Bs, np.zeros_like(Bs), np.ones_like(Bs)], axis=1)
    x = np.zeros((1, Bs.size, 1, 1), dtype=np.int8)
    wl = W("allZ-one-key", x.shape, 0, 1, theta, logits=x)
    for flags in (0, 1):
        _check(ctx, oracle, wl, flags)
    # (b) Z below 256: a single valid key (causal row 0) of a table designed for 256 keys
    H = 127
    theta = np.array([(h + 1, 0, 1) for h in range(H)], dtype=np.int32)
    rng = np.random.default_rng(1)
    x = rng.integers(-128, 128, size=(1, H, 4, 64), dtype=np.int8)
    wl = W("allZ-small", x.shape, 4, 256, theta, logits=x)
    for flags in (4, 5, 6):
        _check(ctx, oracle, wl, flags)
    # (c) 64-key rows in the fast kernel: S = 1, D = 127, floor score F; a row whose closeness
    # values r_j = 127 - (max - x_j) sum to R has Z = 64*F + R, R in 127..8128
    Fs = [4, 129, 254, 379, 384]
    theta = np.array([(F + 127, 1, 127) for F in Fs], dtype=np.int32)
    R = np.arange(127, 8129)
    x = np.full((1, len(Fs), R.size, 64), 0, dtype=np.int8)
    rest = R - 127                                     # spread over the 63 other keys
    base, extra = rest // 63, rest % 63
    r = np.repeat(base[:, None], 63, axis=1)
    r += (np.arange(63)[None, :] < extra[:, None])
    assert r.max() <= 127 and (r.sum(axis=1) + 127 == R).all()
    rows = np.concatenate([np.full((R.size, 1), 127), 127 - (127 - r)], axis=1)   # x_j = m - delta_j
    rows[:, 1:] = 127 - (127 - r)
    x[0, :] = rows.astype(np.int8)[None]
    wl = W("allZ-64", x.shape, 0, 64, theta, logits=x)
    for flags in (0, 1):
        _check(ctx, oracle, wl, flags)
    reached = {64 * F + int(v) for F in Fs for v in R}
    assert set(range(383, 32705)) <= reached


@pytest.mark.parametrize("Lk", [16, 33, 64, 128, 160, 176, 512, 768, 1024, 2048, 4096])
def test_key_length_mask(ctx, oracle, hccs, Lk):
    """hccs_forward_keylen: the padding mask of encoder workloads, alone and with the causal rule."""
    import torch
    Bt, H, Lq = 9, 3, 6
    wl = hccs.workloads.make_rows(300 + Lk, (Bt, H, Lq, Lk), kind="gauss")
    rng = np.random.default_rng(Lk)
    key_len = rng.integers(1, Lk + 1, size=Bt).astype(np.int32)
    key_len[:4] = (0, Lk, Lk + 5, -3)                            # empty, full, beyond the row, negative
    ctx.hccs_params_upload(wl.theta, wl.n_design)
    x = torch.from_numpy(wl.logits).cuda()
    kl = torch.from_numpy(key_len).cuda()
    for flags in (0, 1, 2, 4, 5):
        odt = torch.uint16 if flags & 1 else torch.uint8
        p = torch.full(wl.logits.shape, 0x5A, dtype=odt, device="cuda")
        ctx.hccs_forward_keylen(x, p, kl, flags)
        torch.cuda.synchronize()
        want = oracle.forward(wl.logits, wl.theta, oracle_mode(oracle, flags), threads=4,
                              key_len=np.clip(key_len, 0, Lk))
        assert_same(p.cpu().numpy(), want, f"keylen Lk={Lk} flags={flags}")
    assert ctx.hccs_device_status() == 0


def test_empty_tensors_and_errors(ctx, hccs):
    import torch
    ctx.hccs_params_upload([(300, 3, 85)] * 4, 64)
    dev = torch.device("cuda", 0)
    e = torch.empty((0, 4, 64, 64), dtype=torch.int8, device=dev)
    ctx.hccs_forward(e, e.view(torch.uint8), 0)                       # no rows: OK, no launch
    e = torch.empty((2, 4, 0, 64), dtype=torch.int8, device=dev)
    ctx.hccs_forward(e, e.view(torch.uint8), 0)
    x = torch.zeros((1, 4, 8, 64), dtype=torch.int8, device=dev)
    p = torch.zeros((1, 4, 8, 64), dtype=torch.uint8, device=dev)
    n0 = ctx.hccs_launch_count()
    ctx.hccs_forward(x, p, 0)
    assert ctx.hccs_launch_count() == n0 + 1
    with pytest.raises(hccs.HccsError) as ei:                         # wrong head count
        ctx.hccs_forward(torch.zeros((1, 3, 8, 64), dtype=torch.int8, device=dev),
                         torch.zeros((1, 3, 8, 64), dtype=torch.uint8, device=dev), 0)
    assert ei.value.status == hccs.HCCS_ERR_INVALID_ARG
    with pytest.raises(hccs.HccsError) as ei:                         # longer than designed
        ctx.hccs_forward(torch.zeros((1, 4, 8, 80), dtype=torch.int8, device=dev),
                         torch.zeros((1, 4, 8, 80), dtype=torch.uint8, device=dev), 0)
    assert ei.value.status == hccs.HCCS_ERR_CONSTRAINT
    with pytest.raises(hccs.HccsError) as ei:                         # unknown flag
        ctx.hccs_forward(x, p, 8)
    assert ei.value.status == hccs.HCCS_ERR_INVALID_ARG
    with pytest.raises(hccs.HccsError) as ei:                         # constraint violation
        ctx.hccs_params_upload([(300, 3, 85), (200, 3, 85)], 64)
    assert ei.value.status == hccs.HCCS_ERR_CONSTRAINT and "head 1" in str(ei.value)
    ctx.hccs_forward(x, p, 0)                                         # the old table is still in force
    fresh = hccs.Context(0)
    with pytest.raises(hccs.HccsError) as ei:
        fresh.hccs_forward(x, p, 0)
    assert ei.value.status == hccs.HCCS_ERR_NOT_UPLOADED
    fresh.close()
    assert ctx.hccs_launch_count() == n0 + 2


def test_forward_host_matches_forward(ctx, oracle, hccs):
    import torch
    for c, batch, flags in ((2, 40, 0), (3, 6, 4), (4, 3, 1), (2, 700, 0)):
        wl = hccs.workloads.make_config(c, batch=batch)
        ctx.hccs_params_upload(wl.theta, wl.n_design)
        f = flags | wl.flags
        xin = torch.from_numpy(wl.logits).pin_memory()
        odt = torch.uint16 if f & 1 else torch.uint8
        out = torch.empty(wl.logits.shape, dtype=odt).pin_memory()
        s_in = torch.empty(wl.logits.shape, dtype=torch.int8, device="cuda")
        s_out = torch.empty(wl.logits.shape, dtype=odt, device="cuda")
        ctx.hccs_forward_host(xin, out, s_in, s_out, f)
        torch.cuda.synchronize()
        want = oracle.forward(wl.logits, wl.theta, oracle_mode(oracle, f), threads=8)
        assert_same(out.numpy(), want, f"forward_host config{c}")
