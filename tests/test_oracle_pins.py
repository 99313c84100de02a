"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of
the oracle's own code (hand-derived worked examples, closed forms, invariants,
error bounds against exact fractions, brute force against a second statement)."""
import itertools
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import hccs_bigint as big
from oracle import hccs_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")
MODES = {"u8_div": 0, "u16_div": orc.MODE_U16, "u8_clb": orc.MODE_CLB,
         "u16_clb": orc.MODE_U16 | orc.MODE_CLB}


def _examples():
    with open(GOLD) as f:
        return {e["name"]: e for e in json.load(f)["examples"]}


# ----------------------------------------------------------------- worked examples
def test_worked_four_keys():
    e = _examples()["four_keys"]
    for name, mode in MODES.items():
        p, Z, rho = orc.row(e["x"], e["theta"], mode)
        assert Z == e["Z"]
        assert rho == e[name]["rho"]
        assert p.tolist() == e[name]["p"]
        assert int(p.sum()) == e[name]["sum"]


def test_worked_constant_row():
    e = _examples()["constant_row_64_keys_B511"]
    x = np.full(e["n"], e["x_fill"], dtype=np.int8)
    for name in ("u8_div", "u16_div"):
        p, Z, rho = orc.row(x, e["theta"], MODES[name])
        assert (Z, rho) == (e["Z"], e[name]["rho"])
        assert set(p.tolist()) == {e[name]["p_fill"]}
        assert int(p.sum()) == e[name]["sum"]


def test_worked_one_hot_and_saturation():
    e = _examples()["one_hot_64_keys"]
    x = np.full(e["n"], e["x_rest"], dtype=np.int8)
    x[0] = e["x_first"]
    for name in ("u8_div", "u16_div"):
        p, Z, rho = orc.row(x, e["theta"], MODES[name])
        assert (Z, rho) == (e["Z"], e[name]["rho"])
        assert p[0] == e[name]["p_first"] and set(p[1:].tolist()) == {e[name]["p_rest"]}
        assert int(p.sum()) == e[name]["sum"]
    p, Z, rho = orc.row(x, e["theta"], MODES["u8_clb"])
    assert rho == e["u8_clb"]["rho"]
    assert (259 * rho) >> 15 == e["u8_clb"]["p_first_unsaturated"]      # would overshoot 255
    assert p[0] == e["u8_clb"]["p_first"] == 255
    assert set(p[1:].tolist()) == {e["u8_clb"]["p_rest"]}


def test_worked_single_valid_key():
    e = _examples()["single_valid_key"]
    for name in ("u8_div", "u16_div"):
        p, Z, rho = orc.row(e["x"], e["theta"], MODES[name])
        assert (Z, rho, p.tolist()) == (e["Z"], e[name]["rho"], e[name]["p"])
    # the same single key reached through a mask: the masked tail must not matter
    x = np.array([-7, 127, 127, 127], dtype=np.int8)
    p, Z, _ = orc.row(x, e["theta"], 0, valid=[1, 0, 0, 0])
    assert Z == 200 and p.tolist() == [254, 0, 0, 0]


# ----------------------------------------------------------------- reciprocal
def test_reciprocal_exhaustive():
    """rho for every admissible Z: defined by T' - Z < rho*Z <= T' (floor), and for the
    leading-bit form by T' - 2^k < rho*2^k <= T' with 2^k <= Z < 2^(k+1)."""
    for mode, Tp in ((0, 255 * 2 ** 15), (orc.MODE_U16, 32767)):
        for Z in range(1, 32768):
            r = orc.rho(Z, mode)
            assert r * Z <= Tp < (r + 1) * Z
            rc = orc.rho(Z, mode | orc.MODE_CLB)
            k = 0
            while 2 ** (k + 1) <= Z:
                k += 1
            assert rc * 2 ** k <= Tp < (rc + 1) * 2 ** k
            assert r <= rc < 2 * r + 2                    # overestimates by less than 2x
    assert orc.rho(256, 0) == 32640 <= 32767            # Z >= 256 keeps rho_u8 in int16
    assert orc.rho(255, 0) == 32768                       # ... and Z = 255 is the first that does not
    assert orc.rho(32767, orc.MODE_U16) == 1              # n*B <= 32767 keeps rho >= 1
    assert orc.rho(32768, orc.MODE_U16) == 0


# ----------------------------------------------------------------- closed forms
def _theta_cases(n):
    f, bmax = -(-256 // n), 32767 // n
    cases = [(bmax, 0, 1), (f, 0, 127)]
    for D in (1, 4, 17, 127):
        room = bmax - f
        if room < D:
            continue
        S = min(127, room // D)
        cases += [(S * D + f, S, D), (bmax, S, D), (bmax, 1, D)]
    return [c for c in cases if orc.check_params(*c, n) == 0]


@pytest.mark.parametrize("n", [1, 2, 7, 32, 64, 128, 512, 1024])
def test_closed_forms(n):
    rng = np.random.default_rng(100 + n)
    for (B, S, D) in _theta_cases(n):
        for mode in MODES.values():
            Tp = 32767 if mode & orc.MODE_U16 else 255 * 2 ** 15
            # constant row: every score is B, Z = n*B
            p, Z, rho = orc.row(np.full(n, int(rng.integers(-128, 128)), np.int8), (B, S, D), mode)
            assert Z == n * B
            want = B * rho if mode & orc.MODE_U16 else min((B * rho) >> 15, 255)
            assert set(p.tolist()) == {want}
            if not mode & orc.MODE_CLB:
                assert rho == Tp // (n * B)
            # the arg-max element always has score B; anything D or more below the max
            # has the floor score B - S*D
            x = rng.integers(-128, 128, size=n).astype(np.int8)
            p, Z, rho = orc.row(x, (B, S, D), mode)
            top = B * rho if mode & orc.MODE_U16 else min((B * rho) >> 15, 255)
            low = (B - S * D) * rho if mode & orc.MODE_U16 else min(((B - S * D) * rho) >> 15, 255)
            assert p[int(np.argmax(x))] == top
            far = np.flatnonzero(int(x.max()) - x.astype(np.int64) >= D)
            assert all(p[j] == low for j in far)
        # S = 0: the output does not depend on the logits at all
        if S == 0:
            a, _, _ = orc.row(rng.integers(-128, 128, size=n).astype(np.int8), (B, S, D), 0)
            b, _, _ = orc.row(np.zeros(n, np.int8), (B, S, D), 0)
            assert a.tolist() == b.tolist()


# ----------------------------------------------------------------- invariants
@pytest.mark.parametrize("n", [3, 16, 64, 128, 512])
def test_invariants_random_rows(n):
    rng = np.random.default_rng(7 * n)
    thetas = _theta_cases(n)
    for trial in range(60):
        B, S, D = thetas[trial % len(thetas)]
        sigma = rng.uniform(2, 60)
        x = np.clip(np.rint(rng.normal(0, sigma, n)), -128, 127).astype(np.int8)
        if trial % 5 == 0:
            x[rng.integers(n)] = 127
        xs = x.astype(np.int64)
        for name, mode in MODES.items():
            T = 32767 if mode & orc.MODE_U16 else 255
            p, Z, rho = orc.row(x, (B, S, D), mode)
            assert (p >= 0).all()                                     # non-negative
            order = np.argsort(xs, kind="stable")
            assert (np.diff(p[order]) >= 0).all()                     # order preserving
            assert all(p[a] == p[b] for a in range(n) for b in range(a) if xs[a] == xs[b]) \
                if n <= 16 else True
            assert 256 <= Z <= 32767                                  # in-band, unmasked row
            # permutation equivariance
            perm = rng.permutation(n)
            pp, _, _ = orc.row(x[perm], (B, S, D), mode)
            assert pp.tolist() == p[perm].tolist()
            # shift invariance (no int8 saturation)
            c = int(rng.integers(-128 - xs.min(), 128 - xs.max()))
            ps, _, _ = orc.row((xs + c).astype(np.int8), (B, S, D), mode)
            assert ps.tolist() == p.tolist()
            # changing an element already D or more below the max (keeping it there) is a no-op
            far = np.flatnonzero(xs.max() - xs >= D)
            if far.size:
                y = x.copy()
                y[far[0]] = -128
                py, _, _ = orc.row(y, (B, S, D), mode)
                assert py.tolist() == p.tolist()
            if name == "u16_div":
                assert 1 <= rho
                assert p.max() <= T
                assert int(p.sum()) == Z * rho and T - Z < int(p.sum()) <= T
                assert B * (32767 // (n * B)) * n <= 32767            # the paper's product bound
            if name == "u8_div":
                assert rho <= 32767
                assert p.max() <= T
                assert T - n - 1 < int(p.sum()) <= T
            if name in ("u8_clb", "u16_clb"):
                _, _, rdiv = orc.row(x, (B, S, D), mode & ~orc.MODE_CLB)
                assert rdiv <= rho < 2 * rdiv + 2
                assert p.max() <= (255 if name == "u8_clb" else 65534)


def test_error_bound_against_exact_fractions():
    """The integer outputs approximate T * s_i / Z (Eq. 5) from below, within the
    truncation the paper describes: u16 loses less than s_i, u8 less than 1 + s_i/2^15."""
    rng = np.random.default_rng(5)
    for n in (4, 64, 128):
        for (B, S, D) in _theta_cases(n):
            x = rng.integers(-60, 60, size=n).astype(np.int8)
            exact = big.exact_probabilities(x.tolist(), (B, S, D))
            # exact p_i come from an independent route: check they are a distribution
            assert sum(exact) == 1
            p16, Z, _ = orc.row(x, (B, S, D), orc.MODE_U16)
            p8, _, _ = orc.row(x, (B, S, D), 0)
            for j in range(n):
                s_j = exact[j] * Z
                assert 32767 * exact[j] - s_j < int(p16[j]) <= 32767 * exact[j]
                assert 255 * exact[j] - s_j * Fraction(1, 2 ** 15) - 1 < int(p8[j]) <= 255 * exact[j]


def test_out_shift_halves():
    x = [10, 7, 3, -20]
    p0, _, _ = orc.row(x, (200, 10, 12), 0, out_shift=0)
    p1, _, _ = orc.row(x, (200, 10, 12), 0, out_shift=1)
    p2, _, _ = orc.row(x, (200, 10, 12), 0, out_shift=2)
    assert p0.tolist() == [87, 74, 57, 35]
    assert p1.tolist() == [43, 37, 28, 17]      # (s*14406) >> 16, by hand
    assert p2.tolist() == [21, 18, 14, 8]


# ----------------------------------------------------------------- brute force
ALPHABET = [-128, -127, -64, -1, 0, 1, 63, 126, 127]
TINY_THETAS = [(8191, 0, 1), (64, 0, 127), (200, 10, 12), (8191, 63, 127), (190, 1, 126),
               (8000, 127, 62), (65, 1, 1)]


def _cmp_row(x, theta, valid=None):
    for u16 in (False, True):
        for clb in (False, True):
            mode = (orc.MODE_U16 if u16 else 0) | (orc.MODE_CLB if clb else 0)
            got, _, _ = orc.row(x, theta, mode, valid=valid)
            want = big.hccs_row(x, theta, u16=u16, clb=clb, valid=valid)
            assert got.tolist() == want, (x, theta, u16, clb, valid)


def test_brute_force_all_rows_of_two():
    """All 65 536 int8 rows of length 2, C oracle vs the pure-Python statement."""
    theta = (200, 10, 12)
    L = orc.lib()
    vals = np.arange(-128, 128, dtype=np.int64)
    for mode, (u16, clb) in ((0, (False, False)), (orc.MODE_U16 | orc.MODE_CLB, (True, True))):
        x = np.stack(np.meshgrid(vals, vals, indexing="ij"), -1).reshape(1, 1, -1, 2).astype(np.int8)
        got = orc.forward(x, [theta], mode).reshape(-1, 2)
        for r in range(0, 65536):
            row = x.reshape(-1, 2)[r].tolist()
            assert got[r].tolist() == big.hccs_row(row, theta, u16=u16, clb=clb)
    assert L is not None


@pytest.mark.parametrize("n", [1, 2, 3, 4])
def test_brute_force_alphabet(n):
    thetas = [t for t in TINY_THETAS if orc.check_params(*t, 4) == 0]
    assert len(thetas) >= 5
    for x in itertools.product(ALPHABET, repeat=n):
        for theta in thetas[: (len(thetas) if n < 4 else 3)]:
            _cmp_row(list(x), theta)
    # with every prefix mask (the causal pattern)
    for x in itertools.product(ALPHABET[::2], repeat=n):
        for nv in range(0, n + 1):
            _cmp_row(list(x), thetas[2], valid=[1] * nv + [0] * (n - nv))


def test_masked_rows_wide_reciprocal():
    """Few valid keys make Z < 256 and rho_u8 > 32767; the arithmetic stays exact in wide ints."""
    theta = (255, 2, 100)             # in band for n = 128
    assert orc.check_params(*theta, 128) == 0
    rng = np.random.default_rng(11)
    x = rng.integers(-128, 128, size=128).astype(np.int8)
    for nv in (0, 1, 2, 3, 5, 128):
        valid = [1] * nv + [0] * (128 - nv)
        for mode in MODES.values():
            got, Z, rho = orc.row(x, theta, mode, valid=valid)
            want = big.hccs_row(x.tolist(), theta, u16=bool(mode & 1), clb=bool(mode & 2), valid=valid)
            assert got.tolist() == want
            assert (got[nv:] == 0).all()
            if nv == 1 and mode == 0:
                assert Z == 255 and rho == 32768 and got[0] == 255


# ----------------------------------------------------------------- tensor layout
def test_forward_head_indexing_and_causal_alignment():
    """Flat row r belongs to head (r // Lq) % H; causal keeps j <= i + (Lk - Lq)."""
    rng = np.random.default_rng(3)
    Bt, H, Lq, Lk = 3, 5, 4, 6
    theta = np.array([(5000 - 700 * h, h + 1, 10 + 3 * h) for h in range(H)], dtype=np.int32)
    for t in theta:
        assert orc.check_params(*map(int, t), Lk) == 0
    x = rng.integers(-128, 128, size=(Bt, H, Lq, Lk)).astype(np.int8)
    for mode in (0, orc.MODE_U16, orc.MODE_CAUSAL, orc.MODE_CAUSAL | orc.MODE_U16 | orc.MODE_CLB):
        out = orc.forward(x, theta, mode)
        for b, h, i in np.ndindex(Bt, H, Lq):
            valid = None
            if mode & orc.MODE_CAUSAL:
                valid = [1 if j <= i + (Lk - Lq) else 0 for j in range(Lk)]
            want = big.hccs_row(x[b, h, i].tolist(), theta[h], u16=bool(mode & 1),
                                clb=bool(mode & 2), valid=valid)
            assert out[b, h, i].tolist() == want
    # Lq > Lk: the first Lq - Lk queries see no key at all
    x2 = rng.integers(-128, 128, size=(1, H, 6, 4)).astype(np.int8)
    out = orc.forward(x2, theta, orc.MODE_CAUSAL)
    assert (out[:, :, :2, :] == 0).all() and (out[:, :, 2, 0] > 0).all()
    assert (out[:, :, 2, 1:] == 0).all()
    # threads and row ranges only partition independent rows
    a = orc.forward(x, theta, 0, threads=3)
    assert (a == orc.forward(x, theta, 0)).all()
    part = orc.forward(x, theta, 0, row_range=(7, 19)).reshape(-1, Lk)
    assert (part[7:19] == a.reshape(-1, Lk)[7:19]).all() and not part[:7].any() and not part[19:].any()


def test_forward_key_length_mask():
    """Padding mask: key j of batch entry b is valid iff j < key_len[b]; combined with causal."""
    rng = np.random.default_rng(8)
    Bt, H, Lq, Lk = 4, 3, 5, 7
    theta = np.array([(4000 - 500 * h, h + 1, 9 + 2 * h) for h in range(H)], dtype=np.int32)
    x = rng.integers(-128, 128, size=(Bt, H, Lq, Lk)).astype(np.int8)
    key_len = np.array([7, 3, 0, 1], dtype=np.int32)
    for mode in (0, orc.MODE_U16 | orc.MODE_CLB, orc.MODE_CAUSAL):
        out = orc.forward(x, theta, mode, key_len=key_len)
        for b, h, i in np.ndindex(Bt, H, Lq):
            valid = [1 if j < key_len[b] and (not mode & orc.MODE_CAUSAL or j <= i + (Lk - Lq)) else 0
                     for j in range(Lk)]
            want = big.hccs_row(x[b, h, i].tolist(), theta[h], u16=bool(mode & 1), clb=bool(mode & 2), valid=valid)
            assert out[b, h, i].tolist() == want
    assert not out[2].any()                                     # a batch entry of length 0 gives zeros
    full = orc.forward(x, theta, 0, key_len=np.full(Bt, Lk, np.int32))
    assert (full == orc.forward(x, theta, 0)).all()             # full lengths = no mask


# ----------------------------------------------------------------- constraints
def test_constraints_one_at_a_time():
    n = 64
    assert orc.check_params(300, 3, 85, n) == 0
    assert orc.check_params(511, 0, 1, n) == 0
    assert orc.check_params(300, 3, 128, n) & 1            # D <= 127
    assert orc.check_params(300, 3, 0, n) & 1
    assert orc.check_params(200, 3, 85, n) & 2             # B - S*D >= 0
    assert orc.check_params(40000, 0, 1, 1) & 4            # B <= 32767
    assert orc.check_params(258, 3, 85, n) == 8            # floor: B - S*D >= ceil(256/64) = 4
    assert orc.check_params(259, 3, 85, n) == 0
    assert orc.check_params(512, 3, 85, n) == 16           # n*B <= 32767: 64*512 = 32768
    assert orc.check_params(511, 3, 85, n) == 0
    assert orc.check_params(300, -1, 85, n) & 32           # S >= 0
    assert orc.check_params(0, 0, 1, n) & 32
    assert orc.check_params(8000, 128, 4, 4) & 64          # S <= 127 (int8 MAC operand)
    # the band of Eq. 11 is exactly the set the checker admits
    for n in (1, 2, 64, 100, 128, 512, 1024, 4096, 32767):
        f, bmax = -(-256 // n), 32767 // n
        for S, D in ((0, 1), (1, 4), (2, 13)):
            for B in range(max(1, S * D + f - 2), S * D + f + 3):
                ok = orc.check_params(B, S, D, n) == 0
                assert ok == (S * D + f <= B <= bmax), (n, B, S, D)
            for B in range(max(1, bmax - 2), bmax + 3):
                ok = orc.check_params(B, S, D, n) == 0
                assert ok == (S * D + f <= B <= bmax), (n, B, S, D)
    assert orc.check_params(1, 0, 1, 32768) != 0           # no admissible B beyond n = 32767


def test_workload_theta_is_in_band():
    from paper_2604_02292_b200 import workloads as wl
    rng = np.random.default_rng(0)
    for n in (1, 3, 16, 64, 128, 512, 1024, 2048, 4096, 8192, 16384, 32767):
        th = wl.sample_theta(rng, 16, n)
        for B, S, D in th.tolist():
            assert orc.check_params(B, S, D, n) == 0, (n, B, S, D)
