"""Pins for the oracle's integer attention (Q.K^T -> requantise -> HCCS -> P.V)."""
import math
from fractions import Fraction

import numpy as np

from oracle import hccs_bigint as big
from oracle import hccs_oracle as orc


def test_requant_is_round_half_up_then_clamp():
    """x = clamp(floor(acc*M / 2^sh + 1/2), -128, 127), checked with exact fractions."""
    rng = np.random.default_rng(1)
    cases = [(0, 1000, 20), (2 ** 18, 3840, 20), (-2 ** 18, 3840, 20), (1, 2 ** 19, 20),
             (-1, 2 ** 19, 20), (3, 2 ** 19, 20), (-3, 2 ** 19, 20), (5, 1, 0), (-5, 3, 1)]
    cases += [(int(a), int(m), 20) for a, m in zip(rng.integers(-2 ** 18, 2 ** 18, 400),
                                                   rng.integers(768, 3841, 400))]
    for acc, M, sh in cases:
        exact = Fraction(acc * M, 2 ** sh) + Fraction(1, 2)
        want = max(-128, min(127, math.floor(exact)))
        assert orc.requant(acc, M, sh) == want, (acc, M, sh)
    assert orc.requant(-1, 2 ** 19, 20) == 0        # -0.5 rounds up to 0
    assert orc.requant(-3, 2 ** 19, 20) == -1       # -1.5 rounds up to -1
    assert orc.requant(1, 2 ** 19, 20) == 1         # +0.5 rounds up to 1


def test_attention_matches_matrix_route():
    """The naive triple loops against the same composition done with library matrix
    products (int64 matmul), vectorised requantisation and the pure-Python HCCS row."""
    rng = np.random.default_rng(2)
    Bt, H, L, d = 2, 3, 24, 8
    Q = rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8)
    K = rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8)
    V = rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8)
    M = np.array([90000, 170000, 400000], dtype=np.int32)     # spreads logits over int8
    sh = 20
    theta = np.array([(1300, 9, 100), (800, 30, 20), (1365, 127, 10)], dtype=np.int32)
    for t in theta:
        assert orc.check_params(*map(int, t), L) == 0
    for mode in (0, orc.MODE_CLB, orc.MODE_CAUSAL):
        O, lg, pr = orc.attention(Q, K, V, M, sh, theta, mode, want_intermediates=True)
        acc = np.einsum("bhid,bhjd->bhij", Q.astype(np.int64), K.astype(np.int64))
        x = np.clip((acc * M.astype(np.int64).reshape(1, H, 1, 1) + 2 ** (sh - 1)) >> sh, -128, 127)
        assert (lg == x).all()
        assert x.min() < -100 and x.max() > 100                # the clamp is exercised
        P = np.zeros((Bt, H, L, L), dtype=np.int64)
        for b, h, i in np.ndindex(Bt, H, L):
            valid = [1 if j <= i else 0 for j in range(L)] if mode & orc.MODE_CAUSAL else None
            P[b, h, i] = big.hccs_row(x[b, h, i].tolist(), theta[h], clb=bool(mode & orc.MODE_CLB),
                                      valid=valid)
        assert (pr == P).all()
        want = P @ V.astype(np.int64)
        assert (O == want).all()
    # slices and row ranges only select independent work
    O_all = orc.attention(Q, K, V, M, sh, theta, 0)
    O_part = orc.attention(Q, K, V, M, sh, theta, 0, bh_range=(2, 5), q_range=(3, 11))
    assert (O_part.reshape(-1, L, d)[2:5, 3:11] == O_all.reshape(-1, L, d)[2:5, 3:11]).all()
    assert not O_part.reshape(-1, L, d)[:2].any() and not O_part.reshape(-1, L, d)[2:5, :3].any()
    assert (orc.attention(Q, K, V, M, sh, theta, 0, threads=4) == O_all).all()


def test_key_length_mask_equals_attention_over_the_truncated_keys():
    """Padding keys take no part: attention with key_len[b] = n must equal attention over the first
    n keys and values alone (for the queries both have), also under the causal rule; n = 0 gives
    zeros and n >= L changes nothing."""
    rng = np.random.default_rng(31)
    Bt, H, L, d = 4, 2, 24, 8
    Q, K, V = (rng.integers(-128, 128, size=(Bt, H, L, d), dtype=np.int8) for _ in range(3))
    theta = np.array([[200, 3, 40], [120, 1, 90]], dtype=np.int32)
    M = np.array([900, 3000], dtype=np.int32)
    key_len = np.array([7, 0, 24, 31], dtype=np.int32)
    for mode in (0, orc.MODE_CAUSAL, orc.MODE_CLB):
        got = orc.attention(Q, K, V, M, 12, theta, mode, key_len=key_len)
        full = orc.attention(Q, K, V, M, 12, theta, mode)
        for b in range(Bt):
            n = int(min(max(key_len[b], 0), L))
            if n == 0:
                assert (got[b] == 0).all()
                continue
            if n == L:
                assert np.array_equal(got[b], full[b])
                continue
            # the same queries against the first n keys only: a call of its own on sliced tensors
            Qb = np.ascontiguousarray(Q[b:b + 1, :, :n]); Kb = np.ascontiguousarray(K[b:b + 1, :, :n])
            Vb = np.ascontiguousarray(V[b:b + 1, :, :n])
            want = orc.attention(Qb, Kb, Vb, M, 12, theta, mode)
            assert np.array_equal(got[b, :, :n], want[0]), (mode, b)
            if not mode & orc.MODE_CAUSAL:
                # queries beyond n still attend to the n keys: check one against a by-hand row
                i = L - 1
                for h in range(H):
                    acc = Q[b, h, i].astype(np.int64) @ K[b, h, :n].astype(np.int64).T
                    x = np.array([orc.requant(int(a_), int(M[h]), 12) for a_ in acc], dtype=np.int8)
                    p = orc.forward(x.reshape(1, 1, 1, n), theta[h:h + 1], mode).reshape(n).astype(np.int64)
                    assert np.array_equal(got[b, h, i], (p @ V[b, h, :n].astype(np.int64)).astype(np.int32))


def test_output_requantisation_head_index_and_rounding():
    """int8 output of the fused path: element (b, h, i, c) takes head h's multiplier, and each value is
    clamp(floor(O*Mo / 2^sh + 1/2), -128, 127), checked with exact fractions on every element of a small
    tensor that holds the half-way cases, both clamps and all-zero rows."""
    rng = np.random.default_rng(9)
    Bt, H, L, d = 2, 3, 5, 4
    O = rng.integers(-40000, 40001, size=(Bt, H, L, d)).astype(np.int32)
    sh = 15
    Mo = np.array([1, 2 ** 14, 173], dtype=np.int32)       # head 1: acc * 2^14 / 2^15 = acc / 2, half-way for odd acc
    O[0, 1, 0] = (-3, -1, 1, 3)                            # -1.5 -> -1, -0.5 -> 0, 0.5 -> 1, 1.5 -> 2
    O[1, 2, 1] = (24149, 24150, -24339, -24340)            # last value inside and first beyond each clamp (multiplier 173)
    O[1, 0, 4] = 0
    got = orc.requant_output(O, Mo, sh)
    assert got.dtype == np.int8 and got.shape == O.shape
    for b in range(Bt):
        for h in range(H):
            for i in range(L):
                for c in range(d):
                    exact = Fraction(int(O[b, h, i, c]) * int(Mo[h]), 2 ** sh) + Fraction(1, 2)
                    want = max(-128, min(127, math.floor(exact)))
                    assert int(got[b, h, i, c]) == want, (b, h, i, c)
    assert got[0, 1, 0].tolist() == [-1, 0, 1, 2]
    assert got[1, 2, 1].tolist() == [127, 127, -128, -128]
    assert (got[1, 0, 4] == 0).all()
