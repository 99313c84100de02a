"""The fused kernel finds lo_t = ceil((t * 2^sh - 2^(sh-1)) / M) -- the smallest accumulator whose
requantised logit reaches t -- as round-to-nearest of the numerator times the double 1 / M, plus one
upward correction.  The same IEEE arithmetic in numpy, against exact integer ceilings, over every
multiplier, every shift of the single-multiply flow and every t the kernel can meet."""
import numpy as np


def test_double_reciprocal_quotient_is_the_ceiling_or_one_less():
    M = np.arange(1, 1 << 13, dtype=np.int64)[:, None]            # multipliers 1 .. 8191
    inv = 1.0 / M.astype(np.float64)
    t = np.arange(-255, 256, dtype=np.int64)[None, :]             # t = m - D with m, D in int8 range
    for sh in range(1, 25):
        num = t * (1 << sh) - (1 << (sh - 1))                      # broadcast below
        num = np.broadcast_to(num, (M.shape[0], t.shape[1]))
        q = np.rint(num.astype(np.float64) * inv).astype(np.int64)
        q = q + (q * M < num)
        want = -((-num) // M)                                      # exact ceiling
        assert np.array_equal(q, want), f"shift {sh}"
