/*
 * hccs_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, scalar CPU statement of the Head-Calibrated Clipped-Linear
 * Softmax (HCCS) inference step, written from the paper's Section III
 * (Eq. 1-4, the reciprocal rho, the int8 output path, the leading-bit (CLB)
 * reciprocal) and Algorithm 1.  Every intermediate is int64; there is no
 * blocking, vectorisation or reordering beyond what Algorithm 1 states.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * build or call this file.  It shares no code, header, table or constant
 * with the CUDA library.
 *
 * Readings of the paper where it is silent (each a named constant or a
 * comment here, so another reading is a one-line change):
 *   - OUT_SHIFT is an argument (the paper uses it in the int8 output path
 *     without defining it); the default everywhere is 0.
 *   - right shifts truncate toward minus infinity ("right-shifted").
 *   - CLB reciprocal = floor(T' / 2^k), k = floor(log2 Z).
 *   - u8 output with the CLB reciprocal saturates at 255; u16 does not
 *     saturate (the product stays below 2*32767 and fits uint16).
 *   - masking is not in the paper: masked positions take no part in the
 *     max or the sum and are written as 0; an all-masked row is all zeros.
 *   - rho is kept in a wide integer (never clamped to int16).
 */
#include <stdint.h>
#include <stddef.h>

#define ORACLE_T_U16      32767      /* T for int16 output (Eq. rho)            */
#define ORACLE_T_U8       255        /* T for int8 output                      */
#define ORACLE_INV_SHIFT  15         /* R = INV_SHIFT of the int8 output path  */
#define ORACLE_U8_CLB_SATURATES 1    /* reading: u8+CLB clamps to 255          */

/* mode bits (the oracle's own; the tests map the library's flags onto these) */
#define ORACLE_MODE_U16    1
#define ORACLE_MODE_CLB    2
#define ORACLE_MODE_CAUSAL 4

/* Integer range constraints (Section "Integer Range Constraints") for a design
 * row length n.  Returns a bit mask of the violated items, 0 when admissible:
 *   bit0  D_max <= 127 (and D_max >= 1)
 *   bit1  B - S*D_max >= 0                       (non-negative scores)
 *   bit2  B <= 32767                             (int16 storage)
 *   bit3  n*(B - S*D_max) >= 256, enforced as B - S*D_max >= ceil(256/n)
 *   bit4  n*B <= 32767
 *   bit5  S >= 0   (Eq. 3: S_h >= 0)   and B > 0
 *   bit6  S <= 127 (reading: S is an operand of "a single int8 MAC")
 */
int hccs_oracle_check_params(int64_t B, int64_t S, int64_t D, int64_t n)
{
    int bad = 0;
    if (D > 127 || D < 1) bad |= 1;
    if (B - S * D < 0) bad |= 2;
    if (B > 32767) bad |= 4;
    {
        int64_t floor_score = (256 + n - 1) / n;          /* ceil(256/n) */
        if (B - S * D < floor_score) bad |= 8;
    }
    if (n * B > 32767) bad |= 16;
    if (S < 0 || B <= 0) bad |= 32;
    if (S > 127) bad |= 64;
    return bad;
}

static int64_t floor_log2_i64(int64_t z)
{
    int64_t k = 0;
    while ((z >> (k + 1)) != 0) ++k;     /* z >= 1 */
    return k;
}

/* The reciprocal of Algorithm 1 ("rho <- floor(T/Z)") in its four forms. */
int64_t hccs_oracle_rho(int64_t Z, int mode)
{
    int64_t Tprime;
    if (Z <= 0) return 0;
    if (mode & ORACLE_MODE_U16) Tprime = ORACLE_T_U16;                       /* Eq. rho    */
    else Tprime = (int64_t)ORACLE_T_U8 * ((int64_t)1 << ORACLE_INV_SHIFT);   /* Eq. rho_u8 */
    if (mode & ORACLE_MODE_CLB) {
        int64_t k = floor_log2_i64(Z);                                       /* CLB        */
        return Tprime >> k;
    }
    return Tprime / Z;                   /* both positive: truncation == floor */
}

/*
 * One row, Algorithm 1.  x[0..n) are the row's int8 logits; valid[j] != 0
 * marks the positions that take part (NULL = all).  p_out[0..n) receives the
 * scaled integer probabilities as int64 (the caller narrows them).  Z_out and
 * rho_out may be NULL.  Returns the number of valid positions.
 */
int64_t hccs_oracle_row(const int8_t *x, const uint8_t *valid, int64_t n,
                        int64_t B, int64_t S, int64_t D, int mode, int64_t out_shift,
                        int64_t *p_out, int64_t *Z_out, int64_t *rho_out)
{
    int64_t i, n_valid = 0, m = 0, Z = 0, rho;
    /* m <- max_i x_i over the valid set */
    for (i = 0; i < n; ++i) {
        if (valid && !valid[i]) continue;
        if (n_valid == 0 || (int64_t)x[i] > m) m = (int64_t)x[i];
        ++n_valid;
    }
    if (n_valid == 0) {
        for (i = 0; i < n; ++i) p_out[i] = 0;
        if (Z_out) *Z_out = 0;
        if (rho_out) *rho_out = 0;
        return 0;
    }
    /* delta_i <- min(m - x_i, D_max);  s_i <- B - S*delta_i;  Z <- sum s_i.
     * The scores are parked in p_out between the two loops. */
    for (i = 0; i < n; ++i) {
        int64_t delta, s;
        if (valid && !valid[i]) { p_out[i] = 0; continue; }
        delta = m - (int64_t)x[i];
        if (delta > D) delta = D;
        s = B - S * delta;
        p_out[i] = s;
        Z += s;
    }
    rho = hccs_oracle_rho(Z, mode);
    /* p_i <- s_i * rho (then the int8 path's right shift by R + OUT_SHIFT) */
    for (i = 0; i < n; ++i) {
        int64_t prod;
        if (valid && !valid[i]) continue;
        prod = p_out[i] * rho;
        if (mode & ORACLE_MODE_U16) {
            p_out[i] = prod;
        } else {
            int64_t q = prod >> (ORACLE_INV_SHIFT + out_shift);
            if (ORACLE_U8_CLB_SATURATES && (mode & ORACLE_MODE_CLB) && q > ORACLE_T_U8)
                q = ORACLE_T_U8;
            p_out[i] = q;
        }
    }
    if (Z_out) *Z_out = Z;
    if (rho_out) *rho_out = rho;
    return n_valid;
}

/*
 * Rows [row_begin, row_end) of a contiguous [Bt,H,Lq,Lk] int8 tensor.  The
 * head of flat row r is (r / Lq) mod H; params is H triples (B,S,D) as int32.
 * Causal: position j of query i is valid when j <= i + (Lk - Lq).  key_len (optional): key j of
 * batch entry b is valid when j < key_len[b] (padding mask; both rules combine).
 * probs is uint8 (u8 modes) or uint16 (u16 modes), same shape.
 * Returns 0, or -1 when a value would not fit the output type.
 */
int hccs_oracle_forward(const int8_t *logits, void *probs,
                        int64_t Bt, int64_t H, int64_t Lq, int64_t Lk,
                        const int32_t *params, int mode, int64_t out_shift,
                        int64_t row_begin, int64_t row_end,
                        int64_t *p_tmp /* Lk */, uint8_t *valid_tmp /* Lk */,
                        const int32_t *key_len /* Bt entries or NULL: padding mask */)
{
    int64_t r, j;
    (void)Bt;
    for (r = row_begin; r < row_end; ++r) {
        int64_t h = (r / Lq) % H;
        int64_t i = r % Lq;
        const int8_t *x = logits + r * Lk;
        const uint8_t *valid = NULL;
        if ((mode & ORACLE_MODE_CAUSAL) || key_len) {
            int64_t b = r / (Lq * H);
            for (j = 0; j < Lk; ++j) {
                int ok = 1;
                if ((mode & ORACLE_MODE_CAUSAL) && !(j <= i + (Lk - Lq))) ok = 0;
                if (key_len && !(j < (int64_t)key_len[b])) ok = 0;      /* key j is padding */
                valid_tmp[j] = (uint8_t)ok;
            }
            valid = valid_tmp;
        }
        hccs_oracle_row(x, valid, Lk, params[3 * h + 0], params[3 * h + 1], params[3 * h + 2],
                        mode, out_shift, p_tmp, NULL, NULL);
        if (mode & ORACLE_MODE_U16) {
            uint16_t *o = (uint16_t *)probs + r * Lk;
            for (j = 0; j < Lk; ++j) {
                if (p_tmp[j] < 0 || p_tmp[j] > 65535) return -1;
                o[j] = (uint16_t)p_tmp[j];
            }
        } else {
            uint8_t *o = (uint8_t *)probs + r * Lk;
            for (j = 0; j < Lk; ++j) {
                if (p_tmp[j] < 0 || p_tmp[j] > 255) return -1;
                o[j] = (uint8_t)p_tmp[j];
            }
        }
    }
    return 0;
}

/* Requantisation of an int32 Q.K^T accumulator to an int8 logit (not in the
 * paper; the reading is round-half-up fixed point, arithmetic shift, clamp):
 *   x = clamp((acc*M + 2^(sh-1)) >> sh, -128, 127). */
int64_t hccs_oracle_requant(int64_t acc, int64_t M, int64_t sh)
{
    int64_t t = acc * M;
    int64_t x;
    if (sh > 0) t += (int64_t)1 << (sh - 1);
    x = t >> sh;                          /* arithmetic shift: floor */
    if (x < -128) x = -128;
    if (x > 127) x = 127;
    return x;
}

/*
 * int8 output of the fused path: every int32 element of O [B*H, L, d] requantised with its head's
 * multiplier by the same rounding rule as the logits (hccs_oracle_requant): not in the paper,
 * which stops at the integer probabilities; the reading is the library's requantisation rule
 * applied once more.  Mo holds one multiplier per head.
 */
void hccs_oracle_requant_output(const int32_t *O, int8_t *out, const int32_t *Mo, int64_t sh,
                                int64_t BH, int64_t H, int64_t L, int64_t d)
{
    int64_t bh, k;
    for (bh = 0; bh < BH; ++bh)
        for (k = 0; k < L * d; ++k)
            out[bh * L * d + k] = (int8_t)hccs_oracle_requant(O[bh * L * d + k], Mo[bh % H], sh);
}

/*
 * Integer attention for (batch*head) slices [bh_begin, bh_end) and query rows
 * [q_begin, q_end) of each: Q,K,V int8 [Bt,H,L,d]; logits x_ij =
 * requant(sum_d Q[i,d]*K[j,d], M[h], sh); P = HCCS(x_i.) in u8 mode with the
 * exact divide (or CLB / causal per `mode`); O[i,:] = sum_j P[i,j]*V[j,:],
 * int32 [Bt,H,L,d].  x_tmp, p_tmp: L entries each; valid_tmp: L bytes.
 * logits_out / probs_out (may be NULL) receive the intermediate int8 logits and
 * uint8 probabilities of the computed rows, laid out [Bt,H,L,L].
 * key_len (may be NULL): int32 [Bt]; keys at and beyond key_len[b] are padding of
 * batch entry b: like causally masked keys they take no part in max and sum and get
 * probability 0 (masking is not in the paper; the valid keys are always a prefix).
 */
int hccs_oracle_attention(const int8_t *Q, const int8_t *K, const int8_t *V, int32_t *O,
                          const int32_t *M, int64_t sh, const int32_t *params,
                          int64_t Bt, int64_t H, int64_t L, int64_t d,
                          int mode, int64_t out_shift,
                          int64_t bh_begin, int64_t bh_end, int64_t q_begin, int64_t q_end,
                          int8_t *x_tmp, int64_t *p_tmp, uint8_t *valid_tmp,
                          int8_t *logits_out, uint8_t *probs_out, const int32_t *key_len)
{
    int64_t bh, i, j, c;
    (void)Bt;
    if (mode & ORACLE_MODE_U16) return -2;
    for (bh = bh_begin; bh < bh_end; ++bh) {
        int64_t h = bh % H;
        const int8_t *q = Q + bh * L * d;
        const int8_t *k = K + bh * L * d;
        const int8_t *v = V + bh * L * d;
        int32_t *o = O + bh * L * d;
        for (i = q_begin; i < q_end; ++i) {
            const uint8_t *valid = NULL;
            for (j = 0; j < L; ++j) {
                int64_t acc = 0;
                for (c = 0; c < d; ++c) acc += (int64_t)q[i * d + c] * (int64_t)k[j * d + c];
                x_tmp[j] = (int8_t)hccs_oracle_requant(acc, M[h], sh);
            }
            if ((mode & ORACLE_MODE_CAUSAL) || key_len) {
                /* valid keys form a prefix: the causal rule and / or the batch entry's key length */
                int64_t limit = L;
                if (key_len) {
                    limit = key_len[bh / H];
                    if (limit < 0) limit = 0;
                    if (limit > L) limit = L;
                }
                for (j = 0; j < L; ++j)
                    valid_tmp[j] = (uint8_t)(j < limit && (!(mode & ORACLE_MODE_CAUSAL) || j <= i));
                valid = valid_tmp;
            }
            hccs_oracle_row(x_tmp, valid, L, params[3 * h + 0], params[3 * h + 1],
                            params[3 * h + 2], mode, out_shift, p_tmp, NULL, NULL);
            for (c = 0; c < d; ++c) {
                int64_t acc = 0;
                for (j = 0; j < L; ++j) acc += p_tmp[j] * (int64_t)v[j * d + c];
                if (acc > 2147483647LL || acc < -2147483648LL) return -1;
                o[i * d + c] = (int32_t)acc;
            }
            if (logits_out)
                for (j = 0; j < L; ++j) logits_out[(bh * L + i) * L + j] = x_tmp[j];
            if (probs_out)
                for (j = 0; j < L; ++j) probs_out[(bh * L + i) * L + j] = (uint8_t)p_tmp[j];
        }
    }
    return 0;
}
