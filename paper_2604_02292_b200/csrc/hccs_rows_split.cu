// Register-resident row kernel for Lk = 32*G*V (G lanes per row, V 32-byte chunks per lane):
// the powers of two from 32 to 8192 and the multiples of 32 below 4096 whose odd part is 3, 5 or 7
// (and, with 16-byte chunks or padded lane groups, every other multiple of 16 up to 4096 and tensors that
// are only 16-byte aligned: see launch_shape).  Algorithm 1 of the paper, stage by stage, on 16-bit pairs.
//
// Why 16-bit pairs: on sm_100a the byte-wise SIMD min/max intrinsics are emulated (about ten
// instructions each), while min/max on s16x2 and the three-operand forms max(a+b, c) are single
// instructions.  Each 32-bit word of four int8 logits is therefore split once into two words of
// two sign-extended 16-bit lanes (bytes 0,2 and bytes 1,3; one PRMT each), and every later stage
// works on those:
//   stage 1  m = max x                      one three-input max.s16x2 per word
//   stage 2+3  instead of delta = min(m - x, D) the kernel keeps the "closeness"
//            r = D - delta = max(x + (D - m), 0)   one viaddmax.s16x2 per split word
//            so that the score is s = B - S*delta = F + S*r with F = B - S*D (Eq. 2, Eq. 3);
//            every quantity stays non-negative
//   stage 4  Z = n_valid*F + S*sum(r)       two dot products with ones per word (dp2a, multiply pipe)
//   stage 5  rho once per row; p = (F*rho' + S*rho'*r) >> 16 with rho' = rho << (1 - OUT_SHIFT)
// For uint8 output X = s*rho' < 2^24 (s <= Z), and the two elements of a 16-bit pair are normalised by
// two 32-bit multiply-adds on the pair: the coefficients are split at 8 bits so that every partial
// result fits its 16-bit lane (see the kernel).  A 32x32->64-bit multiply-add with the two elements
// 24 bits apart does the same in one instruction, but its 64-bit addend costs two more on the integer
// pipe, which is the pipe this kernel is bound by.
// For uint16 output one 32-bit multiply-add handles a pair directly (s*rho < 2^16).
//
// Causal rows: masked bytes are replaced by -128 right after the load (they can then never raise
// the max), their closeness r_m = max(D - m - 128, 0) is subtracted from the sum in closed form,
// and the output words are masked; the byte masks are computed from the count of valid bytes.
#include <cuda_runtime.h>
#include <stdint.h>

#include "hccs_device.cuh"
#include "hccs_internal.h"

namespace hccs {

namespace {

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Streaming accesses: nothing is read or written twice, so neither loads nor stores allocate in L1.
// EVICT_FIRST also marks the loaded lines as the first to leave L2 (which shapes use it: see the kernel).
template <bool EVICT_FIRST>
__device__ __forceinline__ void ldg256(const void *p, uint32_t (&r)[8]) {
    if (EVICT_FIRST) {
        uint64_t pol;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
        asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8], %9;"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                       "=r"(r[7])
                     : "l"(p), "l"(pol));
    } else {
        asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                       "=r"(r[7])
                     : "l"(p));
    }
}

__device__ __forceinline__ void stg256(void *p, const uint32_t (&r)[8]) {
    asm volatile("st.global.L1::no_allocate.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

// The same for 16-byte chunks; these do allocate in L1: two neighbouring chunks of a lane share a
// 32-byte sector (measured: 2 to 8 % faster).
template <bool EVICT_FIRST>
__device__ __forceinline__ void ldg128(const void *p, uint32_t (&r)[4]) {
    if (EVICT_FIRST) {
        uint64_t pol;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
        asm volatile("ld.global.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                     : "l"(p), "l"(pol));
    } else {
        asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                     : "l"(p));
    }
}
__device__ __forceinline__ void stg128(void *p, const uint32_t (&r)[4]) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]),
                 "r"(r[3])
                 : "memory");
}

constexpr uint32_t kSelEven = 0xA280u;   // bytes 0 and 2, each sign-extended to 16 bits
constexpr uint32_t kSelOdd = 0xB391u;    // bytes 1 and 3, each sign-extended to 16 bits
constexpr uint32_t kMinus128x4 = 0x80808080u;

// Byte mask of word k of a chunk whose first cnt bytes are valid: 0xff for each valid byte.  Two
// instructions (add-and-clamp at zero, funnel shift that saturates at 32): a shared-memory table of
// these masks costs every CTA a fill and a barrier before its first load can be used.
__device__ __forceinline__ uint32_t byte_mask(int cnt, int k) {
    return __funnelshift_lc(0xffffffffu, 0u, (uint32_t)__viaddmax_s32(8 * cnt, -32 * k, 0));
}

// CW: 32-bit words per chunk, 8 (32-byte chunks) or 4 (16-byte chunks, for the row lengths that are a
// multiple of 16 but not of 32, or whose number of 32-byte chunks has an odd part above 7).
// PAD: the G*V chunks of a lane group cover more than the row (any multiple of 16 keys: the chunks beyond
// the row's end are never loaded, count as masked and are not stored); needs the masked instantiation.
//
// Masked instantiations decide per chunk index v, once per warp, whether every lane holds a full chunk
// (then the chunk runs through the unmasked code: no byte masks, no substitution, no output mask), whether
// no row of the warp reaches it (then it is skipped and stored as zeros), or neither (masked code).  With
// a causal mask the diagonal crosses exactly one chunk index of a warp, so one chunk per warp pays for masks.
template <int G, int V, bool U16, bool CLB, bool CAUSAL, int CW = 8, bool PAD = false>
__global__ void __launch_bounds__(256) rows_split_kernel(const int8_t *x_all, void *p_all, RowArgs a) {
    static_assert(!PAD || CAUSAL, "padded lane groups run through the masked path");
    constexpr int RW = 32 / G;      // rows per warp
    constexpr int NW = CW * V;      // 32-bit words of logits per lane
    constexpr int CB = 4 * CW;      // bytes (keys) per chunk
    // Two ways through L2, chosen by measurement (side by side, per shape).  A lane that holds a whole row of
    // 96 and more keys, or 16-byte chunks, marks its loaded lines evict-first and prefetches nothing (2 to 5 %
    // faster than the other way on 48, 96, 144 and 160 keys).  Every other shape -- lane groups, and a lane per
    // row of 32 or 64 keys -- loads at normal priority behind one bulk prefetch per CTA (64 keys: 1.2 % faster
    // than evict-first loads without a prefetch, 2 to 5 % in the leading-bit form and on longer launches;
    // evict-first loads behind a prefetch are the worst combination).
    constexpr bool kEvictFirst = G == 1 && (V > 2 || CW != 8);
    const int lane = threadIdx.x & 31;
    const int sub = lane % G;
    const uint32_t row = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * RW + lane / G;
    const bool live = row < (uint32_t)a.rows;
    // A lane beyond the last row repeats the last row's loads and arithmetic and stores nothing: cheaper
    // than a fill value for its registers, and every shuffle and vote below stays warp-wide.
    const uint32_t lrow = min(row, (uint32_t)a.rows - 1u);
    uint32_t bidx, head, qi;
    row_coords(lrow, a, bidx, head, qi);
    int nv = valid_keys_causal<CAUSAL>(qi, a);
    // Programmatic dependent launch: everything above touches no global memory, so it may run
    // while the previous kernel in the stream drains; all reads and writes come after the wait.
    asm volatile("griddepcontrol.launch_dependents;");
    // Before the wait: one bulk prefetch of the CTA's rows (they are contiguous) into L2.  A prefetch is safe
    // whatever the previous kernel of the stream still writes, because L2 is the point of coherence; in the first
    // wave it runs while that kernel drains, and in every wave the request leaves a prologue earlier than the
    // lanes' own loads: 4 to 7 % on 128-key causal heads, 1 % on 512-key rows.  Not for the evict-first shapes
    // (a prefetched line keeps its normal priority and crowds the output out of L2).
    if (!kEvictFirst && threadIdx.x == 0) {
        const uint32_t cta_row0 = blockIdx.x * (blockDim.x >> 5) * RW;        // (they are contiguous; row0 < rows)
        const uint32_t bytes = min((blockDim.x >> 5) * RW, (uint32_t)a.rows - cta_row0) * (uint32_t)a.Lk;   // a multiple of 16
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(x_all + (int64_t)cta_row0 * a.Lk), "r"(bytes));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const HeadEntry th = a.table[head];
    if (CAUSAL && a.key_len) nv = min(nv, max(a.key_len[bidx], 0));   // padding mask

    // Masked: a chunk index v whose columns lie beyond every row of this warp is skipped altogether
    // (warp-uniform), e.g. the right half of the first 64 queries of a 128-key causal head.
    const int warp_nv = CAUSAL ? __reduce_max_sync(0xffffffffu, nv) : a.Lk;
    auto chunk_used = [&](int v) { return !CAUSAL || v == 0 || v * G * CB < warp_nv; };
    int skipped_cols = 0;           // masked columns of this row that were never materialised
#pragma unroll
    for (int v = 1; v < V; ++v)
        if (!chunk_used(v)) skipped_cols += CB * G;

    // ---- loads: V independent requests per lane
    uint32_t e[NW], o[NW];          // first the raw words (in e), then the split lanes
    int cnt[V];                     // valid bytes of this lane's chunk v
    bool full[V];                   // warp-uniform: every lane's chunk v is complete
    const int8_t *x_row = x_all + (int64_t)lrow * a.Lk;
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int col = (sub + v * G) * CB;
        cnt[v] = CAUSAL ? min(max(nv - col, 0), CB) : CB;
        full[v] = !CAUSAL || __all_sync(0xffffffffu, cnt[v] == CB);
        uint32_t w[CW];
        if (cnt[v] > 0) {
            if constexpr (CW == 8) ldg256<kEvictFirst>(x_row + col, w);
            else ldg128<kEvictFirst>(x_row + col, w);
        } else {
#pragma unroll
            for (int k = 0; k < CW; ++k) w[k] = kMinus128x4;
        }
#pragma unroll
        for (int k = 0; k < CW; ++k) e[CW * v + k] = w[k];
    }

    // ---- split into 16-bit lanes; stage 1: row max
    uint32_t M = 0x80008000u;
#pragma unroll
    for (int v = 0; v < V; ++v) {
        if (!chunk_used(v)) continue;
        if (full[v]) {
#pragma unroll
            for (int k = CW * v; k < CW * v + CW; ++k) {
                const uint32_t w = e[k];
                e[k] = prmt(w, 0, kSelEven);
                o[k] = prmt(w, 0, kSelOdd);
                M = __vimax3_s16x2(M, e[k], o[k]);
            }
        } else {
#pragma unroll
            for (int k = 0; k < CW; ++k) {
                const uint32_t bm = byte_mask(cnt[v], k);
                const uint32_t w = (e[CW * v + k] & bm) | (kMinus128x4 & ~bm);
                e[CW * v + k] = prmt(w, 0, kSelEven);
                o[CW * v + k] = prmt(w, 0, kSelOdd);
                M = __vimax3_s16x2(M, e[CW * v + k], o[CW * v + k]);
            }
        }
    }
    int m = max((int)(short)(M & 0xffffu), (int)M >> 16);
#pragma unroll
    for (int s = G / 2; s; s >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, s));

    // ---- stages 2-4: closeness r = max(x + (D - m), 0) and its row sum
    const int cm = th.D - m;                               // in [-126, 255]
    const uint32_t c2 = prmt((uint32_t)cm, 0, 0x1010u);    // (cm, cm) as 16-bit lanes
    uint32_t racc = 0;
#pragma unroll
    for (int v = 0; v < V; ++v) {
        if (!chunk_used(v)) continue;
#pragma unroll
        for (int k = CW * v; k < CW * v + CW; ++k) {
            e[k] = __viaddmax_s16x2(e[k], c2, 0u);
            o[k] = __viaddmax_s16x2(o[k], c2, 0u);
            racc = __dp2a_lo(o[k], 0x0101u, __dp2a_lo(e[k], 0x0101u, racc));   // both lanes of both words, on the multiply pipe
        }
    }
    int rsum = (int)racc;
#pragma unroll
    for (int s = G / 2; s; s >>= 1) rsum += __shfl_xor_sync(0xffffffffu, rsum, s);
    // masked keys that were materialised were counted at x = -128
    if (CAUSAL) rsum -= ((PAD ? G * V * CB : a.Lk) - nv - skipped_cols) * max(cm - 128, 0);
    const int F = th.B - th.S * th.D;                      // floor score
    const uint32_t Z = (uint32_t)(nv * F + th.S * rsum);
    const uint32_t rho = reciprocal<U16, CLB>(max(Z, 1u));
    if (!live) return;

    // ---- stage 5: normalise and store
    if (U16) {
        const uint32_t a1 = (uint32_t)F * rho * 0x00010001u, b1 = (uint32_t)th.S * rho;
        uint16_t *p_row = (uint16_t *)p_all + (int64_t)row * a.Lk;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int col = (sub + v * G) * CB;
            if (PAD && col >= a.Lk) continue;
            uint32_t out[2 * CW];
            if (!chunk_used(v)) {
#pragma unroll
                for (int k = 0; k < 2 * CW; ++k) out[k] = 0;
            } else {
#pragma unroll
                for (int k = 0; k < CW; ++k) {
                    const uint32_t pe = e[CW * v + k] * b1 + a1, po = o[CW * v + k] * b1 + a1;
                    out[2 * k] = prmt(pe, po, 0x5410u);
                    out[2 * k + 1] = prmt(pe, po, 0x7632u);
                }
                if (!full[v]) {
#pragma unroll
                    for (int k = 0; k < CW; ++k) {
                        const uint32_t bm = byte_mask(cnt[v], k);
                        out[2 * k] &= prmt(bm, 0, 0x1100u);
                        out[2 * k + 1] &= prmt(bm, 0, 0x3322u);
                    }
                }
            }
            if constexpr (CW == 8) {
                uint32_t lo[8], hi[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) { lo[k] = out[k]; hi[k] = out[8 + k]; }
                stg256(p_row + col, lo);
                stg256(p_row + col + 16, hi);
            } else {
                // 16-byte chunks also serve tensors that are only 16-byte aligned: two 16-byte stores
                uint32_t lo[4], hi[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) { lo[k] = out[k]; hi[k] = out[4 + k]; }
                stg128(p_row + col, lo);
                stg128(p_row + col + 8, hi);
            }
        }
    } else {
        // rho' = rho << (1 - OUT_SHIFT) and p = X >> 16 for the divide; rho' = rho >> OUT_SHIFT (exact: the
        // leading-bit rho is 255 * 2^(15-k), k <= 14) and p = min(X >> 15, 255) for the leading-bit form, so
        // that X = s * rho' stays below 2^24 in both (s <= Z < 2^(k+1)).  That covers OUT_SHIFT 0 and 1; a
        // larger OUT_SHIFT is computed as OUT_SHIFT = 1 (no result above 127 / 255, no saturation) and the
        // packed bytes are shifted right by the rest afterwards: floor(floor(a / b) / c) = floor(a / (b c)).
        const int eff_shift = min(a.out_shift, 1), post_shift = a.out_shift - eff_shift;
        const uint32_t post_mask = (0xffu >> post_shift) * 0x01010101u;
        const uint32_t rp = CLB ? (rho >> eff_shift) : (rho << (1 - eff_shift));
        const uint32_t a1 = (uint32_t)F * rp, b1 = (uint32_t)th.S * rp;
        // X = a1 + b1*r.  With a1 = ah*256 + al and
        // b1 = bh*256 + bl, X >> 8 = ah + bh*r + ((al + bl*r) >> 8) =: Y < 2^16, and both ah + bh*r and
        // al + bl*r (r <= 127) fit 16 bits: a pair of elements takes two 32-bit multiply-adds on its 16-bit
        // lanes, one byte permute for the carry, one add, and p is the high byte of each lane of Y.
        const uint32_t ah2 = (a1 >> 8) * 0x00010001u, al2 = (a1 & 255u) * 0x00010001u;
        const uint32_t bh = b1 >> 8, bl = b1 & 255u;
        uint8_t *p_row = (uint8_t *)p_all + (int64_t)row * a.Lk;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int col = (sub + v * G) * CB;
            if (PAD && col >= a.Lk) continue;
            uint32_t out[CW];
            if (!chunk_used(v)) {
#pragma unroll
                for (int k = 0; k < CW; ++k) out[k] = 0;
            } else {
#pragma unroll
                for (int k = 0; k < CW; ++k) {
                    const uint32_t re = e[CW * v + k], ro = o[CW * v + k];
                    if (!CLB) {
                        const uint32_t ye = re * bh + ah2 + prmt(re * bl + al2, 0, 0x4341u);
                        const uint32_t yo = ro * bh + ah2 + prmt(ro * bl + al2, 0, 0x4341u);
                        out[k] = prmt(ye, yo, 0x7351u);
                    } else {
                        // the leading-bit reciprocal can overshoot: Y saturates at 255*128 + 127 in the add
                        // itself, and p = Y >> 7 is the high byte of each lane of 2*Y (the doubling runs on the multiply pipe)
                        const uint32_t ye = __viaddmin_u16x2(re * bh + ah2, prmt(re * bl + al2, 0, 0x4341u), 0x7fff7fffu);
                        const uint32_t yo = __viaddmin_u16x2(ro * bh + ah2, prmt(ro * bl + al2, 0, 0x4341u), 0x7fff7fffu);
                        out[k] = prmt(ye * 2u, yo * 2u, 0x7351u);
                    }
                }
                if (post_shift) {                              // uniform: OUT_SHIFT >= 2
#pragma unroll
                    for (int k = 0; k < CW; ++k) out[k] = (out[k] >> post_shift) & post_mask;
                }
                if (!full[v]) {
#pragma unroll
                    for (int k = 0; k < CW; ++k) out[k] &= byte_mask(cnt[v], k);
                }
            }
            if constexpr (CW == 8) stg256(p_row + col, out);
            else stg128(p_row + col, out);
        }
    }
}

template <int G, int V, bool U16, bool CLB, bool CAUSAL, int CW = 8, bool PAD = false>
cudaError_t launch_gv(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    constexpr int ROWS_PER_CTA = 8 * (32 / G);
    const unsigned blocks = (unsigned)(((int64_t)a.rows + ROWS_PER_CTA - 1) / ROWS_PER_CTA);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rows_split_kernel<G, V, U16, CLB, CAUSAL, CW, PAD>, x, p, a);
}

// align32: both tensors start on a 32-byte boundary (the 32-byte-chunk shapes need it; the 16-byte-chunk
// shapes only need 16-byte alignment, which the caller has checked).
template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_shape(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st, bool align32, bool *taken) {
    *taken = true;
    if (align32) switch (a.Lk) {
        case 32: return launch_gv<1, 1, U16, CLB, CAUSAL>(x, p, a, st);
        case 64:    // int16 output: two lanes per row (30.7 against 31.3 us for 2^20 rows); uint8: a lane per row
            if constexpr (U16) return launch_gv<2, 1, U16, CLB, CAUSAL>(x, p, a, st);
            else return launch_gv<1, 2, U16, CLB, CAUSAL>(x, p, a, st);
        case 128: return launch_gv<2, 2, U16, CLB, CAUSAL>(x, p, a, st);
        case 256: return launch_gv<4, 2, U16, CLB, CAUSAL>(x, p, a, st);
        case 512: return launch_gv<8, 2, U16, CLB, CAUSAL>(x, p, a, st);
        case 1024: return launch_gv<16, 2, U16, CLB, CAUSAL>(x, p, a, st);
        case 2048: return launch_gv<32, 2, U16, CLB, CAUSAL>(x, p, a, st);
        case 4096: return launch_gv<32, 4, U16, CLB, CAUSAL>(x, p, a, st);
        case 8192: return launch_gv<32, 8, U16, CLB, CAUSAL>(x, p, a, st);
        // three, five or seven 32-byte chunks per lane: the multiples of 32 whose odd part is 3, 5 or 7
        case 96: return launch_gv<1, 3, U16, CLB, CAUSAL>(x, p, a, st);
        case 192: return launch_gv<2, 3, U16, CLB, CAUSAL>(x, p, a, st);
        case 384: return launch_gv<4, 3, U16, CLB, CAUSAL>(x, p, a, st);
        case 768: return launch_gv<8, 3, U16, CLB, CAUSAL>(x, p, a, st);
        case 1536: return launch_gv<16, 3, U16, CLB, CAUSAL>(x, p, a, st);
        case 3072: return launch_gv<32, 3, U16, CLB, CAUSAL>(x, p, a, st);
        case 160: return launch_gv<1, 5, U16, CLB, CAUSAL>(x, p, a, st);
        case 320: return launch_gv<2, 5, U16, CLB, CAUSAL>(x, p, a, st);
        case 640: return launch_gv<4, 5, U16, CLB, CAUSAL>(x, p, a, st);
        case 1280: return launch_gv<8, 5, U16, CLB, CAUSAL>(x, p, a, st);
        case 2560: return launch_gv<16, 5, U16, CLB, CAUSAL>(x, p, a, st);
        case 224: return launch_gv<1, 7, U16, CLB, CAUSAL>(x, p, a, st);
        case 448: return launch_gv<2, 7, U16, CLB, CAUSAL>(x, p, a, st);
        case 896: return launch_gv<4, 7, U16, CLB, CAUSAL>(x, p, a, st);
        case 1792: return launch_gv<8, 7, U16, CLB, CAUSAL>(x, p, a, st);
        case 3584: return launch_gv<16, 7, U16, CLB, CAUSAL>(x, p, a, st);
        default: break;
    }
    // 16-byte chunks: Lk = 16 * G * V with V odd, 3 <= V <= 15 -- every multiple of 16 up to 7680 whose odd
    // part is at most 15 and that the cases above do not take (48, 80, 112, 144, 176, ..., 288, 576, ...)
    if (a.Lk % 16 == 0) {
        int v = a.Lk / 16, g = 1;
        while ((v & 1) == 0) { v >>= 1; g <<= 1; }
        if (g <= 32 && v >= 3 && v <= 15) {
#define HCCS_SPLIT16(GG, VV) if (g == GG && v == VV) return launch_gv<GG, VV, U16, CLB, CAUSAL, 4>(x, p, a, st);
#define HCCS_SPLIT16_G(VV) HCCS_SPLIT16(1, VV) HCCS_SPLIT16(2, VV) HCCS_SPLIT16(4, VV) HCCS_SPLIT16(8, VV) \
                           HCCS_SPLIT16(16, VV) HCCS_SPLIT16(32, VV)
            HCCS_SPLIT16_G(3) HCCS_SPLIT16_G(5) HCCS_SPLIT16_G(7) HCCS_SPLIT16_G(9) HCCS_SPLIT16_G(11)
            HCCS_SPLIT16_G(13) HCCS_SPLIT16_G(15)
#undef HCCS_SPLIT16_G
#undef HCCS_SPLIT16
        }
        // every other multiple of 16 up to 4096 (and every one when the tensors are only 16-byte aligned): eight
        // 16-byte chunks per lane, the smallest power of two of lanes that covers the row, the excess chunks
        // padded (masked path, also without a mask)
        const int chunks = a.Lk / 16;
        if (chunks <= 8 * 32) {
            if (chunks <= 8) return launch_gv<1, 8, U16, CLB, true, 4, true>(x, p, a, st);
            if (chunks <= 16) return launch_gv<2, 8, U16, CLB, true, 4, true>(x, p, a, st);
            if (chunks <= 32) return launch_gv<4, 8, U16, CLB, true, 4, true>(x, p, a, st);
            if (chunks <= 64) return launch_gv<8, 8, U16, CLB, true, 4, true>(x, p, a, st);
            if (chunks <= 128) return launch_gv<16, 8, U16, CLB, true, 4, true>(x, p, a, st);
            return launch_gv<32, 8, U16, CLB, true, 4, true>(x, p, a, st);
        }
        // ... and the multiples of 32 from there to 8192: eight 32-byte chunks per lane, a whole warp per row
        if (align32 && a.Lk % 32 == 0 && a.Lk <= 8192) return launch_gv<32, 8, U16, CLB, true, 8, true>(x, p, a, st);
    }
    *taken = false;
    return cudaSuccess;
}

}  // namespace

cudaError_t try_launch_split(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                             cudaStream_t stream, bool *taken) {
    *taken = false;
    if ((((uintptr_t)logits | (uintptr_t)probs) & 15u) != 0) return cudaSuccess;
    const bool align32 = (((uintptr_t)logits | (uintptr_t)probs) & 31u) == 0;
    switch (flags & 7u) {
        case 0: return launch_shape<false, false, false>(logits, probs, a, stream, align32, taken);
        case 1: return launch_shape<true, false, false>(logits, probs, a, stream, align32, taken);
        case 2: return launch_shape<false, true, false>(logits, probs, a, stream, align32, taken);
        case 3: return launch_shape<true, true, false>(logits, probs, a, stream, align32, taken);
        case 4: return launch_shape<false, false, true>(logits, probs, a, stream, align32, taken);
        case 5: return launch_shape<true, false, true>(logits, probs, a, stream, align32, taken);
        case 6: return launch_shape<false, true, true>(logits, probs, a, stream, align32, taken);
        default: return launch_shape<true, true, true>(logits, probs, a, stream, align32, taken);
    }
}

}  // namespace hccs
