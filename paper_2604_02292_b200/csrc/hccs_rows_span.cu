// Row kernel for any row length up to 1024 keys and any alignment of the tensors: rows whose
// length is no multiple of 32 bytes cannot be fetched by the register-resident kernel with one
// aligned vector load per lane, because a row then starts at an arbitrary byte.
//
// A CTA takes a run of consecutive rows -- one contiguous span of bytes, rows being back to back --
// and moves it as a span: aligned 16-byte loads of the span's interior into shared memory (the
// few bytes before the first and after the last 16-byte boundary go one by one), the rows are
// worked on from shared memory, the results are laid down in a second span in shared memory and
// leave it the same way.  Global memory traffic is therefore coalesced whatever Lk is.
//
// Inside the CTA G lanes own a row (G a power of two, up to 8 words of four keys per lane): a lane
// assembles each of its words from the two aligned shared-memory words that hold it (the row
// starts at an arbitrary byte), and from there Algorithm 1 runs on 16-bit pairs exactly as in
// the register-resident kernel: stage 1 row max, stages 2-4 closeness r = max(x + (D - m), 0)
// and its sum, stage 5 one reciprocal per row and p = (F*rho' + S*rho'*r) >> 16.  Word slots and
// bytes beyond the row's valid keys (row end, causal rule, key length) are set to -128, can
// then never raise the max, and their closeness is taken out of the sum in closed form.
#include <cuda_runtime.h>
#include <stdint.h>

#include "hccs_device.cuh"
#include "hccs_internal.h"

namespace hccs {

namespace {

constexpr int kSpanThreads = 256;
constexpr int kMaxWordsPerLane = 8;
constexpr uint32_t kMinus128x4 = 0x80808080u;

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t prefix_mask(int nbytes) {        // low nbytes bytes set (0..4, clamped)
    return nbytes >= 4 ? 0xffffffffu : (nbytes <= 0 ? 0u : (1u << (8 * nbytes)) - 1u);
}

// Copies `bytes` bytes between global and shared memory; the two addresses are congruent modulo 16,
// so the interior moves as aligned 16-byte vectors.  TO_SHARED: global -> shared, else shared -> global.
template <bool TO_SHARED>
__device__ __forceinline__ void copy_span(uint8_t *sm, uint8_t *gm, int64_t bytes) {
    const int head = (int)min((int64_t)((16 - ((uintptr_t)gm & 15)) & 15), bytes);
    const int64_t nvec = (bytes - head) >> 4;
    const int tail = (int)(bytes - head - (nvec << 4));
    for (int64_t v = threadIdx.x; v < nvec; v += kSpanThreads) {
        uint4 *s = reinterpret_cast<uint4 *>(sm + head + (v << 4));
        uint4 *g = reinterpret_cast<uint4 *>(gm + head + (v << 4));
        if (TO_SHARED) *s = *g; else *g = *s;
    }
    const int edge = (int)threadIdx.x;
    if (edge < head) { if (TO_SHARED) sm[edge] = gm[edge]; else gm[edge] = sm[edge]; }
    if (edge >= 32 && edge - 32 < tail) {
        const int64_t o = head + (nvec << 4) + (edge - 32);
        if (TO_SHARED) sm[o] = gm[o]; else gm[o] = sm[o];
    }
}

template <int kWordsPerLane, bool U16, bool CLB, bool MASKED>
__global__ void __launch_bounds__(kSpanThreads) rows_span_kernel(const int8_t *x_all, void *p_all, RowArgs a,
                                                                  int rows_per_cta, int log2_g) {
    extern __shared__ __align__(16) uint8_t smem[];
    constexpr int OSZ = U16 ? 2 : 1;
    const int Lk = a.Lk;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_cta;
    const int nr = (int)min((int64_t)rows_per_cta, (int64_t)a.rows - r0);
    const int64_t in_bytes = (int64_t)nr * Lk, out_bytes = in_bytes * OSZ;
    uint8_t *g_in = const_cast<uint8_t *>(reinterpret_cast<const uint8_t *>(x_all)) + r0 * Lk;
    uint8_t *g_out = reinterpret_cast<uint8_t *>(p_all) + r0 * Lk * OSZ;
    // shared-memory images start at the same offset modulo 16 as their global spans
    const int mis_in = (int)((uintptr_t)g_in & 15), mis_out = (int)((uintptr_t)g_out & 15);
    const int in_room = (rows_per_cta * Lk + 47) & ~15;             // image + misalignment + one word of slack
    uint8_t *s_in = smem + mis_in;
    uint8_t *s_out = smem + in_room + mis_out;

    copy_span<true>(s_in, g_in, in_bytes);
    __syncthreads();

    const int G = 1 << log2_g;
    const int sub = threadIdx.x & (G - 1);
    const int groups = kSpanThreads >> log2_g;                        // rows worked on at once
    const int W = (Lk + 3) >> 2;                                      // words of a row, the last one maybe partial
    const uint32_t *s_in_w = reinterpret_cast<const uint32_t *>(smem);
    for (int i0 = 0; i0 < nr; i0 += groups) {                         // same trip count for every thread
        const int i = i0 + (threadIdx.x >> log2_g);
        const bool live = i < nr;
        uint32_t bidx = 0, head = 0, qi = 0;
        if (live) row_coords((uint32_t)(r0 + i), a, bidx, head, qi);
        const int nv = live ? valid_keys<MASKED>(bidx, qi, a) : 0;
        const HeadEntry th = a.table[head];

        // ---- the lane's words: word j of the row lies at byte mis_in + i*Lk + 4j of the image.
        // valid bytes of word j: min(nv - 4j, 4); without a mask only the row's last word can be partial
        const int rb = mis_in + i * Lk;
        const uint32_t sel = 0x3210u + 0x1111u * (uint32_t)(rb & 3);
        const uint32_t tail_mask = prefix_mask(Lk - 4 * (W - 1));
        auto word_mask = [&](int j) -> uint32_t {
            if (MASKED) return __funnelshift_rc(0xffffffffu, 0u, 32 - 8 * min(max(nv - 4 * j, 0), 4));
            return j == W - 1 ? tail_mask : 0xffffffffu;
        };
        uint32_t e[kWordsPerLane], o[kWordsPerLane];
        uint32_t M = 0x80008000u;
        {
            int j = sub, wi = (rb >> 2) + sub;
#pragma unroll
            for (int k = 0; k < kWordsPerLane; ++k, j += G, wi += G) {
                uint32_t w = kMinus128x4;
                if (live && j < W && (!MASKED || 4 * j < nv)) {
                    w = prmt(s_in_w[wi], s_in_w[wi + 1], sel);
                    const uint32_t bm = word_mask(j);
                    w = (w & bm) | (kMinus128x4 & ~bm);
                }
                const uint32_t ev = prmt(w, 0, 0xA280u), od = prmt(w, 0, 0xB391u);
                e[k] = ev;
                o[k] = od;
                M = __vimax3_s16x2(M, ev, od);
            }
        }
        int m = max((int)(short)(M & 0xffffu), (int)M >> 16);
        for (int s = G >> 1; s; s >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, s));

        // ---- closeness and its sum; every slot that holds no valid key was counted at x = -128
        const int cm = th.D - m;
        const uint32_t c2 = prmt((uint32_t)cm, 0, 0x1010u);
        uint32_t rsum2 = 0;
#pragma unroll
        for (int k = 0; k < kWordsPerLane; ++k) {
            e[k] = __viaddmax_s16x2(e[k], c2, 0u);
            o[k] = __viaddmax_s16x2(o[k], c2, 0u);
            rsum2 = rsum2 + e[k] + o[k];
        }
        int rsum = (int)(rsum2 & 0xffffu) + (int)(rsum2 >> 16);
        for (int s = G >> 1; s; s >>= 1) rsum += __shfl_xor_sync(0xffffffffu, rsum, s);
        rsum -= (4 * kWordsPerLane * G - nv) * max(cm - 128, 0);
        const int F = th.B - th.S * th.D;
        const uint32_t Z = (uint32_t)(nv * F + th.S * rsum);
        const uint32_t rho = reciprocal<U16, CLB>(max(Z, 1u));
        if (!live) continue;

        // ---- normalise into the output image (rows start at arbitrary bytes there too): word j of the
        // row goes to byte ob + 4j*OSZ of the shared-memory array; whole aligned words in one store
        const int ob = in_room + mis_out + i * Lk * OSZ;
        const bool row_aligned = (ob & 3) == 0;
        if (U16) {
            const uint32_t a1 = (uint32_t)F * rho * 0x00010001u, b1 = (uint32_t)th.S * rho;
            int j = sub;
#pragma unroll
            for (int k = 0; k < kWordsPerLane; ++k, j += G) {
                if (j >= W) continue;
                const uint32_t pe = e[k] * b1 + a1, po = o[k] * b1 + a1;   // (p0, p2) and (p1, p3) as 16-bit pairs
                uint32_t q0 = prmt(pe, po, 0x5410u), q1 = prmt(pe, po, 0x7632u);
                const uint32_t bm = word_mask(j);
                q0 &= prmt(bm, 0, 0x1100u);
                q1 &= prmt(bm, 0, 0x3322u);
                const int left = Lk - 4 * j;                                      // keys of the row from this word on
                uint8_t *dst = smem + ob + 8 * j;
                if (row_aligned && left >= 4) {
                    reinterpret_cast<uint32_t *>(dst)[0] = q0;
                    reinterpret_cast<uint32_t *>(dst)[1] = q1;
                } else {
                    uint16_t *d16 = reinterpret_cast<uint16_t *>(dst);           // uint16 tensors are 2-byte aligned
                    d16[0] = (uint16_t)q0;
                    if (left > 1) d16[1] = (uint16_t)(q0 >> 16);
                    if (left > 2) d16[2] = (uint16_t)q1;
                    if (left > 3) d16[3] = (uint16_t)(q1 >> 16);
                }
            }
        } else {
            // the pair arithmetic of the register-resident kernel: X = s * rho' < 2^24 with the coefficients split
            // at 8 bits, two 32-bit multiply-adds per pair of keys on 16-bit lanes
            // an OUT_SHIFT above 1 is computed as OUT_SHIFT = 1 and the packed bytes are shifted by the rest
            const int eff_shift = min(a.out_shift, 1), post_shift = a.out_shift - eff_shift;
            const uint32_t post_mask = (0xffu >> post_shift) * 0x01010101u;
            const uint32_t rp = CLB ? (rho >> eff_shift) : (rho << (1 - eff_shift));
            const uint32_t a1 = (uint32_t)F * rp, b1 = (uint32_t)th.S * rp;
            const uint32_t ah2 = (a1 >> 8) * 0x00010001u, al2 = (a1 & 255u) * 0x00010001u;
            const uint32_t bh = b1 >> 8, bl = b1 & 255u;
            int j = sub;
#pragma unroll
            for (int k = 0; k < kWordsPerLane; ++k, j += G) {
                if (j >= W) continue;
                uint32_t q;
                if (!CLB) {
                    const uint32_t ye = e[k] * bh + ah2 + prmt(e[k] * bl + al2, 0, 0x4341u);
                    const uint32_t yo = o[k] * bh + ah2 + prmt(o[k] * bl + al2, 0, 0x4341u);
                    q = prmt(ye, yo, 0x7351u);
                } else {
                    const uint32_t ye = __viaddmin_u16x2(e[k] * bh + ah2, prmt(e[k] * bl + al2, 0, 0x4341u), 0x7fff7fffu);
                    const uint32_t yo = __viaddmin_u16x2(o[k] * bh + ah2, prmt(o[k] * bl + al2, 0, 0x4341u), 0x7fff7fffu);
                    q = prmt(ye * 2u, yo * 2u, 0x7351u);
                }
                if (post_shift) q = (q >> post_shift) & post_mask;
                q &= word_mask(j);
                const int left = Lk - 4 * j;
                uint8_t *dst = smem + ob + 4 * j;
                if (row_aligned && left >= 4) {
                    *reinterpret_cast<uint32_t *>(dst) = q;
                } else {
                    dst[0] = (uint8_t)q;
                    if (left > 1) dst[1] = (uint8_t)(q >> 8);
                    if (left > 2) dst[2] = (uint8_t)(q >> 16);
                    if (left > 3) dst[3] = (uint8_t)(q >> 24);
                }
            }
        }
    }
    __syncthreads();
    copy_span<false>(s_out, g_out, out_bytes);
}

template <int WPL, bool U16, bool CLB, bool MASKED>
cudaError_t launch_span_w(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st, int log2_g) {
    constexpr int OSZ = U16 ? 2 : 1;
    // rows per CTA: both images within 48 KB of shared memory, at most four passes of all lane groups
    const int budget = 47 * 1024 - 64;
    int rows_per_cta = budget / (a.Lk * (1 + OSZ));
    const int groups = kSpanThreads >> log2_g;
    if (rows_per_cta > 4 * groups) rows_per_cta = 4 * groups;
    if (rows_per_cta < 1) rows_per_cta = 1;
    const size_t smem = (size_t)((rows_per_cta * a.Lk + 47) & ~15) + (size_t)((rows_per_cta * a.Lk * OSZ + 31) & ~15) + 16;
    const unsigned blocks = (unsigned)(((int64_t)a.rows + rows_per_cta - 1) / rows_per_cta);
    rows_span_kernel<WPL, U16, CLB, MASKED><<<blocks, kSpanThreads, smem, st>>>(x, p, a, rows_per_cta, log2_g);
    return cudaGetLastError();
}

template <bool U16, bool CLB, bool MASKED>
cudaError_t launch_span(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    // G lanes per row, the smallest power of two that covers the row's words with at most 8 per lane;
    // then as few words per lane as cover it (the unused slots of a lane cost as much as the used ones)
    const int W = (a.Lk + 3) / 4;
    int log2_g = 0;
    while ((kMaxWordsPerLane << log2_g) < W) ++log2_g;
    const int wpl = (W + (1 << log2_g) - 1) >> log2_g;
    switch (wpl) {
        case 1: return launch_span_w<1, U16, CLB, MASKED>(x, p, a, st, log2_g);
        case 2: return launch_span_w<2, U16, CLB, MASKED>(x, p, a, st, log2_g);
        case 3: return launch_span_w<3, U16, CLB, MASKED>(x, p, a, st, log2_g);
        case 4: return launch_span_w<4, U16, CLB, MASKED>(x, p, a, st, log2_g);
        case 5: return launch_span_w<5, U16, CLB, MASKED>(x, p, a, st, log2_g);
        case 6: return launch_span_w<6, U16, CLB, MASKED>(x, p, a, st, log2_g);
        case 7: return launch_span_w<7, U16, CLB, MASKED>(x, p, a, st, log2_g);
        default: return launch_span_w<8, U16, CLB, MASKED>(x, p, a, st, log2_g);
    }
}

}  // namespace

cudaError_t try_launch_span(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                            cudaStream_t stream, bool *taken) {
    *taken = false;
    if (a.Lk < 1 || a.Lk > 4 * kMaxWordsPerLane * 32) return cudaSuccess;  // 1024 keys at most
    *taken = true;
    switch (flags & 7u) {
        case 0: return launch_span<false, false, false>(logits, probs, a, stream);
        case 1: return launch_span<true, false, false>(logits, probs, a, stream);
        case 2: return launch_span<false, true, false>(logits, probs, a, stream);
        case 3: return launch_span<true, true, false>(logits, probs, a, stream);
        case 4: return launch_span<false, false, true>(logits, probs, a, stream);
        case 5: return launch_span<true, false, true>(logits, probs, a, stream);
        case 6: return launch_span<false, true, true>(logits, probs, a, stream);
        default: return launch_span<true, true, true>(logits, probs, a, stream);
    }
}

}  // namespace hccs
