// Row kernels of hccs_forward: Algorithm 1 of the paper applied to independent rows.
//
// Three kernels, all integer-only and bit-exact by construction (integer max and sum are
// order-independent, so any reduction tree gives the one correct result):
//   rows_split_kernel      (hccs_rows_split.cu) Lk = 32 ... 2048 in powers of two, 32-byte aligned:
//                          the fast path.
//   rows_lanegroup_kernel  other Lk % 16 == 0 up to 1024, 16-byte aligned: a group of G lanes
//                          owns a row, each lane holds V 16-byte vectors of it in registers.
//   rows_cta_kernel        (hccs_rows_cta.cu) longer rows with Lk % 16 == 0: one CTA per row, the
//                          row staged in shared memory by bulk asynchronous copies (TMA).
//   rows_span_kernel       (hccs_rows_span.cu) any other Lk up to 1024 and any alignment: runs of rows
//                          moved through shared memory as contiguous spans.
//   rows_generic_kernel    everything else (any Lk, any alignment): one warp per row, bytes.
//
// Word-parallel identities used by the fast kernels (all exact):
//   * the int8 logits are biased to unsigned once (x ^ 0x80 per byte); max and differences
//     are unchanged by the bias;
//   * delta = m*0x01010101 - w is one 32-bit subtract for four elements, because every byte of
//     the minuend is >= the byte below it (no borrow crosses a byte);
//   * Z = sum_j (B - S*delta_j) = n_valid*B - S*sum_j delta_j, so the sum stage only needs the
//     byte sum of the clamped distances (Eq. 3 and Eq. 5 combined);
//   * int8 output with OUT_SHIFT <= 1: p_j = (a - b*delta_j) >> 16 with a = B*rho << (1-OUT_SHIFT),
//     b = S*rho << (1-OUT_SHIFT); a < 2^25 always because B <= Z implies B*rho <= 255*2^15
//     (< 2 * that for the leading-bit reciprocal), so the result sits in byte 2 of an int32.
#include <cuda_runtime.h>
#include <stdint.h>

#include "hccs_device.cuh"
#include "hccs_internal.h"

namespace hccs {

namespace {

// ------------------------------------------------------------------------------------------
// Generic kernel: one warp per row, byte accesses, three passes over the (cached) row.
// ------------------------------------------------------------------------------------------
template <bool U16, bool CLB, bool CAUSAL>
__global__ void __launch_bounds__(256) rows_generic_kernel(const int8_t *__restrict__ x_all,
                                                           void *p_all, RowArgs a) {
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    for (int64_t r = (int64_t)blockIdx.x * warps_per_block + (threadIdx.x >> 5); r < a.rows;
         r += (int64_t)gridDim.x * warps_per_block) {
        uint32_t b, head, i;
        row_coords((uint32_t)r, a, b, head, i);
        const HeadEntry th = a.table[head];
        const int nv = valid_keys<CAUSAL>(b, i, a);
        const int8_t *x = x_all + r * a.Lk;
        // pass 1: m = max over the valid keys (Eq. 1)
        int m = -128;
        for (int j = lane; j < nv; j += 32) m = max(m, (int)x[j]);
        for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        // pass 2: Z = sum of the scores (Eq. 2, 3, 5)
        int z = 0;
        for (int j = lane; j < nv; j += 32) z += th.B - th.S * min(m - (int)x[j], th.D);
        for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
        const uint32_t rho = nv > 0 ? reciprocal<U16, CLB>((uint32_t)z) : 0u;
        // pass 3: p_j = s_j * rho (>> 15 + OUT_SHIFT for the int8 output path)
        if (U16) {
            uint16_t *p = (uint16_t *)p_all + r * a.Lk;
            for (int j = lane; j < a.Lk; j += 32) {
                uint32_t v = 0;
                if (j < nv) v = (uint32_t)(th.B - th.S * min(m - (int)x[j], th.D)) * rho;
                p[j] = (uint16_t)v;
            }
        } else {
            uint8_t *p = (uint8_t *)p_all + r * a.Lk;
            const int sh = 15 + a.out_shift;
            for (int j = lane; j < a.Lk; j += 32) {
                uint32_t v = 0;
                if (j < nv) {
                    v = ((uint32_t)(th.B - th.S * min(m - (int)x[j], th.D)) * rho) >> sh;
                    if (CLB) v = min(v, 255u);
                }
                p[j] = (uint8_t)v;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Lane-group kernel.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prefix_byte_mask(int nbytes) {   // nbytes in (-inf, +inf)
    if (nbytes >= 4) return 0xffffffffu;
    if (nbytes <= 0) return 0u;
    return (1u << (8 * nbytes)) - 1u;
}

template <int G, int V, bool U16, bool CLB, bool CAUSAL, int U>
__global__ void __launch_bounds__(256) rows_lanegroup_kernel(const int8_t *__restrict__ x_all,
                                                             void *p_all, RowArgs a, int slabs) {
    constexpr int ROWS_PER_SLAB = 32 / G;      // rows a warp holds at once
    const int lane = threadIdx.x & 31;
    const int sub = lane % G;                  // position of this lane inside its row group
    const int warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int slab0 = warp * U;
    if (slab0 >= slabs) return;

    uint4 w[U][V];
    int nv[U];
    int cnt[U][V];       // valid bytes of each vector (0..16)
    uint32_t rowid[U];
    HeadEntry th[U];

    // ---- all loads first, so that every lane has U*V 16-byte requests in flight
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t r = (uint32_t)(slab0 + u) * ROWS_PER_SLAB + lane / G;
        rowid[u] = r;
        const bool live = (slab0 + u) < slabs && r < (uint32_t)a.rows;
        uint32_t b = 0, head = 0, i = 0;
        if (live) row_coords(r, a, b, head, i);
        nv[u] = live ? valid_keys<CAUSAL>(b, i, a) : 0;
        th[u] = a.table[head];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int col = (sub + v * G) * 16;
            int c = live && col < a.Lk ? max(min(nv[u] - col, 16), 0) : -1;
            cnt[u][v] = c;                                   // -1: nothing to write either
            w[u][v] = make_uint4(0, 0, 0, 0);
            if (c > 0)
                w[u][v] = __ldg(reinterpret_cast<const uint4 *>(x_all + (int64_t)r * a.Lk + col));
        }
    }

#pragma unroll
    for (int u = 0; u < U; ++u) {
        uint32_t wu[V][4];
        // ---- stage 1: bias to unsigned, row max
        uint32_t mx = 0;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            wu[v][0] = w[u][v].x ^ 0x80808080u;
            wu[v][1] = w[u][v].y ^ 0x80808080u;
            wu[v][2] = w[u][v].z ^ 0x80808080u;
            wu[v][3] = w[u][v].w ^ 0x80808080u;
            if (CAUSAL) {
#pragma unroll
                for (int k = 0; k < 4; ++k) wu[v][k] &= prefix_byte_mask(cnt[u][v] - 4 * k);
            } else if (cnt[u][v] <= 0) {
#pragma unroll
                for (int k = 0; k < 4; ++k) wu[v][k] = 0;
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) mx = __vmaxu4(mx, wu[v][k]);
        }
        mx = __vmaxu4(mx, mx >> 16);
        mx = __vmaxu4(mx, mx >> 8) & 0xffu;
#pragma unroll
        for (int o = G / 2; o; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        // ---- stage 2: unsigned distance and clamp; stage 4: sum (of the distances)
        const uint32_t mrep = mx * 0x01010101u;
        uint32_t dsum = 0;
#pragma unroll
        for (int v = 0; v < V; ++v) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t d = __vminu4(mrep - wu[v][k], th[u].Drep);
                if (CAUSAL) d &= prefix_byte_mask(cnt[u][v] - 4 * k);
                else if (cnt[u][v] <= 0) d = 0;
                wu[v][k] = d;
                dsum = __dp4a(d, 0x01010101u, dsum);
            }
        }
#pragma unroll
        for (int o = G / 2; o; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
        // ---- stage 3 + 4: Z = n_valid*B - S*sum(delta); stage 5: reciprocal and normalise
        const uint32_t Z = (uint32_t)(nv[u] * th[u].B) - (uint32_t)th[u].S * dsum;
        const uint32_t rho = reciprocal<U16, CLB>(max(Z, 1u));
        if (U16) {
            const uint32_t a0 = (uint32_t)th[u].B * rho, b0 = (uint32_t)th[u].S * rho;
            uint16_t *p_row = (uint16_t *)p_all + (int64_t)rowid[u] * a.Lk;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (cnt[u][v] < 0) continue;
                const int col = (sub + v * G) * 16;
                uint32_t o[8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t d = wu[v][k];
                    // two 16-bit lanes per multiply: neither half can borrow (s_j >= 0) or
                    // overflow (s_j * rho < 2^16)
                    uint32_t lo = a0 * 0x00010001u - b0 * __byte_perm(d, 0, 0x4140);
                    uint32_t hi = a0 * 0x00010001u - b0 * __byte_perm(d, 0, 0x4342);
                    if (CAUSAL) {
                        const int nb = cnt[u][v] - 4 * k;
                        if (nb < 1) lo = 0; else if (nb < 2) lo &= 0xffffu;
                        if (nb < 3) hi = 0; else if (nb < 4) hi &= 0xffffu;
                    }
                    o[2 * k] = lo;
                    o[2 * k + 1] = hi;
                }
                if (!CAUSAL && cnt[u][v] <= 0) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) o[k] = 0;
                }
                uint4 *dst = reinterpret_cast<uint4 *>(p_row + col);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        } else {
            const int e = 1 - a.out_shift;          // 0 or 1 (the dispatcher guarantees it)
            const uint32_t a0 = ((uint32_t)th[u].B * rho) << e, b0 = ((uint32_t)th[u].S * rho) << e;
            uint8_t *p_row = (uint8_t *)p_all + (int64_t)rowid[u] * a.Lk;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (cnt[u][v] < 0) continue;
                const int col = (sub + v * G) * 16;
                uint32_t o[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t d = wu[v][k];
                    uint32_t x0 = a0 - b0 * (d & 0xffu);
                    uint32_t x1 = a0 - b0 * __byte_perm(d, 0, 0x4441);
                    uint32_t x2 = a0 - b0 * __byte_perm(d, 0, 0x4442);
                    uint32_t x3 = a0 - b0 * (d >> 24);
                    if (CLB) {   // the leading-bit reciprocal can overshoot 255: saturate
                        x0 = min(x0, 0x00ffffffu);
                        x1 = min(x1, 0x00ffffffu);
                        x2 = min(x2, 0x00ffffffu);
                        x3 = min(x3, 0x00ffffffu);
                    }
                    uint32_t q = __byte_perm(__byte_perm(x0, x1, 0x0062), __byte_perm(x2, x3, 0x0062),
                                             0x5410);
                    if (CAUSAL) q &= prefix_byte_mask(cnt[u][v] - 4 * k);
                    o[k] = q;
                }
                if (!CAUSAL && cnt[u][v] <= 0) o[0] = o[1] = o[2] = o[3] = 0;
                *reinterpret_cast<uint4 *>(p_row + col) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
}

template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_generic(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    const int warps_per_block = 8;
    int64_t blocks = ((int64_t)a.rows + warps_per_block - 1) / warps_per_block;
    if (blocks > 148 * 64) blocks = 148 * 64;
    rows_generic_kernel<U16, CLB, CAUSAL><<<(unsigned)blocks, warps_per_block * 32, 0, st>>>(x, p, a);
    return cudaGetLastError();
}

template <int G, int V, bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_lanegroup_gv(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    constexpr int U = (U16 || V > 1) ? 1 : 2;
    constexpr int ROWS_PER_SLAB = 32 / G;
    const int slabs = (a.rows + ROWS_PER_SLAB - 1) / ROWS_PER_SLAB;
    const int warps = (slabs + U - 1) / U;
    const int blocks = (warps + 7) / 8;
    rows_lanegroup_kernel<G, V, U16, CLB, CAUSAL, U><<<blocks, 256, 0, st>>>(x, p, a, slabs);
    return cudaGetLastError();
}

template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_lanegroup(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    const int nvec = a.Lk / 16;
    if (nvec <= 1) return launch_lanegroup_gv<1, 1, U16, CLB, CAUSAL>(x, p, a, st);
    if (nvec <= 2) return launch_lanegroup_gv<2, 1, U16, CLB, CAUSAL>(x, p, a, st);
    if (nvec <= 4) return launch_lanegroup_gv<4, 1, U16, CLB, CAUSAL>(x, p, a, st);
    if (nvec <= 8) return launch_lanegroup_gv<8, 1, U16, CLB, CAUSAL>(x, p, a, st);
    if (nvec <= 16) return launch_lanegroup_gv<16, 1, U16, CLB, CAUSAL>(x, p, a, st);
    if (nvec <= 32) return launch_lanegroup_gv<32, 1, U16, CLB, CAUSAL>(x, p, a, st);
    return launch_lanegroup_gv<32, 2, U16, CLB, CAUSAL>(x, p, a, st);
}

template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_mode(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    const bool aligned = (((uintptr_t)x | (uintptr_t)p) & 15u) == 0 && a.Lk % 16 == 0;
    const bool shift_ok = U16 || a.out_shift <= 1;
    if (aligned && shift_ok) {
        bool taken = false;
        cudaError_t e = try_launch_split(x, p, a, (U16 ? 1u : 0u) | (CLB ? 2u : 0u) | (CAUSAL ? 4u : 0u), st,
                                         &taken);
        if (taken) return e;
    }
    if (aligned && shift_ok && a.Lk <= 1024) return launch_lanegroup<U16, CLB, CAUSAL>(x, p, a, st);
    if (shift_ok && a.Lk <= 1024) {         // any other length or alignment: rows moved as contiguous spans
        bool taken = false;
        cudaError_t e = try_launch_span(x, p, a, (U16 ? 1u : 0u) | (CLB ? 2u : 0u) | (CAUSAL ? 4u : 0u), st, &taken);
        if (taken) return e;
    }
    if (aligned) {
        bool taken = false;
        cudaError_t e = try_launch_cta(x, p, a, (U16 ? 1u : 0u) | (CLB ? 2u : 0u) | (CAUSAL ? 4u : 0u), st,
                                       &taken);
        if (taken) return e;
    }
    return launch_generic<U16, CLB, CAUSAL>(x, p, a, st);
}

}  // namespace

cudaError_t launch_rows(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                        cudaStream_t stream, uint64_t *launches) {
    cudaError_t e;
    const uint32_t sel = (flags & 3u) | (((flags & 4u) || a.key_len) ? 4u : 0u);   // bit 2: any masking
    switch (sel) {
        case 0: e = launch_mode<false, false, false>(logits, probs, a, stream); break;
        case 1: e = launch_mode<true, false, false>(logits, probs, a, stream); break;
        case 2: e = launch_mode<false, true, false>(logits, probs, a, stream); break;
        case 3: e = launch_mode<true, true, false>(logits, probs, a, stream); break;
        case 4: e = launch_mode<false, false, true>(logits, probs, a, stream); break;
        case 5: e = launch_mode<true, false, true>(logits, probs, a, stream); break;
        case 6: e = launch_mode<false, true, true>(logits, probs, a, stream); break;
        default: e = launch_mode<true, true, true>(logits, probs, a, stream); break;
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace hccs
