// Row kernels of hccs_forward: Algorithm 1 of the paper applied to independent rows.
//
// Four kernels, all integer-only and bit-exact by construction (integer max and sum are
// order-independent, so any reduction tree gives the one correct result).  launch_mode picks, in this order:
//   rows_split_kernel    (hccs_rows_split.cu) Lk % 16 == 0 up to 4096 (and the multiples of 32 up to 8192),
//                        16-byte aligned tensors: rows held in registers by groups of lanes, 32- or 16-byte
//                        chunks; the fast path.
//   rows_span_kernel     (hccs_rows_span.cu) any other Lk up to 1024 and any alignment: runs of rows moved
//                        through shared memory as contiguous spans.
//   rows_cta_kernel      (hccs_rows_cta.cu) longer rows with Lk % 16 == 0 and 16-byte aligned tensors: one CTA
//                        per row, the row staged in shared memory by bulk asynchronous copies (TMA).
//   rows_generic_kernel  (this file) everything else (any Lk, any alignment): one warp per row, byte accesses.
// Every kernel takes every OUT_SHIFT of the int8 output path.
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

template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_generic(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    const int warps_per_block = 8;
    int64_t blocks = ((int64_t)a.rows + warps_per_block - 1) / warps_per_block;
    if (blocks > 148 * 64) blocks = 148 * 64;
    rows_generic_kernel<U16, CLB, CAUSAL><<<(unsigned)blocks, warps_per_block * 32, 0, st>>>(x, p, a);
    return cudaGetLastError();
}

template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_mode(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    const bool aligned = (((uintptr_t)x | (uintptr_t)p) & 15u) == 0 && a.Lk % 16 == 0;
    if (aligned) {
        bool taken = false;
        cudaError_t e = try_launch_split(x, p, a, (U16 ? 1u : 0u) | (CLB ? 2u : 0u) | (CAUSAL ? 4u : 0u), st,
                                         &taken);
        if (taken) return e;
    }
    if (a.Lk <= 1024) {                     // any other length or alignment: rows moved as contiguous spans
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
