// Device helpers shared by the row kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "hccs_internal.h"

namespace hccs {

constexpr uint32_t kTprimeU8 = 255u << 15;   // 255 * 2^R, R = INV_SHIFT = 15 (Eq. 8)
constexpr uint32_t kTprimeU16 = 32767u;      // T for int16 output (Eq. 6)

__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv &f) {
    return (__umulhi(n, f.mul) + n) >> f.shift;
}

// (batch entry, head, query index) of flat row r: slice = r / Lq + slice0, b = slice / H,
// head = slice mod H, i = r mod Lq.
__device__ __forceinline__ void row_coords(uint32_t r, const RowArgs &a, uint32_t &b, uint32_t &head, uint32_t &i) {
    uint32_t bh = fast_div(r, a.div_Lq);
    i = r - bh * (uint32_t)a.Lq;
    bh += (uint32_t)a.slice0;
    b = fast_div(bh, a.div_H);
    head = bh - b * (uint32_t)a.H;
}

// Stage 5 of the kernel overview: the one scalar operation per row, rho = floor(T'/Z) (Eq. 6,
// Eq. 8) or T' >> floor(log2 Z) (Eq. 9).  Z >= 1.
//
// The exact quotient is taken without an integer divide: a float estimate that is never above
// T'/Z and less than one below it, then one upward correction.  rcp.approx and the
// round-toward-zero multiply are each within 2^-22 relative; the numerator is pre-scaled by
// (1 - 2^-20), so the estimate lies in (T'/Z * (1 - 2^-19.5) - 1, T'/Z]; for quotients up to
// 2^15 the relative part is below 0.05, hence floor(estimate) is q or q - 1.  Quotients above
// 2^15 (int8 path with Z < 256: rows with few valid keys) take the plain divide.
template <bool U16, bool CLB>
__device__ __forceinline__ uint32_t reciprocal(uint32_t Z) {
    constexpr uint32_t Tp = U16 ? kTprimeU16 : kTprimeU8;
    if (CLB) return Tp >> (31 - __clz((int)Z));
    if (!U16 && Z < 256u) return Tp / Z;
    constexpr float kScaled = U16 ? 32766.96875f : 8355832.0f;   // T' * (1 - 2^-20), exact in fp32
    float rz;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rz) : "f"(__uint2float_rz(Z)));
    const uint32_t q = __float2uint_rz(__fmul_rz(kScaled, rz));
    const uint32_t rem = Tp - q * Z;
    return q + (rem >= Z ? 1u : 0u);
}

// Number of valid keys of query i of batch entry b: always a prefix of the row.  MASKED kernels
// apply the causal rule (when a.causal) and the per-batch key length (when a.key_len is set).
template <bool MASKED>
__device__ __forceinline__ int valid_keys_causal(uint32_t i, const RowArgs &a) {
    if (!MASKED || !a.causal) return a.Lk;
    return min(max((int)i + a.causal_off + 1, 0), a.Lk);
}
template <bool MASKED>
__device__ __forceinline__ int valid_keys(uint32_t b, uint32_t i, const RowArgs &a) {
    int nv = valid_keys_causal<MASKED>(i, a);
    if (MASKED && a.key_len) nv = min(nv, max(a.key_len[b], 0));   // reads global memory
    return nv;
}

// ---- mbarrier waits with a limit (shared by the TMA-staged row kernel, the fused kernel and the
// wait-limit probe): no wait in this library spins without one.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
// Waits for the phase with the given parity for at most `limit_cycles` SM clock cycles; false when the
// limit ran out (the caller records it in the status word and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long limit_cycles) {
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > limit_cycles) return false;
    }
}
// The same for a CTA whose threads wait on many barriers: the first wait that runs out raises the CTA's
// abort flag and sets `status_bit` in the status word; every other wait sees the flag and gives up too.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                                    uint32_t *status, uint32_t status_bit, long long limit_cycles) {
    long long t0 = 0;
    for (uint32_t polls = 0;; ++polls) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((polls & 31u) != 31u) continue;          // look at the flag and the clock now and then
        if (*abort_flag) return false;
        const long long now = clock64();
        if (t0 == 0) t0 = now;
        if (now - t0 > limit_cycles) {
            *abort_flag = 1;
            atomicOr(status, status_bit);
            return false;
        }
    }
}

}  // namespace hccs
