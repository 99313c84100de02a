// Internal declarations shared by the translation units of libhccs (not installed).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "hccs.h"

namespace hccs {

// One head's theta in the form the kernels read with a single 16-byte load.
struct __align__(16) HeadEntry {
    int32_t B;        // B_h
    int32_t S;        // S_h
    int32_t D;        // Dmax_h
    int32_t pad;      // (keeps the entry at one 16-byte load)
};

// Division of a 31-bit dividend by a runtime constant: q = (umulhi(n, mul) + n) >> shift.
struct FastDiv {
    uint32_t mul;
    uint32_t shift;
    uint32_t d;
};
FastDiv make_fastdiv(uint32_t d);

// Everything a row kernel needs besides the two tensors.
struct RowArgs {
    const HeadEntry *table;   // device, num_heads entries
    uint32_t *status;         // device status word (bounded waits report here)
    long long wait_cycles;    // limit of every device-side wait, in SM clock cycles
    int32_t rows;             // B*H*Lq
    int32_t H, Lq, Lk;
    int32_t causal_off;       // Lk - Lq
    int32_t causal;           // 1: key j of query i valid iff j <= i + causal_off
    const int32_t *key_len;   // device, one entry per batch entry, or NULL: keys beyond key_len[b] are padding
    int32_t out_shift;        // OUT_SHIFT of Eq. 8
    int32_t slice0;           // b*H + h of flat row 0 (views that start mid-tensor)
    FastDiv div_Lq, div_H;
};

// Bits of the device status word.
enum : uint32_t {
    STATUS_ROW_TMA_TIMEOUT = 1u,     // CTA-per-row kernel: a bulk copy never completed
    STATUS_FUSED_TIMEOUT = 2u,       // fused kernel: an mbarrier wait gave up
};

struct FusedArgs {
    const int8_t *Q, *K, *V;
    void *O;                       // int32 [B,H,L,d]; float when out_mode == 1; int8 when out_mode == 2
    const HeadEntry *table;
    const int32_t *requant_mult;   // device, 8 words per head: see fused_common in hccs_api.cu
    int32_t out_mode;              // 0: int32 accumulators; 1: float(acc) * scale_h; 2: acc requantised to int8
    int32_t out_requant_shift;     // out_mode 2: shift of the output requantisation (multipliers: word 5 of the table)
    const int32_t *key_len;        // device, one entry per batch entry, or NULL: keys beyond key_len[b] are padding
    uint32_t *status;
    long long wait_cycles;         // limit of every device-side wait, in SM clock cycles
    int32_t requant_shift;
    int32_t B, H, L, d;
    int32_t out_shift;
    uint32_t flags;
};

// Launchers.  Each returns the CUDA error of the launch and adds to *launches.
cudaError_t launch_rows(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                        cudaStream_t stream, uint64_t *launches);
// Register-resident split-lane kernel (hccs_rows_split.cu): *taken tells whether the shape fit.
cudaError_t try_launch_split(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                             cudaStream_t stream, bool *taken);
// Span kernel for any row length up to 1024 keys and any alignment (hccs_rows_span.cu).
cudaError_t try_launch_span(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                            cudaStream_t stream, bool *taken);
// CTA-per-row kernel for long rows (hccs_rows_cta.cu).
cudaError_t try_launch_cta(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                           cudaStream_t stream, bool *taken);
cudaError_t launch_fused(const FusedArgs &a, cudaStream_t stream, uint64_t *launches);
bool fused_shape_supported(int32_t L, int32_t d);
// One CTA that waits on an mbarrier nobody arrives on, through the production wait helpers, with the given
// limit: mode 0 the plain bounded wait (STATUS_ROW_TMA_TIMEOUT), mode 1 the abortable one (STATUS_FUSED_TIMEOUT).
cudaError_t launch_wait_probe(uint32_t *status, int mode, long long limit_cycles, cudaStream_t stream);

constexpr long long kDefaultWaitCycles = 2000000000ll;   // about one second of SM clocks

}  // namespace hccs
