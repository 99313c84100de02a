// CTA-per-row kernel for long rows (Lk % 16 == 0, up to 32752 keys): Algorithm 1 with the row
// staged in shared memory.
//
// Persistent CTAs walk over the rows with a stride of the grid size (neighbouring rows go to different
// CTAs, which also spreads the cheap and the costly rows of a causal mask; no counter, no scratch word
// that two launches could share).  For every row one thread issues a 1-D bulk asynchronous copy (TMA,
// cp.async.bulk) of the row's valid prefix into one of two shared-memory stages; the copy of
// the next row is in flight while the CTA makes its three passes over the current one:
//   pass 1  row max (Eq. 1)            pass 2  sum of the clamped scores (Eq. 2, 3, 5)
//   once    reciprocal (Eq. 6 / 8 / 9) pass 3  normalise (Eq. 7 / int8 output path) into an
//                                              output stage, written back by a bulk store.
// The element arithmetic is the same 16-bit-pair formulation as the register-resident kernel.
// Every wait on an mbarrier is bounded (RowArgs::wait_cycles): when it runs out the CTA records
// STATUS_ROW_TMA_TIMEOUT in the status word and stops taking rows.  No multicast, no clusters.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "hccs_device.cuh"
#include "hccs_internal.h"

namespace hccs {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem),
                 "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

__device__ __forceinline__ uint32_t byte_prefix_mask(int nb) {
    return nb >= 4 ? 0xffffffffu : (nb <= 0 ? 0u : (1u << (8 * nb)) - 1u);
}

__device__ __forceinline__ int block_reduce(int v, bool is_max, int *scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int s = 16; s; s >>= 1) {
        const int other = __shfl_xor_sync(0xffffffffu, v, s);
        v = is_max ? max(v, other) : v + other;
    }
    __syncthreads();                       // the previous user of scratch is done
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    int r = scratch[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) r = is_max ? max(r, scratch[w]) : r + scratch[w];
    return r;
}

struct RowJob {
    int32_t row;        // -1: no more rows
    int32_t nv;         // valid keys
    uint32_t head;
    uint32_t bytes;     // bytes to copy in (nv rounded up to 16)
};

template <bool U16, bool CLB, bool CAUSAL>
__global__ void __launch_bounds__(kThreads) rows_cta_kernel(const int8_t *x_all, void *p_all, RowArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    // layout: [stage 0 | stage 1 | output stage], each Lk (output: Lk * element size) bytes
    uint8_t *in_stage[2] = {smem, smem + a.Lk};
    uint8_t *out_stage = smem + 2 * a.Lk;
    __shared__ __align__(8) uint64_t full_bar[2];
    __shared__ RowJob job[2];
    __shared__ int red[kThreads / 32];
    const int tid = threadIdx.x;
    const uint32_t bar[2] = {smem_u32(&full_bar[0]), smem_u32(&full_bar[1])};

    // thread 0: this CTA's next row (stride = grid size); start its copy into stage s
    int64_t next_row = blockIdx.x;
    auto fetch = [&](int s) {
        RowJob j;
        j.row = (int32_t)min(next_row, (int64_t)a.rows);
        next_row += gridDim.x;
        j.nv = 0; j.head = 0; j.bytes = 0;
        if (j.row >= a.rows) {
            j.row = -1;
        } else {
            uint32_t b, qi;
            row_coords((uint32_t)j.row, a, b, j.head, qi);
            j.nv = valid_keys<CAUSAL>(b, qi, a);
            j.bytes = (uint32_t)((j.nv + 15) & ~15);
            if (j.bytes) {
                mbar_expect_tx(bar[s], j.bytes);
                bulk_load(smem_u32(in_stage[s]), x_all + (int64_t)j.row * a.Lk, j.bytes, bar[s]);
            }
        }
        job[s] = j;
    };

    if (tid == 0) {
        mbar_init(bar[0], 1);
        mbar_init(bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        fetch(0);
    }
    __syncthreads();

    uint32_t phase[2] = {0, 0};
    const int osz = U16 ? 2 : 1;
    for (int it = 0;; ++it) {
        const int s = it & 1;
        // stage s^1 was consumed in the previous iteration (all threads passed its last barrier)
        if (tid == 0) fetch(s ^ 1);
        const RowJob j = job[s];
        if (j.row < 0) break;
        bool ok = true;
        if (j.bytes) {
            ok = mbar_wait_bounded(bar[s], phase[s], a.wait_cycles);
            phase[s] ^= 1;
        }
        if (!__syncthreads_and(ok)) {                 // uniform decision: give up together
            if (tid == 0) {
                atomicOr(a.status, STATUS_ROW_TMA_TIMEOUT);
                // shared memory must outlive the copies in flight: this stage's and the one started for
                // the other stage get the full default limit to land, whatever limit the wait above had
                (void)mbar_wait_bounded(bar[s], phase[s] ^ 1, kDefaultWaitCycles);
                if (job[s ^ 1].row >= 0 && job[s ^ 1].bytes)
                    (void)mbar_wait_bounded(bar[s ^ 1], phase[s ^ 1], kDefaultWaitCycles);
            }
            break;
        }
        const HeadEntry th = a.table[j.head];
        const uint8_t *xin = in_stage[s];
        const int nvec = (int)(j.bytes >> 4);         // 16-byte vectors that hold valid keys

        // ---- pass 1: row max
        uint32_t M = 0x80008000u;
        for (int v = tid; v < nvec; v += kThreads) {
            const uint4 w4 = *reinterpret_cast<const uint4 *>(xin + 16 * v);
            uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (CAUSAL) {
                    const uint32_t bm = byte_prefix_mask(j.nv - 16 * v - 4 * k);
                    w[k] = (w[k] & bm) | (0x80808080u & ~bm);
                }
                M = __vmaxs2(M, __vmaxs2(prmt(w[k], 0, 0xA280u), prmt(w[k], 0, 0xB391u)));
            }
        }
        const int m = block_reduce(max((int)(short)(M & 0xffffu), (int)M >> 16), true, red);

        // ---- pass 2: sum of the closeness values r = max(x + (D - m), 0) over the valid keys
        const int cm = th.D - m;
        const uint32_t c2 = prmt((uint32_t)cm, 0, 0x1010u);
        uint32_t rsum2 = 0;
        for (int v = tid; v < nvec; v += kThreads) {
            const uint4 w4 = *reinterpret_cast<const uint4 *>(xin + 16 * v);
            uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t ev = __viaddmax_s16x2(prmt(w[k], 0, 0xA280u), c2, 0u);
                uint32_t od = __viaddmax_s16x2(prmt(w[k], 0, 0xB391u), c2, 0u);
                if (CAUSAL) {
                    const uint32_t bm = byte_prefix_mask(j.nv - 16 * v - 4 * k);
                    ev &= prmt(bm, 0, 0x2200u);       // 16-bit lane masks of bytes 0,2 / 1,3
                    od &= prmt(bm, 0, 0x3311u);
                }
                rsum2 += ev + od;                     // at most 8 vectors per thread: no overflow
            }
        }
        const int rsum = block_reduce((int)(rsum2 & 0xffffu) + (int)(rsum2 >> 16), false, red);
        const int F = th.B - th.S * th.D;
        const uint32_t Z = (uint32_t)(j.nv * F + th.S * rsum);
        const uint32_t rho = reciprocal<U16, CLB>(max(Z, 1u));

        // ---- the output stage may still be read by the previous row's bulk store
        if (tid == 0) bulk_store_wait_read();
        __syncthreads();

        // ---- pass 3: normalise into the output stage
        const int total_vec = a.Lk >> 4;
        if (U16) {
            const uint32_t a1 = (uint32_t)F * rho * 0x00010001u, b1 = (uint32_t)th.S * rho;
            for (int v = tid; v < total_vec; v += kThreads) {
                uint32_t o[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                if (v < nvec) {
                    const uint4 w4 = *reinterpret_cast<const uint4 *>(xin + 16 * v);
                    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t pe = __viaddmax_s16x2(prmt(w[k], 0, 0xA280u), c2, 0u) * b1 + a1;
                        const uint32_t po = __viaddmax_s16x2(prmt(w[k], 0, 0xB391u), c2, 0u) * b1 + a1;
                        uint32_t q0 = prmt(pe, po, 0x5410u), q1 = prmt(pe, po, 0x7632u);
                        if (CAUSAL) {
                            const uint32_t bm = byte_prefix_mask(j.nv - 16 * v - 4 * k);
                            q0 &= prmt(bm, 0, 0x1100u);
                            q1 &= prmt(bm, 0, 0x3322u);
                        }
                        o[2 * k] = q0;
                        o[2 * k + 1] = q1;
                    }
                }
                uint4 *dst = reinterpret_cast<uint4 *>(out_stage + 32 * v);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        } else if (a.out_shift <= 1) {
            // the same pair arithmetic as the register-resident kernel: X = s * rho' < 2^24, coefficients split
            // at 8 bits so that every partial result fits a 16-bit lane
            const uint32_t rp = CLB ? (rho >> a.out_shift) : (rho << (1 - a.out_shift));
            const uint32_t a1 = (uint32_t)F * rp, b1 = (uint32_t)th.S * rp;
            const uint32_t ah2 = (a1 >> 8) * 0x00010001u, al2 = (a1 & 255u) * 0x00010001u;
            const uint32_t bh = b1 >> 8, bl = b1 & 255u;
            for (int v = tid; v < total_vec; v += kThreads) {
                uint32_t o[4] = {0, 0, 0, 0};
                if (v < nvec) {
                    const uint4 w4 = *reinterpret_cast<const uint4 *>(xin + 16 * v);
                    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t ev = __viaddmax_s16x2(prmt(w[k], 0, 0xA280u), c2, 0u);
                        const uint32_t od = __viaddmax_s16x2(prmt(w[k], 0, 0xB391u), c2, 0u);
                        uint32_t q;
                        if (!CLB) {
                            const uint32_t ye = ev * bh + ah2 + prmt(ev * bl + al2, 0, 0x4341u);
                            const uint32_t yo = od * bh + ah2 + prmt(od * bl + al2, 0, 0x4341u);
                            q = prmt(ye, yo, 0x7351u);
                        } else {
                            const uint32_t ye = __viaddmin_u16x2(ev * bh + ah2, prmt(ev * bl + al2, 0, 0x4341u), 0x7fff7fffu);
                            const uint32_t yo = __viaddmin_u16x2(od * bh + ah2, prmt(od * bl + al2, 0, 0x4341u), 0x7fff7fffu);
                            q = prmt(ye * 2u, yo * 2u, 0x7351u);
                        }
                        if (CAUSAL) q &= byte_prefix_mask(j.nv - 16 * v - 4 * k);
                        o[k] = q;
                    }
                }
                *reinterpret_cast<uint4 *>(out_stage + 16 * v) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        } else {
            // OUT_SHIFT >= 2: the result is not byte-aligned in the product; shift each element
            const uint32_t a1 = (uint32_t)F * rho, b1 = (uint32_t)th.S * rho;
            const int sh = 15 + a.out_shift;
            for (int v = tid; v < total_vec; v += kThreads) {
                uint32_t o[4] = {0, 0, 0, 0};
                if (v < nvec) {
                    const uint4 w4 = *reinterpret_cast<const uint4 *>(xin + 16 * v);
                    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t ev = __viaddmax_s16x2(prmt(w[k], 0, 0xA280u), c2, 0u);
                        const uint32_t od = __viaddmax_s16x2(prmt(w[k], 0, 0xB391u), c2, 0u);
                        const uint32_t x0 = min((a1 + b1 * (ev & 0xffffu)) >> sh, 255u);
                        const uint32_t x1 = min((a1 + b1 * (od & 0xffffu)) >> sh, 255u);
                        const uint32_t x2 = min((a1 + b1 * (ev >> 16)) >> sh, 255u);
                        const uint32_t x3 = min((a1 + b1 * (od >> 16)) >> sh, 255u);
                        uint32_t q = x0 | (x1 << 8) | (x2 << 16) | (x3 << 24);
                        if (CAUSAL) q &= byte_prefix_mask(j.nv - 16 * v - 4 * k);
                        o[k] = q;
                    }
                }
                *reinterpret_cast<uint4 *>(out_stage + 16 * v) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        // make the generic-proxy writes visible to the bulk store, then hand the row over
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0)
            bulk_store((uint8_t *)p_all + (int64_t)j.row * a.Lk * osz, smem_u32(out_stage),
                       (uint32_t)(a.Lk * osz));
    }
    if (tid == 0) bulk_store_wait_all();   // shared memory must outlive the last store
}

template <bool U16, bool CLB, bool CAUSAL>
cudaError_t launch_cta(const int8_t *x, void *p, const RowArgs &a, cudaStream_t st) {
    const size_t smem = (size_t)a.Lk * (U16 ? 4 : 3);
    auto kernel = rows_cta_kernel<U16, CLB, CAUSAL>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int ctas_per_sm = (int)((200u * 1024u) / (smem + 1024));
    if (ctas_per_sm < 1) ctas_per_sm = 1;
    if (ctas_per_sm > 8) ctas_per_sm = 8;
    int64_t blocks = (int64_t)148 * ctas_per_sm;
    if (blocks > a.rows) blocks = a.rows;
    kernel<<<(unsigned)blocks, kThreads, smem, st>>>(x, p, a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t try_launch_cta(const int8_t *logits, void *probs, const RowArgs &a, uint32_t flags,
                           cudaStream_t stream, bool *taken) {
    *taken = false;
    if ((((uintptr_t)logits | (uintptr_t)probs) & 15u) != 0 || a.Lk % 16 != 0 || a.Lk < 256) return cudaSuccess;
    *taken = true;
    switch (flags & 7u) {
        case 0: return launch_cta<false, false, false>(logits, probs, a, stream);
        case 1: return launch_cta<true, false, false>(logits, probs, a, stream);
        case 2: return launch_cta<false, true, false>(logits, probs, a, stream);
        case 3: return launch_cta<true, true, false>(logits, probs, a, stream);
        case 4: return launch_cta<false, false, true>(logits, probs, a, stream);
        case 5: return launch_cta<true, false, true>(logits, probs, a, stream);
        case 6: return launch_cta<false, true, true>(logits, probs, a, stream);
        default: return launch_cta<true, true, true>(logits, probs, a, stream);
    }
}

}  // namespace hccs

// ------------------------------------------------------------------------------------------
// hccs_forward_static_scratch: the CTA-per-row kernel for callers that must not allocate.
// ------------------------------------------------------------------------------------------
// Everything the kernel needs besides the caller's tensors lives in this one file-scope device
// array, which every GPU that loads the library holds until the process exits:
//   word 0            status word (bounded waits report here)
//   from byte 256 on  the per-head parameter table, kStaticMaxHeads entries
namespace {

constexpr int kStaticMaxHeads = 256;
constexpr int kStaticTableOffsetWords = 64;
constexpr int kStaticWords = kStaticTableOffsetWords + kStaticMaxHeads * (int)(sizeof(hccs::HeadEntry) / 4);
static __device__ __align__(256) uint32_t g_static_scratch[kStaticWords];

// The table travels to the device as a kernel argument (4 KB by value): no host buffer has to stay alive
// and nothing is copied from pageable memory, so the call never blocks on earlier work of the stream.
struct StaticTable {
    hccs::HeadEntry entry[kStaticMaxHeads];
};
__global__ void static_scratch_fill_kernel(uint32_t *scratch, StaticTable table, int num_heads) {
    if (threadIdx.x == 0) scratch[0] = 0;                         // status word: starts at zero for every call
    hccs::HeadEntry *dst = reinterpret_cast<hccs::HeadEntry *>(scratch + kStaticTableOffsetWords);
    for (int h = threadIdx.x; h < num_heads; h += blockDim.x) dst[h] = table.entry[h];
}

constexpr int kStaticMaxDevices = 64;
uint32_t *g_static_ptr[kStaticMaxDevices] = {};   // device address of the array, per device
std::mutex g_static_mutex;

// The array's name is only a host-side handle; the address the kernel can use has to be asked
// for, once per device and with that device current.
cudaError_t static_scratch_address(int device, uint32_t **out) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[device] = static_cast<uint32_t *>(p);
    }
    *out = g_static_ptr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" hccs_status_t hccs_forward_static_scratch(const hccs_head_params_t *params, int32_t num_heads,
                                                     int32_t n_design, int32_t out_shift,
                                                     const int8_t *logits, void *probs, int32_t B,
                                                     int32_t H, int32_t Lq, int32_t Lk, uint32_t flags,
                                                     uint32_t *timed_out, void *cuda_stream) {
    if (timed_out) *timed_out = 0;
    if (B < 0 || H < 0 || Lq < 0 || Lk < 0 || (flags & ~7u)) return HCCS_ERR_INVALID_ARG;
    if (out_shift < 0 || out_shift > 8) return HCCS_ERR_INVALID_ARG;
    hccs_status_t st = hccs_params_check(params, num_heads, n_design, nullptr);
    if (st != HCCS_OK) return st;
    if (H != num_heads) return HCCS_ERR_INVALID_ARG;
    if (num_heads > kStaticMaxHeads) return HCCS_ERR_UNSUPPORTED;      // beyond the static table
    if (Lk > n_design) return HCCS_ERR_CONSTRAINT;
    const int64_t rows = (int64_t)B * H * Lq;
    if (rows >= (1ll << 31)) return HCCS_ERR_UNSUPPORTED;
    if (rows * Lk == 0) return HCCS_OK;
    if (!logits || !probs) return HCCS_ERR_INVALID_ARG;
    if (Lk % 16 != 0 || (((uintptr_t)logits | (uintptr_t)probs) & 15u) != 0) return HCCS_ERR_UNSUPPORTED;
    if ((flags & HCCS_OUT_U16) && (const void *)logits == probs) return HCCS_ERR_INVALID_ARG;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kStaticMaxDevices) {
        (void)cudaGetLastError();
        return HCCS_ERR_CUDA;
    }
    uint32_t *scratch = nullptr;
    if (static_scratch_address(device, &scratch) != cudaSuccess) {
        (void)cudaGetLastError();
        return HCCS_ERR_CUDA;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    // The array keeps whatever the previous call left: a one-CTA kernel on the caller's stream rewrites
    // the table and clears the status word before the row kernel runs.
    StaticTable table;
    for (int32_t h = 0; h < num_heads; ++h) {
        table.entry[h].B = params[h].B;
        table.entry[h].S = params[h].S;
        table.entry[h].D = params[h].Dmax;
        table.entry[h].pad = 0;
    }
    hccs::HeadEntry *d_table = reinterpret_cast<hccs::HeadEntry *>(scratch + kStaticTableOffsetWords);
    static_scratch_fill_kernel<<<1, 256, 0, stream>>>(scratch, table, num_heads);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return HCCS_ERR_CUDA;

    hccs::RowArgs a;
    a.table = d_table;
    a.status = scratch;
    a.wait_cycles = hccs::kDefaultWaitCycles;
    a.rows = (int32_t)rows;
    a.H = H;
    a.Lq = Lq;
    a.Lk = Lk;
    a.causal_off = Lk - Lq;
    a.causal = (flags & HCCS_CAUSAL) ? 1 : 0;
    a.key_len = nullptr;
    a.out_shift = out_shift;
    a.slice0 = 0;
    a.div_Lq = hccs::make_fastdiv((uint32_t)Lq);
    a.div_H = hccs::make_fastdiv((uint32_t)H);
    switch (flags & 7u) {
        case 0: e = hccs::launch_cta<false, false, false>(logits, probs, a, stream); break;
        case 1: e = hccs::launch_cta<true, false, false>(logits, probs, a, stream); break;
        case 2: e = hccs::launch_cta<false, true, false>(logits, probs, a, stream); break;
        case 3: e = hccs::launch_cta<true, true, false>(logits, probs, a, stream); break;
        case 4: e = hccs::launch_cta<false, false, true>(logits, probs, a, stream); break;
        case 5: e = hccs::launch_cta<true, false, true>(logits, probs, a, stream); break;
        case 6: e = hccs::launch_cta<false, true, true>(logits, probs, a, stream); break;
        default: e = hccs::launch_cta<true, true, true>(logits, probs, a, stream); break;
    }
    if (e != cudaSuccess) { (void)cudaGetLastError(); return HCCS_ERR_CUDA; }
    if (timed_out) {
        e = cudaMemcpyAsync(timed_out, scratch, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return HCCS_ERR_CUDA; }
        if (*timed_out) return HCCS_ERR_DEVICE_TIMEOUT;
    }
    return HCCS_OK;
}

// ------------------------------------------------------------------------------------------
// Wait-limit probe: the give-up path of the bounded waits, exercised without any copy in flight.
// ------------------------------------------------------------------------------------------
namespace hccs {

namespace {

// One CTA of two warps.  Thread 0 initialises an mbarrier that expects one arrival which never comes and
// waits on it through the helper the production kernels use, with the caller's limit; the wait runs out,
// the status bit is set and the kernel returns.  In mode 1 a thread of the second warp waits through the
// abortable helper as well, with a limit sixteen times longer: it leaves because it sees the abort flag.
__global__ void wait_probe_kernel(uint32_t *status, int mode, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar_word;
    __shared__ int abort_flag;
    const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&bar_word);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int *abortp = &abort_flag;
    if (mode == 0) {
        if (threadIdx.x == 0 && !mbar_wait_bounded(bar, 0, limit_cycles)) atomicOr(status, STATUS_ROW_TMA_TIMEOUT);
    } else {
        if (threadIdx.x == 0) (void)mbar_wait_abortable(bar, 0, abortp, status, STATUS_FUSED_TIMEOUT, limit_cycles);
        if (threadIdx.x == 32) (void)mbar_wait_abortable(bar, 0, abortp, status, STATUS_FUSED_TIMEOUT, limit_cycles * 16);
    }
}

}  // namespace

cudaError_t launch_wait_probe(uint32_t *status, int mode, long long limit_cycles, cudaStream_t stream) {
    wait_probe_kernel<<<1, 64, 0, stream>>>(status, mode, limit_cycles);
    return cudaGetLastError();
}

}  // namespace hccs
