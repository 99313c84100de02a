// Fused int8 attention for one (batch, head, 128-query tile) per CTA:
//     S = Q.K^T (int32)  ->  x = requantise(S) (int8)  ->  P = HCCS(x) (uint8)  ->  O = P.V (int32)
// The two contractions run on the 5th-generation tensor cores (tcgen05.mma kind::i8, operands in
// shared memory staged by TMA, accumulators in tensor memory); the softmax surrogate itself is
// plain integer ALU work (Algorithm 1 of the paper) done by the thread that owns the row.
//
// Why it is organised this way:
//   * HCCS needs the whole row before it can normalise (the clamp makes the usual online
//     rescaling of exp-softmax impossible), so the CTA keeps the full 128 x L int8 logit panel in
//     shared memory (128 KB at L = 1024).  The panel is laid out as the K-major, 128-byte-swizzled
//     operand the second contraction wants, so P is produced in place and never moves.
//   * tcgen05.ld with the 32x32b shape gives thread t of the four row warps TMEM lane t, i.e. one
//     query row with all its keys: max, sum, reciprocal and normalisation need no cross-thread
//     reduction at all.
//   * K tiles are consumed during the first contraction only and V tiles during the second, so V
//     is loaded into the buffer K occupied, while the row warps do the HCCS passes.
//   * V is used as stored ([key][64], keys outermost): that is exactly the MN-major, 64-byte
//     swizzled B operand, so no transposition is needed.
//
// Warp roles (672 threads): warps 0-15 are row warps, four threads per query row (threads t,
// t + 128, t + 256, t + 384 own row t mod 128; TMEM lane quarter = warp index mod 4): bits 7-8
// of the thread index select which 32 of the 128 keys of every block the thread handles, so all
// row threads work on the same block while the tensor core fills the other S buffers.
// The four exchange their partial row max and row sum through shared memory; the many warps are
// what hides the latency of the dependent integer chains.  Five more warps each run one
// single-lane role: warps 16 and 20 issue the TMA loads (alternate blocks), warps 17 and 19
// the first contraction (alternate blocks), warp 18 the second (one thread doing it all fell
// behind the row warps: its serial chain of waits, descriptor arithmetic and issues cost several
// hundred cycles per block).
// All mbarrier waits are bounded; a wait that runs
// out sets STATUS_FUSED_TIMEOUT, raises an abort flag that every other wait observes, and the CTA
// leaves through the common exit, which frees its tensor memory.  No clusters, no multicast.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hccs_device.cuh"
#include "hccs_internal.h"

namespace hccs {

namespace {

constexpr int kRowThreads = 512;           // four per query row
constexpr int kThreads = 672;            // 16 row warps and five single-lane role warps
constexpr int kTmaWarp = 16, kQkWarp = 17, kPvWarp = 18, kQk2Warp = 19, kTma2Warp = 20;
constexpr int kHalf = 64;                 // operand rows are staged 64 bytes at a time (64-byte swizzle): d = 64 is one
                                          // such half tile per Q, K or V tile, d = 128 two
constexpr int kTile = 128;                // queries per CTA, keys per block
constexpr int kHalfBytes = kTile * kHalf;  // 8 KB: 128 rows x 64 bytes
constexpr int kPanelBlockBytes = kTile * 128;   // 16 KB: 128 rows x 128 keys of the panel
constexpr int kMaxBlocks = 8;             // L <= 1024
constexpr uint32_t kTmemCols = 512;       // S0 [0,128)  S1 [128,256)  S2 [256,384)  O [384,448)
constexpr int kSBufs = 3;                 // S blocks in flight between the tensor core and the row warps
constexpr uint32_t kTmemO = 384;
constexpr uint32_t kOBoxBytes = 128 * 128; // one staged box of the output tile: 128 rows x 32 int32 columns

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint64_t make_u64(uint32_t lo, uint32_t hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}
__device__ __forceinline__ int64_t mad_wide_s32(int32_t a, int32_t b, int64_t c) {
    int64_t d;
    asm("mad.wide.s32 %0, %1, %2, %3;" : "=l"(d) : "r"(a), "r"(b), "l"(c));
    return d;
}
// d = { sat8(b), sat8(a), c.lo16 } from low byte up: two signed 32-bit values clamped to int8 and
// packed below the low half of c.
__device__ __forceinline__ uint32_t cvt_pack_s8(int32_t a, int32_t b, uint32_t c) {
    uint32_t d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded, abort-aware wait.  Returns false when the wait was given up (here or elsewhere).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          uint32_t *status, long long limit_cycles) {
    return mbar_wait_abortable(bar, parity, abort_flag, status, STATUS_FUSED_TIMEOUT, limit_cycles);
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
// Tiled store of one shared-memory box to a 3-D tensor (rows past the tensor's extent are dropped).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, int x, int y, int z, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];" ::"l"(map),
                 "r"(x), "r"(y), "r"(z), "r"(src)
                 : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], int8 operands, int32 accumulator.
__device__ __forceinline__ void tcgen05_mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// (load and wait in one statement: no use of the registers can be scheduled between the two)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// ---------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor: start address, leading/stride byte offsets (all >> 4), the
// Blackwell version field (1 at bit 46) and the swizzle mode in bits [61,64).
constexpr uint64_t kSwizzle128 = 2, kSwizzle64 = 4;
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t swizzle) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46) | (swizzle << 61);
}
// Instruction descriptor of kind::i8: D = int32 (2 at bit 4), operand formats at bits 7 and 10
// (0 = uint8, 1 = int8), B MN-major flag at bit 16, N >> 3 at bit 17, M >> 4 at bit 24.
constexpr uint32_t instr_desc(uint32_t a_signed, uint32_t b_signed, uint32_t b_mn_major, uint32_t M, uint32_t N) {
    return (2u << 4) | (a_signed << 7) | (b_signed << 10) | (b_mn_major << 16) | ((N >> 3) << 17) | ((M >> 4) << 24);
}
constexpr uint32_t kIdescQK = instr_desc(1, 1, 0, 128, 128);   // S = Q.K^T : int8 x int8, both K-major
constexpr uint32_t kIdescPV = instr_desc(0, 1, 1, 128, 64);    // O = P.V   : uint8 x int8, V MN-major

struct FusedSmemBarriers {
    uint64_t q_full;
    uint64_t k_full[kMaxBlocks];
    uint64_t k_done;        // every MMA of the first contraction has finished reading K
    uint64_t v_full[kMaxBlocks];
    uint64_t s_full[kSBufs];
    uint64_t s_free[kSBufs];
    uint64_t p_ready[kMaxBlocks];   // block kb of the probability panel is complete
    uint64_t o_full;
    uint64_t ring_full[4];          // ring mode: the copy into slot s has landed
    uint64_t ring_free[4];          // ring mode: every MMA that reads slot s has completed
};

// RING (d = 128 with more than 512 keys): K, V and the panel no longer fit the SM together, so the K blocks of
// the first round, the K blocks of the second round and the V blocks of a tile stream, in that order, through
// a ring of four 16 KB slots.  Load number j (counted over all tiles of the CTA) uses slot j % 4 for the
// (j / 4)-th time; every role derives slot and phase parities from j alone.  A slot is handed back by a
// tcgen05.commit behind the MMAs that read it.
constexpr int kRingSlots = 4;

template <int D, bool CLB, bool CAUSAL, bool RING = false>
__global__ void __launch_bounds__(kThreads, 1)
fused_attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o,
                       FusedArgs a, int num_tiles) {
    constexpr int kHalves = D / kHalf;                    // half tiles per Q, K or V tile
    constexpr int kTileBytes = kTile * D;                 // one Q, K or V tile: 8 or 16 KB
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) FusedSmemBarriers bars;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag, leave_flag;
    __shared__ int part_max[4][kTile], part_sum[4][kTile];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nblk = (a.L + kTile - 1) / kTile;           // key blocks (and query tiles) per head
    const bool causal = (a.flags & HCCS_CAUSAL) != 0;
    volatile int *abortp = &abort_flag;
    const bool two_rounds = a.requant_shift <= 24;        // see the row warps' scan flow

    // shared-memory carve-up (1024-byte aligned: required by the swizzled layouts)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t s_q = base;                                            // Q tile
    const uint32_t s_kpre = s_q + kTileBytes;                             // K blocks 0 and 1 (prefetched)
    const uint32_t s_kv = s_kpre + 2 * kTileBytes;                        // K blocks 2.., later all V blocks
    const uint32_t s_ring = s_q + kTileBytes;                             // ring mode: the four K / V slots
    const uint32_t s_p = RING ? s_ring + kRingSlots * kTileBytes : s_kv + (uint32_t)nblk * kTileBytes;   // logit / probability panel
    uint8_t *panel = gen_base + (RING ? (1 + kRingSlots) * kTileBytes : 3 * kTileBytes + (size_t)nblk * kTileBytes);
    const int ring_stages = (two_rounds ? 2 : 1) + 1;    // K once per round of the first contraction, then V
    auto k_slot = [&](int kb) { return kb < 2 ? s_kpre + kb * kTileBytes : s_kv + kb * kTileBytes; };

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bars.q_full), 1);
        for (int i = 0; i < kMaxBlocks; ++i) mbar_init(smem_u32(&bars.k_full[i]), 1);
        mbar_init(smem_u32(&bars.k_done), 2);
        for (int i = 0; i < kMaxBlocks; ++i) mbar_init(smem_u32(&bars.v_full[i]), 1);
        for (int i = 0; i < kSBufs; ++i) {
            mbar_init(smem_u32(&bars.s_full[i]), 1);
            mbar_init(smem_u32(&bars.s_free[i]), kRowThreads);
        }
        for (int i = 0; i < kMaxBlocks; ++i) mbar_init(smem_u32(&bars.p_ready[i]), kRowThreads);
        mbar_init(smem_u32(&bars.o_full), 1);
        for (int i = 0; i < kRingSlots; ++i) {
            mbar_init(smem_u32(&bars.ring_full[i]), 1);
            mbar_init(smem_u32(&bars.ring_free[i]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kTmaWarp) {   // one warp allocates the tensor memory for the CTA
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = tmem_base_slot;

    // Key blocks a tile goes through: all of the head's, or only those that hold a valid key for some row
    // of the tile (causal rule, per-batch key length); at least one, so that O is written.
    auto blocks_at = [&](int qt_, int batch_) -> int {      // query tile qt_ of a head of batch entry batch_
        int n = nblk;
        if (CAUSAL) {
            if (causal) n = qt_ + 1;
            if (a.key_len) {
                const int kl = min(max(a.key_len[batch_], 0), a.L);
                n = min(n, max((kl + kTile - 1) / kTile, 1));
            }
        }
        return n;
    };
    auto blocks_of = [&](int tile) -> int { return CAUSAL ? blocks_at(tile % nblk, tile / nblk / a.H) : nblk; };
    // A CTA walks over the tiles blockIdx.x, blockIdx.x + gridDim.x, ...  Every mbarrier completes
    // one phase per use, so both sides count their uses (per barrier, because a causal tile uses
    // only its first qt + 1 key blocks) and wait on the parity of that count.
    if (warp == kTmaWarp || warp == kTma2Warp) {
        // ===================================================== copy threads: every TMA load.  A thread gets
        // through one copy per ~600 cycles whatever its size, copies of different warps overlap: the
        // first thread takes Q and the even K and V blocks, the second the odd ones.
        if (lane == 0) {
            const int me = warp == kTmaWarp ? 0 : 1;
            bool ok = true;
            // Q and the first two K blocks of a tile go to buffers of their own, so they can be
            // fetched while the previous tile is still in its softmax passes.
            // one Q, K or V tile: its 64-byte column halves land one after the other
            auto load_tile = [&](uint32_t dst, const CUtensorMap *map, int row, uint32_t bar) {
                mbar_expect_tx(bar, kTileBytes);
#pragma unroll
                for (int h = 0; h < kHalves; ++h) tma_load_2d(dst + h * kHalfBytes, map, h * kHalf, row, bar);
            };
            auto prefetch = [&](int tile) {
                const int bh = tile / nblk, qt = tile % nblk;
                const int kblocks = blocks_of(tile);
                load_tile(s_q, &map_q, bh * a.L + qt * kTile, smem_u32(&bars.q_full));
                for (int kb = 0; kb < min(2, kblocks); ++kb) {
                    load_tile(k_slot(kb), &map_k, bh * a.L + kb * kTile, smem_u32(&bars.k_full[kb]));
                }
            };
            if constexpr (RING) {
                // loads in ring order; this thread takes the even or the odd ones (slots 0, 2 or 1, 3)
                uint32_t base_j = 0;
                for (int tile = blockIdx.x, it = 0; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                    const int bh = tile / nblk, qt = tile % nblk;
                    const int kblocks = blocks_of(tile);
                    if (me == 0) {
                        // Q is read by both rounds of the first contraction: the previous tile's must be complete
                        if (it > 0) ok = mbar_wait(smem_u32(&bars.k_done), (it - 1) & 1, abortp, a.status, a.wait_cycles);
                        if (!ok) break;
                        load_tile(s_q, &map_q, bh * a.L + qt * kTile, smem_u32(&bars.q_full));
                    }
                    for (int st = 0; ok && st < ring_stages; ++st) {
                        for (int kb = 0; kb < kblocks; ++kb) {
                            const uint32_t j = base_j + (uint32_t)(st * kblocks + kb);
                            if ((int)(j & 1u) != me) continue;
                            const uint32_t slot = j % kRingSlots, use = j / kRingSlots;
                            if (use > 0) ok = mbar_wait(smem_u32(&bars.ring_free[slot]), (use - 1) & 1, abortp, a.status, a.wait_cycles);
                            if (!ok) break;
                            load_tile(s_ring + slot * kTileBytes, st + 1 < ring_stages ? &map_k : &map_v, bh * a.L + kb * kTile,
                                      smem_u32(&bars.ring_full[slot]));
                        }
                    }
                    base_j += (uint32_t)(ring_stages * kblocks);
                }
            } else {
            if (me == 0 && (int)blockIdx.x < num_tiles) prefetch(blockIdx.x);
            for (int tile = blockIdx.x, it = 0; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                const int bh = tile / nblk;
                const int kblocks = blocks_of(tile);
                // the other K blocks land where the previous tile's V sits: wait for its last MMA
                if (it > 0) ok = mbar_wait(smem_u32(&bars.o_full), (it - 1) & 1, abortp, a.status, a.wait_cycles);
                if (!ok) break;
                for (int kb = 2 + me; kb < kblocks; kb += 2) {
                    load_tile(k_slot(kb), &map_k, bh * a.L + kb * kTile, smem_u32(&bars.k_full[kb]));
                }
                // V takes the K buffer once the first contraction has read the last K block; Q and
                // the first K blocks of the next tile are fetched as well
                ok = mbar_wait(smem_u32(&bars.k_done), it & 1, abortp, a.status, a.wait_cycles);
                if (!ok) break;
                // (the next tile's Q and K go after the first V block, early enough for its first round
                // to start behind the probability pass)
                for (int kb = me; kb < kblocks; kb += 2) {
                    load_tile(s_kv + kb * kTileBytes, &map_v, bh * a.L + kb * kTile, smem_u32(&bars.v_full[kb]));
                    if (kb == 0 && tile + (int)gridDim.x < num_tiles) prefetch(tile + gridDim.x);
                }
            }
            }   // resident K and V
        }
    } else if (warp == kQkWarp || warp == kQk2Warp) {
        // ===================================================== first contraction: S = Q . K^T, block by block.
        // Two issuers take the blocks alternately: what one thread spends per block (two waits, the
        // descriptors, two MMAs, the commit) is more than the tensor core needs for it.
        if (lane == 0) {
            const uint32_t me = warp == kQkWarp ? 0u : 1u;
            bool ok = true;
            uint32_t k_par = 0;                          // bit kb = parity of this tile's phase of k_full[kb]
            uint32_t g = 0;                              // blocks issued so far by both issuers
            uint32_t s_buf = 0, s_cyc = 0;               // = g % kSBufs, g / kSBufs: S buffer of block g and its use
            uint32_t ring_base = 0;                      // ring mode: load number of this tile's first block
            // descriptors differ only in the start address field (address >> 4): low word + offset
            const uint64_t dq = smem_desc(s_q, 16, 512, kSwizzle64);
            const uint64_t dk = smem_desc(s_kpre, 16, 512, kSwizzle64);
            const uint32_t dq_lo = (uint32_t)dq, dq_hi = (uint32_t)(dq >> 32);
            const uint32_t dk_lo = (uint32_t)dk, dk_hi = (uint32_t)(dk >> 32);
            for (int tile = blockIdx.x, it = 0; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                const int kblocks = blocks_of(tile);
                ok = mbar_wait(smem_u32(&bars.q_full), it & 1, abortp, a.status, a.wait_cycles);
                // the scan flow of the row warps reads every S block twice: once for the row maximum,
                // once to requantise
                for (int round = 0; ok && round < (two_rounds ? 2 : 1); ++round) {
#pragma unroll
                    for (int kb = 0; kb < kMaxBlocks; ++kb) {
                        if (kb >= kblocks || !ok) break;
                        const uint32_t sb = s_buf, cyc = s_cyc;
                        const bool mine = (g & 1u) == me;
                        ++g;
                        if (++s_buf == kSBufs) { s_buf = 0; ++s_cyc; }
                        if (!mine) continue;
                        if (cyc > 0) ok = mbar_wait(smem_u32(&bars.s_free[sb]), (cyc - 1) & 1, abortp, a.status, a.wait_cycles);
                        // the K block's copy must have landed: in the second round too, where the
                        // block may fall to the issuer that did not wait for it in the first
                        uint32_t koff;                        // the K block's distance from s_kpre, in 16-byte units
                        uint32_t ring_slot = 0;
                        if constexpr (RING) {
                            const uint32_t j = ring_base + (uint32_t)(round * kblocks + kb);
                            ring_slot = j % kRingSlots;
                            if (ok) ok = mbar_wait(smem_u32(&bars.ring_full[ring_slot]), (j / kRingSlots) & 1, abortp, a.status, a.wait_cycles);
                            koff = (ring_slot * kTileBytes) >> 4;          // s_ring is where s_kpre is
                        } else {
                            if (ok) ok = mbar_wait(smem_u32(&bars.k_full[kb]), (k_par >> kb) & 1, abortp, a.status, a.wait_cycles);
                            // K block kb sits (kb < 2 ? kb : kb + 2) tiles above the first prefetch slot
                            koff = (uint32_t)((kb < 2 ? kb : kb + 2) * kTileBytes) >> 4;
                        }
                        if (!ok) break;
                        tcgen05_fence_after();
                        // two k-steps of 32 per 64-byte half of d
#pragma unroll
                        for (int h = 0; h < kHalves; ++h)
#pragma unroll
                            for (int ks = 0; ks < 2; ++ks) {
                                const uint32_t off = (uint32_t)(h * kHalfBytes + ks * 32) >> 4;
                                tcgen05_mma_i8(tmem + sb * 128, make_u64(dq_lo + off, dq_hi), make_u64(dk_lo + koff + off, dk_hi),
                                               kIdescQK, (h | ks) != 0);
                            }
                        tcgen05_commit(smem_u32(&bars.s_full[sb]));
                        if constexpr (RING) tcgen05_commit(smem_u32(&bars.ring_free[ring_slot]));   // the slot goes back
                    }
                }
                if (!ok) break;
                k_par ^= (1u << kblocks) - 1u;               // every k_full[kb < kblocks] completed one phase
                ring_base += (uint32_t)(ring_stages * kblocks);
                tcgen05_commit(smem_u32(&bars.k_done));      // both issuers: the barrier counts two
            }
        }
    } else if (warp == kPvWarp) {
        // ===================================================== second contraction: O += P_kb . V_kb as the
        // row warps finish the probability blocks; four k-steps of 32 keys per block
        if (lane == 0) {
            bool ok = true;
            uint32_t p_par = 0;                          // bit kb = parity of the next use of p_ready[kb] and v_full[kb]
            uint32_t ring_base = 0;                      // ring mode: load number of this tile's first block
            const uint64_t dp = smem_desc(s_p, 16, 1024, kSwizzle128);
            const uint64_t dv = smem_desc(RING ? s_ring : s_kv, 512, 512, kSwizzle64);
            const uint32_t dp_lo = (uint32_t)dp, dp_hi = (uint32_t)(dp >> 32);
            const uint32_t dv_lo = (uint32_t)dv, dv_hi = (uint32_t)(dv >> 32);
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int kblocks = blocks_of(tile);
#pragma unroll
                for (int kb = 0; kb < kMaxBlocks; ++kb) {
                    if (kb >= kblocks) break;
                    uint32_t vbase = (uint32_t)(kb * kTileBytes) >> 4;     // the V block's distance from the descriptor's base, in 16-byte units
                    uint32_t ring_slot = 0;
                    if constexpr (RING) {
                        const uint32_t j = ring_base + (uint32_t)((ring_stages - 1) * kblocks + kb);
                        ring_slot = j % kRingSlots;
                        ok = mbar_wait(smem_u32(&bars.ring_full[ring_slot]), (j / kRingSlots) & 1, abortp, a.status, a.wait_cycles);
                        vbase = (ring_slot * kTileBytes) >> 4;
                    } else {
                        ok = mbar_wait(smem_u32(&bars.v_full[kb]), (p_par >> kb) & 1, abortp, a.status, a.wait_cycles);
                    }
                    if (ok) ok = mbar_wait(smem_u32(&bars.p_ready[kb]), (p_par >> kb) & 1, abortp, a.status, a.wait_cycles);
                    if (!ok) break;
                    p_par ^= 1u << kb;
                    tcgen05_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint32_t poff = (uint32_t)(kb * kPanelBlockBytes + ks * 32) >> 4;
#pragma unroll
                        for (int h = 0; h < kHalves; ++h) {      // 64 output columns per half tile of V
                            const uint32_t voff = vbase + ((uint32_t)(h * kHalfBytes + ks * 32 * kHalf) >> 4);
                            tcgen05_mma_i8(tmem + kTmemO + h * kHalf, make_u64(dp_lo + poff, dp_hi), make_u64(dv_lo + voff, dv_hi),
                                           kIdescPV, (kb | ks) != 0);
                        }
                    }
                    if constexpr (RING) tcgen05_commit(smem_u32(&bars.ring_free[ring_slot]));   // the slot goes back
                }
                if (!ok) break;
                ring_base += (uint32_t)(ring_stages * kblocks);
                tcgen05_commit(smem_u32(&bars.o_full));
            }
        }
    } else {
        // ===================================================== row warps: threads t, t+128, t+256, t+384 own query row t
        const int t = tid & (kTile - 1);                     // TMEM lane = row of the tile
        const int grp = tid >> 7;                            // 0..3: keys 32*grp .. 32*grp+31 of every block
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint8_t *row_base = panel + (t >> 3) * 1024 + (t & 7) * 128;
        const int swz = t & 7;
        uint32_t s_buf = 0, s_cyc = 0;                       // S buffer of the next block and its use count
        bool ok = true;
        // one S block of the first round: the running maximum of the row's raw accumulators
        auto first_round_block = [&](int kb, int nv_row, int &amax) {
            const uint32_t sb = s_buf;
            ok = mbar_wait(smem_u32(&bars.s_full[sb]), s_cyc & 1, abortp, a.status, a.wait_cycles);
            if (!ok) return;
            if (++s_buf == kSBufs) { s_buf = 0; ++s_cyc; }
            tcgen05_fence_after();
            uint32_t acc[32];
            tmem_ld32(tmem + lane_addr + sb * 128 + grp * 32, acc);
            tcgen05_fence_before();                      // the accumulators are in registers: the buffer goes back now
            mbar_arrive(smem_u32(&bars.s_free[sb]));
            const int c0 = kb * kTile + grp * 32;
            if (CAUSAL && c0 + 32 > nv_row) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (c0 + e >= nv_row) acc[e] = (uint32_t)(-(1 << 30));
            }
#pragma unroll
            for (int e = 0; e < 32; e += 2) amax = __vimax3_s32(amax, (int)acc[e], (int)acc[e + 1]);
        };
        int amax_carry = -(1 << 30), r1_carry = 0;           // first-round blocks of a tile taken ahead of it
        // number of valid keys (always a prefix) of this thread's row in a tile of batch entry batch_ that
        // starts at query q0_
        auto valid_keys = [&](int batch_, int q0_) -> int {
            int n = a.L;
            if (CAUSAL) {
                if (causal) n = min(q0_ + t + 1, n);
                if (a.key_len) n = min(n, max(a.key_len[batch_], 0));
            }
            return n;
        };
        // Where a tile is and the constants of its head.  Both are kept one tile ahead: the position advances
        // by additions (no division per tile), and the head's constants are loaded while the previous tile is
        // in its last phases -- at the top of a tile their latency (a trip to L2 behind two divisions) stood
        // in front of every row warp at once.
        struct TileAt { int bh, qt, head, batch; };
        struct HeadConsts { int4 th, rq, rx; };   // {B, S, D, -}, {M << k, C << k, -lo, hi - lo}, {out scale, out multiplier, 1/M (double)}
        const int step_qt = (int)gridDim.x % nblk, step_bh = (int)gridDim.x / nblk;
        const int step_head = step_bh % a.H, step_batch = step_bh / a.H;
        auto advance = [&](TileAt p) -> TileAt {
            p.qt += step_qt;
            const int carry = p.qt >= nblk ? 1 : 0;
            p.qt -= carry ? nblk : 0;
            p.bh += step_bh + carry;
            p.head += step_head + carry;
            p.batch += step_batch;
            if (p.head >= a.H) { p.head -= a.H; ++p.batch; }
            return p;
        };
        auto load_consts = [&](int head_) -> HeadConsts {
            HeadConsts c;
            c.th = *reinterpret_cast<const int4 *>(a.table + head_);
            c.rq = *reinterpret_cast<const int4 *>(a.requant_mult + 8 * head_);       // host-prepared constants
            c.rx = *reinterpret_cast<const int4 *>(a.requant_mult + 8 * head_ + 4);
            return c;
        };
        TileAt cur;
        cur.bh = (int)blockIdx.x / nblk; cur.qt = (int)blockIdx.x % nblk;
        cur.head = cur.bh % a.H; cur.batch = cur.bh / a.H;
        HeadConsts cc = load_consts(cur.head);

        for (int tile = blockIdx.x, it = 0; tile < num_tiles; tile += gridDim.x, ++it) {
            const int bh = cur.bh, qt = cur.qt;
            const int q0 = qt * kTile;
            const int kblocks = blocks_at(qt, cur.batch);
            HeadEntry th;
            th.B = cc.th.x; th.S = cc.th.y; th.D = cc.th.z;
            const int4 rq = cc.rq;
            const float out_scale = __int_as_float(cc.rx.x);
            const int32_t out_mult = cc.rx.y;
            const double inv_m = __hiloint2double(cc.rx.w, cc.rx.z);                     // 1 / M_h
            // valid keys of this row: all L of them, the causal prefix, the batch entry's key length
            // (keys at and beyond L exist only as padding of the last block when L is no multiple of 128)
            const int nv = valid_keys(cur.batch, q0);

            // the previous tile's O rows were staged in the panel: their bulk copies must have
            // read them before the panel is written again
            // (the scan flow first writes the panel after its first round, whose closing barrier serves)
            if (it > 0 && !two_rounds) {
                if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                asm volatile("bar.sync 1, 512;" ::: "memory");
            }

            // ---- phases 1 and 2: the panel receives the closeness r = max(x + (D - m), 0) of every
            // logit x = clamp(floor((acc*M + R) / 2^sh), -128, 127), R = 2^(sh-1), and the row gets m and
            // the sum of r.
            //
            // Scan flow (shifts up to 24).  The requantisation is monotone, so m is the image of the
            // largest accumulator: a first round over the S blocks only takes that maximum, and the
            // first contraction is then issued again.  In the second round, with
            // t = m - D, every accumulator is clamped to [lo_t, hi] -- lo_t the smallest accumulator
            // whose logit reaches max(t, -128), hi the largest one that gives 127 -- which performs the
            // clamp of x and the clip of the distance at once (M < 2^(sh-1) makes the steps of the map
            // smaller than one).  With y = clamp(acc - lo_t, 0, hi - lo_t) (one instruction) and
            // k = 24 - sh, y*(M << k) + (((lo_t*M + R) << k) - (t << 24)) lies in [0, 2^31) and r is
            // its top byte: one 32-bit multiply-add per logit, the bytes picked up by the packing
            // PRMTs, their sum by one dot-product instruction per word.  Keys outside the mask get
            // r = 0, so Z needs no correction.
            //
            // Shifts above 24 take the 64-bit multiply and keep the logits in the panel for a
            // separate closeness pass.
            int xmax = -128;
            uint32_t rsum = 0;
            int cm = 0;
            if (two_rounds) {
                const uint32_t mk = (uint32_t)rq.x, ck = (uint32_t)rq.y;
                const int neg_lo = rq.z, span = rq.w;
                // (the first two blocks were taken at the end of the previous tile, see below)
                int amax = amax_carry;
                for (int kb = r1_carry; ok && kb < kblocks; ++kb) first_round_block(kb, nv, amax);
                xmax = (int)((uint32_t)__viaddmin_s32_relu(amax, neg_lo, span) * mk + ck) >> 24;
                part_max[grp][t] = xmax;
                if (tid == 0 && it > 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                asm volatile("bar.sync 1, 512;" ::: "memory");        // the row threads only
                xmax = max(max(part_max[0][t], part_max[1][t]), max(part_max[2][t], part_max[3][t]));
                cm = th.D - xmax;

                // lo_t = clamp(ceil((t*2^sh - R) / M), lo, hi).  |t*2^sh - R| < 2^33 and M < 2^13: the product
                // with the host's double 1/M is within 2^-18 of the quotient, whose fraction is 0 or at
                // least 1/M, so rounding to nearest gives the ceiling or one less
                const int sh = a.requant_shift, kk = 24 - sh;
                const int M = (int)(mk >> kk), lo = -neg_lo, hi = lo + span;
                const int64_t R = (int64_t)1 << (sh - 1);
                const int64_t num = (int64_t)(-cm) * ((int64_t)1 << sh) - R;    // t * 2^sh - R
                int lo_t = lo;
                if (M > 0) {
                    int64_t q = __double2ll_rn(__ll2double_rn(num) * inv_m);
                    if (q * M < num) ++q;
                    lo_t = (int)min(max(q, (int64_t)lo), (int64_t)hi);
                }
                const int neg_lo_t = -lo_t, span_t = hi - lo_t;
                const uint32_t ck_t =
                    ((uint32_t)((int64_t)lo_t * M + R) << kk) - ((uint32_t)(-cm) << 24);
                for (int kb = 0; ok && kb < kblocks; ++kb) {
                    const uint32_t sb = s_buf;
                    ok = mbar_wait(smem_u32(&bars.s_full[sb]), s_cyc & 1, abortp, a.status, a.wait_cycles);
                    if (!ok) break;
                    if (++s_buf == kSBufs) { s_buf = 0; ++s_cyc; }
                    tcgen05_fence_after();
                    uint8_t *blk = row_base + kb * kPanelBlockBytes;
                    uint32_t acc[32];
                    tmem_ld32(tmem + lane_addr + sb * 128 + grp * 32, acc);
                    tcgen05_fence_before();
                    mbar_arrive(smem_u32(&bars.s_free[sb]));
                    uint32_t w[8];
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        uint32_t tt[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            tt[e] = (uint32_t)__viaddmin_s32_relu((int)acc[4 * g + e], neg_lo_t, span_t) * mk + ck_t;
                            if (CAUSAL && kb * kTile + grp * 32 + 4 * g + e >= nv) tt[e] = 0u;
                        }
                        w[g] = prmt(prmt(tt[0], tt[1], 0x0073u), prmt(tt[2], tt[3], 0x0073u), 0x5410u);
                        rsum = __dp4a(w[g], 0x01010101u, rsum);
                    }
                    *reinterpret_cast<uint4 *>(blk + (((2 * grp) ^ swz) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    *reinterpret_cast<uint4 *>(blk + (((2 * grp + 1) ^ swz) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
                }
            } else {
                const int32_t mult_hi = rq.x << (32 - a.requant_shift);   // x = high word of acc*mult_hi + 2^31
                for (int kb = 0; ok && kb < kblocks; ++kb) {
                    const uint32_t sb = s_buf;
                    ok = mbar_wait(smem_u32(&bars.s_full[sb]), s_cyc & 1, abortp, a.status, a.wait_cycles);
                    if (!ok) break;
                    if (++s_buf == kSBufs) { s_buf = 0; ++s_cyc; }
                    tcgen05_fence_after();
                    uint8_t *blk = row_base + kb * kPanelBlockBytes;
                    uint32_t acc[32];
                    tmem_ld32(tmem + lane_addr + sb * 128 + grp * 32, acc);
                    tcgen05_fence_before();
                    mbar_arrive(smem_u32(&bars.s_free[sb]));
                    uint32_t w[8];
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        int32_t x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            x[e] = (int32_t)(mad_wide_s32((int32_t)acc[4 * g + e], mult_hi, (int64_t)1 << 31) >> 32);
                            if (CAUSAL && kb * kTile + grp * 32 + 4 * g + e >= nv) x[e] = -128;
                        }
                        w[g] = cvt_pack_s8(x[1], x[0], cvt_pack_s8(x[3], x[2], 0u));
                        xmax = max(xmax, max(max(x[0], x[1]), max(x[2], x[3])));
                    }
                    *reinterpret_cast<uint4 *>(blk + (((2 * grp) ^ swz) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    *reinterpret_cast<uint4 *>(blk + (((2 * grp + 1) ^ swz) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
                }
                xmax = min(max(xmax, -128), 127);                     // the stored logits are clamped
                part_max[grp][t] = xmax;
                asm volatile("bar.sync 1, 512;" ::: "memory");
                xmax = max(max(part_max[0][t], part_max[1][t]), max(part_max[2][t], part_max[3][t]));
                cm = th.D - xmax;

                // closeness pass over the stored logits, in place; masked keys were stored as -128 and
                // contribute max(cm - 128, 0) each, which is taken out of the row's sum below
                const uint32_t c2 = prmt((uint32_t)cm, 0, 0x1010u);
                for (int kb = 0; kb < kblocks; ++kb) {
                    uint8_t *blk = row_base + kb * kPanelBlockBytes;
                    uint4 v[2];
#pragma unroll
                    for (int c = 0; c < 2; ++c) v[c] = *reinterpret_cast<const uint4 *>(blk + (((2 * grp + c) ^ swz) << 4));
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
                        uint32_t s2 = 0;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint32_t ev = __viaddmax_s16x2(prmt(w[k], 0, 0xA280u), c2, 0u);
                            const uint32_t od = __viaddmax_s16x2(prmt(w[k], 0, 0xB391u), c2, 0u);
                            s2 += ev + od;
                            w[k] = prmt(ev, od, 0x6240u);             // r bytes back in key order
                        }
                        rsum += (s2 & 0xffffu) + (s2 >> 16);
                        *reinterpret_cast<uint4 *>(blk + (((2 * grp + c) ^ swz) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            part_sum[grp][t] = (int)rsum;
            asm volatile("bar.sync 1, 512;" ::: "memory");
            int rs = part_sum[0][t] + part_sum[1][t] + part_sum[2][t] + part_sum[3][t];
            if (!two_rounds) rs -= (kblocks * kTile - nv) * max(cm - 128, 0);
            const int F = th.B - th.S * th.D;
            const uint32_t Z = (uint32_t)(nv * F + th.S * rs);
            const uint32_t rho = reciprocal<false, CLB>(max(Z, 1u));
            // X = s * rho' = a1 + b1*r < 2^24 with rho' = rho << (1 - OUT_SHIFT) for the divide (p = X >> 16) and
            // rho' = rho >> OUT_SHIFT for the leading-bit form (p = min(X >> 15, 255); its rho is 255 * 2^(15-k),
            // k <= 14).  Two keys share a 32-bit multiply-add on 16-bit lanes: with a1 = ah*256 + al and
            // b1 = b1h*256 + b1l, X >> 8 = ah + b1h*r + ((al + b1l*r) >> 8) < 2^16, and every partial result fits
            // its lane (r <= 127).  (A 64-bit multiply-add with the keys 24 bits apart needs one multiply per
            // pair instead of two, but its 64-bit addend costs two more instructions on the integer pipe.)
            // (an OUT_SHIFT above 1 is computed as OUT_SHIFT = 1 and the packed bytes are shifted by the rest)
            const int eff_shift = min(a.out_shift, 1), post_shift = a.out_shift - eff_shift;
            const uint32_t post_mask = (0xffu >> post_shift) * 0x01010101u;
            const uint32_t rp = CLB ? (rho >> eff_shift) : (rho << (1 - eff_shift));
            const uint32_t a1 = (uint32_t)F * rp, b1 = (uint32_t)th.S * rp;
            const uint32_t ah2 = (a1 >> 8) * 0x00010001u, al2 = (a1 & 255u) * 0x00010001u;
            const uint32_t b1h = b1 >> 8, b1l = b1 & 255u;

            // ---- phase 3: probabilities from the stored closeness values, in place
            for (int kb = 0; kb < kblocks; ++kb) {
                uint8_t *blk = row_base + kb * kPanelBlockBytes;
                uint4 v[2];
#pragma unroll
                for (int c = 0; c < 2; ++c) v[c] = *reinterpret_cast<const uint4 *>(blk + (((2 * grp + c) ^ swz) << 4));
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
                    uint32_t o[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t re = prmt(w[k], 0, 0x4240u), ro = prmt(w[k], 0, 0x4341u);   // keys 0, 2 and 1, 3
                        uint32_t q;
                        if (!CLB) {
                            const uint32_t ye = re * b1h + ah2 + prmt(re * b1l + al2, 0, 0x4341u);
                            const uint32_t yo = ro * b1h + ah2 + prmt(ro * b1l + al2, 0, 0x4341u);
                            q = prmt(ye, yo, 0x7351u);
                        } else {
                            // saturation at 255 folded into the add: Y stops at 255*128 + 127, p = Y >> 7 = high byte of 2*Y
                            const uint32_t ye = __viaddmin_u16x2(re * b1h + ah2, prmt(re * b1l + al2, 0, 0x4341u), 0x7fff7fffu);
                            const uint32_t yo = __viaddmin_u16x2(ro * b1h + ah2, prmt(ro * b1l + al2, 0, 0x4341u), 0x7fff7fffu);
                            q = prmt(ye * 2u, yo * 2u, 0x7351u);
                        }
                        if (CAUSAL) {
                            const int nb = nv - (kb * kTile + (2 * grp + c) * 16 + 4 * k);
                            q &= nb >= 4 ? 0xffffffffu : (nb <= 0 ? 0u : (1u << (8 * nb)) - 1u);
                        }
                        o[k] = q;
                    }
                    if (post_shift) {                              // uniform: OUT_SHIFT >= 2 (masked bytes stay zero)
#pragma unroll
                        for (int k = 0; k < 4; ++k) o[k] = (o[k] >> post_shift) & post_mask;
                    }
                    *reinterpret_cast<uint4 *>(blk + (((2 * grp + c) ^ swz) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
                // the tensor core reads the panel through the async proxy: hand this block over
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(smem_u32(&bars.p_ready[kb]));
            }

            // ---- while the last P.V block finishes: the first round of the NEXT tile over its first two
            // key blocks, whose K tiles (and Q) were prefetched and whose S blocks the tensor core has
            // produced meanwhile (the other K tiles can only be fetched once V is no longer needed)
            amax_carry = -(1 << 30);
            r1_carry = 0;
            const TileAt nxt = advance(cur);
            HeadConsts nc = cc;
            if (tile + (int)gridDim.x < num_tiles) {
                nc = load_consts(nxt.head);                    // used after the next tile's first round
                if (two_rounds) {
                    const int kblocks_n = blocks_at(nxt.qt, nxt.batch);
                    const int nv_n = valid_keys(nxt.batch, nxt.qt * kTile);
                    for (; ok && r1_carry < min(2, kblocks_n); ++r1_carry) first_round_block(r1_carry, nv_n, amax_carry);
                }
            }

            // ---- phase 4: O out of tensor memory.  A thread holds 16 columns of its row; writing them
            // straight to global memory would cost one memory transaction per lane (rows are 256 bytes
            // apart), so the tile goes through shared memory (the panel, free once the second
            // contraction is complete) as two boxes of 128 rows x 32 columns in the 128-byte swizzled
            // layout -- which also spreads a warp's 16-byte stores over all banks -- and one thread
            // sends both boxes off as tiled bulk stores; rows beyond L fall outside the tensor map
            // and are dropped.
            if (ok) ok = mbar_wait(smem_u32(&bars.o_full), it & 1, abortp, a.status, a.wait_cycles);
            if (ok) {
                tcgen05_fence_after();
                constexpr int kCols = D / 4;                      // columns of O per thread: 16 or 32
                uint32_t acc[kCols];
                if constexpr (kCols == 16) tmem_ld16(tmem + lane_addr + kTmemO + grp * kCols, acc);
                else tmem_ld32(tmem + lane_addr + kTmemO + grp * kCols, acc);
                if (a.out_mode == 1) {                            // optional dequantised view of O
#pragma unroll
                    for (int g = 0; g < kCols; ++g) acc[g] = __float_as_uint(__int2float_rn((int)acc[g]) * out_scale);
                }
                const int c0 = grp * kCols;
                if (a.out_mode == 2) {
                    // int8 output: every accumulator requantised with the head's output multiplier by the rule
                    // of the logits, clamp((acc*Mo + 2^(sh-1)) >> sh, -128, 127), in 64 bits (a handful of
                    // values per thread and tile); the tile is staged as plain rows of D bytes
                    const int64_t round = (int64_t)1 << (a.out_requant_shift - 1);
                    uint32_t packed[kCols / 4];
#pragma unroll
                    for (int g = 0; g < kCols / 4; ++g) {
                        int32_t x[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int64_t v = mad_wide_s32((int32_t)acc[4 * g + e], out_mult, round) >> a.out_requant_shift;
                            x[e] = (int32_t)min(max(v, (int64_t)-128), (int64_t)127);
                        }
                        packed[g] = cvt_pack_s8(x[1], x[0], cvt_pack_s8(x[3], x[2], 0u));
                    }
                    uint8_t *o_stage = panel + t * D + c0;
#pragma unroll
                    for (int g = 0; g < kCols / 16; ++g)
                        *reinterpret_cast<uint4 *>(o_stage + 16 * g) =
                            make_uint4(packed[4 * g], packed[4 * g + 1], packed[4 * g + 2], packed[4 * g + 3]);
                } else {
                    // column c of the tile sits in box c / 32, 16-byte chunk (c % 32) / 4 of its row
                    uint8_t *o_stage = panel + (c0 >> 5) * kOBoxBytes + t * 128;
#pragma unroll
                    for (int g = 0; g < kCols / 4; ++g)
                        *reinterpret_cast<uint4 *>(o_stage + (((((c0 & 31) >> 2) + g) ^ swz) << 4)) =
                            make_uint4(acc[4 * g], acc[4 * g + 1], acc[4 * g + 2], acc[4 * g + 3]);
                }
                tcgen05_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            if (tid == 0) leave_flag = *abortp;                   // one reader, so that all row threads agree
            asm volatile("bar.sync 1, 512;" ::: "memory");
            if (tid == 0 && !*(volatile int *)&leave_flag) {
                if (a.out_mode == 2) {
                    tma_store_3d(&map_o, 0, q0, bh, s_p);          // one box of 128 rows x D bytes
                } else {
#pragma unroll
                    for (int b = 0; b < D / 32; ++b) tma_store_3d(&map_o, 32 * b, q0, bh, s_p + b * kOBoxBytes);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            // leave the loop together (the flag was sampled once, before the barrier above)
            if (*(volatile int *)&leave_flag) break;
            cur = nxt;
            cc = nc;
        }
        if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // smem must outlive the reads
    }

    // ===================================================== common exit: free the tensor memory
    __syncthreads();
    if (warp == kTmaWarp) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode_tiled() {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
}

EncodeTiledFn encode_tiled_fn() {
    static const EncodeTiledFn fn = lookup_encode_tiled();   // initialised once, thread-safe
    return fn;
}

// [rows, d] uint8 tensor, boxes of 128 rows x 64 bytes (one column half of a tile), 64-byte swizzle.
bool make_tile_map(CUtensorMap *map, const void *ptr, uint64_t rows, uint32_t d) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d};
    const cuuint32_t box[2] = {(cuuint32_t)kHalf, (cuuint32_t)kTile};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// O as [B*H][L][d] 32-bit words, boxes of 128 rows x 32 words, 128-byte swizzle.  Three dimensions, so
// that a tile of the last, partial row block of a head stops at the head's end.
bool make_output_map(CUtensorMap *map, const void *ptr, uint64_t heads, uint64_t L, uint32_t d) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)L, (cuuint64_t)heads};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 4, (cuuint64_t)d * 4 * L};
    const cuuint32_t box[3] = {32, (cuuint32_t)kTile, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// O as [B*H][L][d] bytes (int8 output), one box of 128 rows x d bytes, no swizzle.
bool make_output_map_i8(CUtensorMap *map, const void *ptr, uint64_t heads, uint64_t L, uint32_t d) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)L, (cuuint64_t)heads};
    const cuuint64_t strides[2] = {(cuuint64_t)d, (cuuint64_t)d * L};
    const cuuint32_t box[3] = {(cuuint32_t)d, (cuuint32_t)kTile, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, bool CLB, bool CAUSAL, bool RING = false>
cudaError_t launch_variant(const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mo,
                           const FusedArgs &a, cudaStream_t st) {
    const int nblk = (a.L + kTile - 1) / kTile;
    constexpr size_t kTileBytes = (size_t)kTile * D;
    size_t panel = (size_t)kTile * nblk * kTile;
    if (panel < (D / 32) * (size_t)kOBoxBytes) panel = (D / 32) * (size_t)kOBoxBytes;   // the staged O boxes reuse the panel
    // resident: Q, two prefetch slots, a slot per K / V block, the panel; ring: Q, four slots, the panel
    const size_t smem = 1024 + (RING ? (1 + kRingSlots) * kTileBytes : 3 * kTileBytes + (size_t)nblk * kTileBytes) + panel;
    auto kernel = fused_attention_kernel<D, CLB, CAUSAL, RING>;
    // the attribute is raised once per instantiation and device to the largest size a launch can ask for
    static bool raised[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !raised[dev]) {
        constexpr size_t kMaxSmem = 1024 + (RING ? (1 + kRingSlots) * kTileBytes : 3 * kTileBytes + (size_t)kMaxBlocks * kTileBytes) +
                                    (size_t)kTile * kMaxBlocks * kTile;
        const size_t want = kMaxSmem < 232448 - 8192 ? kMaxSmem : smem;      // (resident d = 128 never asks for more than 512 keys)
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)want);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64 && want >= kMaxSmem) raised[dev] = true;
    }
    const int64_t tiles = (int64_t)a.B * a.H * nblk;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const unsigned blocks = (unsigned)(tiles < sms ? tiles : sms);      // persistent: one CTA per SM
    kernel<<<blocks, kThreads, smem, st>>>(mq, mk, mv, mo, a, (int)tiles);
    return cudaGetLastError();
}

}  // namespace

// d = 64 or 128 with up to 1024 keys (d = 128 beyond 512 keys streams K and V through a ring: K, V and the
// panel no longer fit the SM's shared memory together).
bool fused_shape_supported(int32_t L, int32_t d) {
    return L >= 1 && L <= kTile * kMaxBlocks && (d == 64 || d == 128);
}

cudaError_t launch_fused(const FusedArgs &a, cudaStream_t stream, uint64_t *launches) {
    CUtensorMap mq, mk, mv, mo;
    const uint64_t rows = (uint64_t)a.B * a.H * a.L;
    if (!fused_shape_supported(a.L, a.d)) return cudaErrorInvalidValue;
    if (!make_tile_map(&mq, a.Q, rows, a.d) || !make_tile_map(&mk, a.K, rows, a.d) || !make_tile_map(&mv, a.V, rows, a.d))
        return cudaErrorInvalidValue;
    if (!(a.out_mode == 2 ? make_output_map_i8(&mo, a.O, (uint64_t)a.B * a.H, (uint64_t)a.L, a.d)
                          : make_output_map(&mo, a.O, (uint64_t)a.B * a.H, (uint64_t)a.L, a.d)))
        return cudaErrorInvalidValue;
    cudaError_t e;
    // the masked instantiation also serves L that is no multiple of 128 (padding keys in the last block)
    // and per-batch key lengths
    const bool clb = (a.flags & HCCS_RECIP_CLB) != 0,
               causal = (a.flags & HCCS_CAUSAL) != 0 || a.L % kTile != 0 || a.key_len != nullptr;
    if (a.d == 64) {
        if (!clb && !causal) e = launch_variant<64, false, false>(mq, mk, mv, mo, a, stream);
        else if (clb && !causal) e = launch_variant<64, true, false>(mq, mk, mv, mo, a, stream);
        else if (!clb && causal) e = launch_variant<64, false, true>(mq, mk, mv, mo, a, stream);
        else e = launch_variant<64, true, true>(mq, mk, mv, mo, a, stream);
    } else if (a.L <= kTile * kMaxBlocks / 2) {
        if (!clb && !causal) e = launch_variant<128, false, false>(mq, mk, mv, mo, a, stream);
        else if (clb && !causal) e = launch_variant<128, true, false>(mq, mk, mv, mo, a, stream);
        else if (!clb && causal) e = launch_variant<128, false, true>(mq, mk, mv, mo, a, stream);
        else e = launch_variant<128, true, true>(mq, mk, mv, mo, a, stream);
    } else {
        if (!clb && !causal) e = launch_variant<128, false, false, true>(mq, mk, mv, mo, a, stream);
        else if (clb && !causal) e = launch_variant<128, true, false, true>(mq, mk, mv, mo, a, stream);
        else if (!clb && causal) e = launch_variant<128, false, true, true>(mq, mk, mv, mo, a, stream);
        else e = launch_variant<128, true, true, true>(mq, mk, mv, mo, a, stream);
    }
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

}  // namespace hccs
