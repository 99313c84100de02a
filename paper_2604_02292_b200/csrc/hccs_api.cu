// C ABI of libhccs: context, parameter-table validation and upload, argument checks, dispatch.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <new>

#include "hccs.h"
#include "hccs_internal.h"

struct hccs_ctx {
    int device = 0;
    hccs::HeadEntry *d_table = nullptr;     // device parameter table
    hccs::HeadEntry *h_table = nullptr;     // pinned staging copy of it
    int32_t *d_mult = nullptr;              // device copy of the fused path's per-head multipliers
    int32_t *h_mult = nullptr;              // pinned staging for them
    int32_t *mult_last = nullptr;           // host copy of what d_mult holds (to skip an unchanged upload)
    int32_t mult_last_heads = 0;            // 0: d_mult holds nothing yet
    int32_t capacity = 0;                   // heads the allocations can hold
    int32_t num_heads = 0;                  // 0 = nothing uploaded
    int32_t n_design = 0;
    int32_t out_shift = 0;
    uint32_t *d_status = nullptr;           // device status word (bounded waits report here)
    uint32_t *h_status = nullptr;           // pinned landing place for it
    cudaEvent_t table_copied = nullptr;     // the staging buffers may be rewritten after this
    cudaEvent_t mult_copied = nullptr;
    cudaStream_t d2h_stream = nullptr;      // hccs_forward_host: output copies
    static constexpr int kMaxPieces = 16;
    cudaEvent_t ev_done[kMaxPieces] = {};
    cudaEvent_t ev_join = nullptr;
    int32_t last_cuda_error = 0;
    uint64_t launches = 0;
};

namespace hccs {

FastDiv make_fastdiv(uint32_t d) {
    // q = (umulhi(n, mul) + n) >> shift is floor(n / d) for every n < 2^31:
    // shift = ceil(log2 d), mul = ceil(2^(32+shift) / d) - 2^32.
    FastDiv f;
    f.d = d;
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    const unsigned __int128 one = 1;
    const unsigned __int128 num = one << (32 + l);
    const unsigned __int128 m = (num + d - 1) / d - (one << 32);
    f.mul = (uint32_t)m;
    f.shift = l;
    return f;
}

}  // namespace hccs

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

hccs_status_t cuda_fail(hccs_ctx *ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = (int32_t)e;
    (void)cudaGetLastError();   // clear the sticky-free error so later calls start clean
    return HCCS_ERR_CUDA;
}

#define HCCS_CUDA(ctx, call)                                   \
    do {                                                       \
        cudaError_t e__ = (call);                              \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__);  \
    } while (0)

// The admissible parameter region (Section "Integer Range Constraints") for row length n.
bool theta_admissible(const hccs_head_params_t &t, int32_t n) {
    const int64_t B = t.B, S = t.S, D = t.Dmax;
    if (D < 1 || D > 127) return false;               // distances stay in signed int8
    if (S < 0 || S > 127) return false;               // S >= 0; int8 MAC operand
    if (B <= 0) return false;
    const int64_t floor_score = (256 + (int64_t)n - 1) / n;
    if (B - S * D < floor_score) return false;        // Z >= 256 (and scores non-negative)
    if ((int64_t)n * B > 32767) return false;         // Z <= 32767, rho >= 1; B <= 32767
    return true;
}

hccs_status_t ensure_capacity(hccs_ctx *ctx, int32_t heads) {
    if (heads <= ctx->capacity) return HCCS_OK;
    // growing the table: wait for everything that may still read the old one
    HCCS_CUDA(ctx, cudaDeviceSynchronize());
    if (ctx->d_table) cudaFree(ctx->d_table);
    if (ctx->h_table) cudaFreeHost(ctx->h_table);
    if (ctx->d_mult) cudaFree(ctx->d_mult);
    if (ctx->h_mult) cudaFreeHost(ctx->h_mult);
    delete[] ctx->mult_last;
    ctx->d_table = nullptr; ctx->h_table = nullptr; ctx->d_mult = nullptr; ctx->h_mult = nullptr;
    ctx->mult_last = nullptr; ctx->mult_last_heads = 0;
    ctx->capacity = 0;
    int32_t cap = heads < 64 ? 64 : heads;
    HCCS_CUDA(ctx, cudaMalloc(&ctx->d_table, sizeof(hccs::HeadEntry) * cap));
    HCCS_CUDA(ctx, cudaHostAlloc(&ctx->h_table, sizeof(hccs::HeadEntry) * cap, cudaHostAllocDefault));
    HCCS_CUDA(ctx, cudaMalloc(&ctx->d_mult, sizeof(int32_t) * 8 * cap));
    HCCS_CUDA(ctx, cudaHostAlloc(&ctx->h_mult, sizeof(int32_t) * 8 * cap, cudaHostAllocDefault));
    ctx->mult_last = new (std::nothrow) int32_t[8 * (size_t)cap];
    if (!ctx->mult_last) return HCCS_ERR_CUDA;
    ctx->capacity = cap;
    return HCCS_OK;
}

hccs_status_t check_forward_args(hccs_ctx *ctx, const void *in, const void *out, int32_t B, int32_t H,
                                 int32_t Lq, int32_t Lk, uint32_t flags) {
    if (!ctx) return HCCS_ERR_INVALID_ARG;
    if (B < 0 || H < 0 || Lq < 0 || Lk < 0) return HCCS_ERR_INVALID_ARG;
    if (flags & ~7u) return HCCS_ERR_INVALID_ARG;
    if (ctx->num_heads == 0) return HCCS_ERR_NOT_UPLOADED;
    if (H != ctx->num_heads) return HCCS_ERR_INVALID_ARG;
    if (Lk > ctx->n_design) return HCCS_ERR_CONSTRAINT;
    const int64_t rows = (int64_t)B * H * Lq;
    if (rows >= (1ll << 31)) return HCCS_ERR_UNSUPPORTED;
    if (rows * Lk != 0 && (!in || !out)) return HCCS_ERR_INVALID_ARG;
    return HCCS_OK;
}

hccs::RowArgs make_row_args(const hccs_ctx *ctx, int32_t rows, int32_t H, int32_t Lq, int32_t Lk, uint32_t flags,
                            const int32_t *key_len) {
    hccs::RowArgs a;
    a.table = ctx->d_table;
    a.status = ctx->d_status;
    a.wait_cycles = hccs::kDefaultWaitCycles;
    a.rows = rows;
    a.H = H;
    a.Lq = Lq;
    a.Lk = Lk;
    a.causal_off = Lk - Lq;
    a.causal = (flags & HCCS_CAUSAL) ? 1 : 0;
    a.key_len = key_len;
    a.out_shift = ctx->out_shift;
    a.slice0 = 0;
    a.div_Lq = hccs::make_fastdiv((uint32_t)Lq);
    a.div_H = hccs::make_fastdiv((uint32_t)H);
    return a;
}

}  // namespace

extern "C" {

hccs_status_t hccs_create(hccs_ctx_t **out, int device) {
    if (!out) return HCCS_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) { (void)cudaGetLastError(); return HCCS_ERR_CUDA; }
    if (device < 0 || device >= count) return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(device);
    if (!g.ok) return HCCS_ERR_CUDA;
    hccs_ctx *ctx = new (std::nothrow) hccs_ctx();
    if (!ctx) return HCCS_ERR_INVALID_ARG;
    ctx->device = device;
    cudaError_t e = cudaMalloc(&ctx->d_status, 64 * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 64 * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaHostAlloc(&ctx->h_status, sizeof(uint32_t), cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->table_copied, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->mult_copied, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
    for (int i = 0; i < hccs_ctx::kMaxPieces && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        hccs_destroy(ctx);
        return HCCS_ERR_CUDA;
    }
    *out = ctx;
    return HCCS_OK;
}

hccs_status_t hccs_destroy(hccs_ctx_t *ctx) {
    if (!ctx) return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (ctx->d_table) cudaFree(ctx->d_table);
    if (ctx->h_table) cudaFreeHost(ctx->h_table);
    if (ctx->d_mult) cudaFree(ctx->d_mult);
    if (ctx->h_mult) cudaFreeHost(ctx->h_mult);
    delete[] ctx->mult_last;
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    if (ctx->table_copied) cudaEventDestroy(ctx->table_copied);
    if (ctx->mult_copied) cudaEventDestroy(ctx->mult_copied);
    if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    for (int i = 0; i < hccs_ctx::kMaxPieces; ++i) {
        if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
    }
    (void)cudaGetLastError();
    delete ctx;
    return HCCS_OK;
}

hccs_status_t hccs_params_check(const hccs_head_params_t *params, int32_t num_heads,
                                int32_t n_design, int32_t *bad_head) {
    if (bad_head) *bad_head = -1;
    if (!params || num_heads < 1 || num_heads > (1 << 20)) return HCCS_ERR_INVALID_ARG;
    if (n_design < 1 || n_design > 32767) return HCCS_ERR_INVALID_ARG;
    for (int32_t h = 0; h < num_heads; ++h) {
        if (!theta_admissible(params[h], n_design)) {
            if (bad_head) *bad_head = h;
            return HCCS_ERR_CONSTRAINT;
        }
    }
    return HCCS_OK;
}

hccs_status_t hccs_params_upload(hccs_ctx_t *ctx, const hccs_head_params_t *params,
                                 int32_t num_heads, int32_t n_design, int32_t out_shift,
                                 int32_t *bad_head, void *cuda_stream) {
    if (bad_head) *bad_head = -1;
    if (!ctx) return HCCS_ERR_INVALID_ARG;
    if (out_shift < 0 || out_shift > 8) return HCCS_ERR_INVALID_ARG;
    hccs_status_t chk = hccs_params_check(params, num_heads, n_design, bad_head);
    if (chk != HCCS_OK) return chk;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    hccs_status_t st = ensure_capacity(ctx, num_heads);
    if (st != HCCS_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the pinned staging copy may still be in flight from the previous upload
    HCCS_CUDA(ctx, cudaEventSynchronize(ctx->table_copied));
    for (int32_t h = 0; h < num_heads; ++h) {
        hccs::HeadEntry e;
        e.B = params[h].B;
        e.S = params[h].S;
        e.D = params[h].Dmax;
        e.pad = 0;
        ctx->h_table[h] = e;
    }
    HCCS_CUDA(ctx, cudaMemcpyAsync(ctx->d_table, ctx->h_table, sizeof(hccs::HeadEntry) * num_heads,
                                   cudaMemcpyHostToDevice, stream));
    HCCS_CUDA(ctx, cudaEventRecord(ctx->table_copied, stream));
    ctx->num_heads = num_heads;
    ctx->n_design = n_design;
    ctx->out_shift = out_shift;
    return HCCS_OK;
}

hccs_status_t hccs_forward(hccs_ctx_t *ctx, const int8_t *logits, void *probs,
                           int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                           uint32_t flags, void *cuda_stream) {
    hccs_status_t st = check_forward_args(ctx, logits, probs, B, H, Lq, Lk, flags);
    if (st != HCCS_OK) return st;
    const int64_t rows = (int64_t)B * H * Lq;
    if (rows * Lk == 0) return HCCS_OK;
    if ((flags & HCCS_OUT_U16) && (const void *)logits == probs) return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    hccs::RowArgs a = make_row_args(ctx, (int32_t)rows, H, Lq, Lk, flags, nullptr);
    HCCS_CUDA(ctx, hccs::launch_rows(logits, probs, a, flags, (cudaStream_t)cuda_stream, &ctx->launches));
    return HCCS_OK;
}

hccs_status_t hccs_forward_keylen(hccs_ctx_t *ctx, const int8_t *logits, void *probs, const int32_t *key_len,
                                  int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                                  uint32_t flags, void *cuda_stream) {
    hccs_status_t st = check_forward_args(ctx, logits, probs, B, H, Lq, Lk, flags);
    if (st != HCCS_OK) return st;
    const int64_t rows = (int64_t)B * H * Lq;
    if (rows * Lk == 0) return HCCS_OK;
    if (!key_len) return HCCS_ERR_INVALID_ARG;
    if ((flags & HCCS_OUT_U16) && (const void *)logits == probs) return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    hccs::RowArgs a = make_row_args(ctx, (int32_t)rows, H, Lq, Lk, flags, key_len);
    HCCS_CUDA(ctx, hccs::launch_rows(logits, probs, a, flags, (cudaStream_t)cuda_stream, &ctx->launches));
    return HCCS_OK;
}

hccs_status_t hccs_forward_host(hccs_ctx_t *ctx, const int8_t *logits_host, void *probs_host,
                                int8_t *logits_staging, void *probs_staging,
                                int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                                uint32_t flags, void *cuda_stream) {
    hccs_status_t st = check_forward_args(ctx, logits_host, probs_host, B, H, Lq, Lk, flags);
    if (st != HCCS_OK) return st;
    const int64_t rows = (int64_t)B * H * Lq;
    if (rows * Lk == 0) return HCCS_OK;
    if (!logits_staging || !probs_staging || (void *)logits_staging == probs_staging)
        return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const int64_t osz = (flags & HCCS_OUT_U16) ? 2 : 1;
    // Pieces are whole (b, h) slices, so that a piece's first row has query index 0 and its
    // head is a pure function of the slice index.  A piece's input copy and its kernel run in order on
    // the caller's stream (the kernel of one piece delays the next copy by microseconds only); the
    // results come down on a second stream, piece by piece behind an event, so that the two copy
    // directions overlap.  One event hand-over per piece: each costs several microseconds of latency.
    const int64_t slices = (int64_t)B * H;
    const int64_t slice_bytes = (int64_t)Lq * Lk;
    int pieces = 1;
    if (slices * slice_bytes >= (8ll << 20)) pieces = 8;
    if (pieces > slices) pieces = (int)slices;
    for (int p = 0; p < pieces; ++p) {
        const int64_t s0 = slices * p / pieces, s1 = slices * (p + 1) / pieces;
        const int64_t off = s0 * slice_bytes, bytes = (s1 - s0) * slice_bytes;
        HCCS_CUDA(ctx, cudaMemcpyAsync(logits_staging + off, logits_host + off, bytes,
                                       cudaMemcpyHostToDevice, stream));
        // a piece starts at slice s0: the kernel runs on a view whose flat row 0 is that slice, and the
        // row arguments carry the starting slice so that (r / Lq) mod H still gives the head
        hccs::RowArgs a = make_row_args(ctx, (int32_t)((s1 - s0) * Lq), H, Lq, Lk, flags, nullptr);
        a.slice0 = (int32_t)s0;
        HCCS_CUDA(ctx, hccs::launch_rows(logits_staging + off, (char *)probs_staging + off * osz, a,
                                         flags, stream, &ctx->launches));
        HCCS_CUDA(ctx, cudaEventRecord(ctx->ev_done[p], stream));
        HCCS_CUDA(ctx, cudaStreamWaitEvent(ctx->d2h_stream, ctx->ev_done[p], 0));
        HCCS_CUDA(ctx, cudaMemcpyAsync((char *)probs_host + off * osz, (char *)probs_staging + off * osz,
                                       bytes * osz, cudaMemcpyDeviceToHost, ctx->d2h_stream));
    }
    HCCS_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->d2h_stream));
    HCCS_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->ev_join, 0));
    return HCCS_OK;
}

// Shared by the int32, fp32 and int8 entry points: out_scale != NULL means fp32 output, out_mult != NULL
// int8 output, neither int32 output.
static hccs_status_t fused_common(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K, const int8_t *V, void *O,
                                  const float *out_scale, const int32_t *out_mult, int32_t out_shift,
                                  const int32_t *key_len, const int32_t *requant_mult,
                                  int32_t requant_shift, int32_t B, int32_t H, int32_t L, int32_t d,
                                  uint32_t flags, void *cuda_stream) {
    if (!ctx || B < 0 || H < 0 || L < 0 || d < 0) return HCCS_ERR_INVALID_ARG;
    if (flags & ~7u) return HCCS_ERR_INVALID_ARG;
    if (flags & HCCS_OUT_U16) return HCCS_ERR_UNSUPPORTED;
    if (ctx->num_heads == 0) return HCCS_ERR_NOT_UPLOADED;
    if (H != ctx->num_heads || !requant_mult) return HCCS_ERR_INVALID_ARG;
    if (requant_shift < 1 || requant_shift > 31) return HCCS_ERR_INVALID_ARG;
    for (int32_t h = 0; h < H; ++h)
        if (requant_mult[h] < 0 || requant_mult[h] >= (1 << 13)) return HCCS_ERR_INVALID_ARG;
    if (out_mult) {
        if (out_shift < 1 || out_shift > 31) return HCCS_ERR_INVALID_ARG;
        for (int32_t h = 0; h < H; ++h)
            if (out_mult[h] < 0 || out_mult[h] >= (1 << 13)) return HCCS_ERR_INVALID_ARG;
    }
    // the kernel requantises with the multiplier pre-shifted by 32 - requant_shift bits
    for (int32_t h = 0; h < H; ++h)
        if ((int64_t)requant_mult[h] << (32 - requant_shift) >= (1ll << 31)) return HCCS_ERR_UNSUPPORTED;
    if (L > ctx->n_design) return HCCS_ERR_CONSTRAINT;
    if ((int64_t)B * H * L * d == 0) return HCCS_OK;
    if (!Q || !K || !V || !O) return HCCS_ERR_INVALID_ARG;
    if (!hccs::fused_shape_supported(L, d)) return HCCS_ERR_UNSUPPORTED;
    if ((((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15u) != 0)
        return HCCS_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // Per head: {multiplier, and for shifts up to 24 the constants of the single-multiply
    // requantisation: multiplier << k, offset, -lo, hi - lo} (see hccs_fused.cu, phase 1), then the
    // fp32 output scale, the int8 output multiplier and 1 / multiplier as a double; eight 32-bit words per head.
    // The words are built on the stack and go up only when they differ from what the device table
    // already holds (the usual case is the same multipliers call after call): then nothing is copied
    // and the host never waits for an earlier call's copy.
    constexpr int32_t kStackHeads = 64;
    int32_t stack_words[8 * kStackHeads];
    int32_t *words = H <= kStackHeads ? stack_words : new (std::nothrow) int32_t[8 * (size_t)H];
    if (!words) return HCCS_ERR_INVALID_ARG;
    for (int32_t h = 0; h < H; ++h) {
        const int64_t M = requant_mult[h];
        int32_t *e = words + 8 * h;
        e[0] = (int32_t)M;
        e[1] = e[2] = e[3] = e[6] = e[7] = 0;
        e[5] = out_mult ? out_mult[h] : 0;
        const float scale = out_scale ? out_scale[h] : 1.0f;
        memcpy(&e[4], &scale, sizeof(float));
        const double inv_m = M > 0 ? 1.0 / (double)M : 0.0;      // words 6 and 7
        memcpy(&e[6], &inv_m, sizeof(double));
        if (requant_shift <= 24) {
            const int sh = requant_shift, k = 24 - sh;
            const int64_t R = (int64_t)1 << (sh - 1), lim = (int64_t)1 << 21;   // |acc| <= d*128*128 <= 2^21
            int64_t lo = -lim, hi = lim;
            if (M > 0) {
                lo = -((((int64_t)128 << sh) + R) / M);          // smallest accumulator that gives -128
                hi = (((int64_t)128 << sh) - 1 - R) / M;         // largest accumulator that gives 127
                if (lo < -lim) lo = -lim;
                if (hi > lim) hi = lim;
            }
            e[0] = (int32_t)(uint32_t)((uint64_t)M << k);
            e[1] = (int32_t)(uint32_t)(uint64_t)((lo * M + R) * ((int64_t)1 << k));
            e[2] = (int32_t)-lo;
            e[3] = (int32_t)(hi - lo);
        }
    }
    const bool same = ctx->mult_last_heads == H && memcmp(ctx->mult_last, words, sizeof(int32_t) * 8 * H) == 0;
    if (!same) {
        // the pinned staging copy may still be in flight from the previous upload
        cudaError_t e = cudaEventSynchronize(ctx->mult_copied);
        if (e == cudaSuccess) {
            memcpy(ctx->h_mult, words, sizeof(int32_t) * 8 * H);
            e = cudaMemcpyAsync(ctx->d_mult, ctx->h_mult, sizeof(int32_t) * 8 * H, cudaMemcpyHostToDevice, stream);
        }
        if (e == cudaSuccess) e = cudaEventRecord(ctx->mult_copied, stream);
        if (e == cudaSuccess) {
            memcpy(ctx->mult_last, words, sizeof(int32_t) * 8 * H);
            ctx->mult_last_heads = H;
        } else {
            ctx->mult_last_heads = 0;
        }
        if (words != stack_words) delete[] words;
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    } else {
        if (words != stack_words) delete[] words;
        // the table went up on the stream of an earlier call: order this stream behind that copy
        HCCS_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->mult_copied, 0));
    }
    hccs::FusedArgs a;
    a.Q = Q; a.K = K; a.V = V; a.O = O;
    a.table = ctx->d_table;
    a.requant_mult = ctx->d_mult;
    a.status = ctx->d_status;
    a.wait_cycles = hccs::kDefaultWaitCycles;
    a.out_mode = out_scale ? 1 : (out_mult ? 2 : 0);
    a.out_requant_shift = out_mult ? out_shift : 1;
    a.key_len = key_len;
    a.requant_shift = requant_shift;
    a.B = B; a.H = H; a.L = L; a.d = d;
    a.out_shift = ctx->out_shift;
    a.flags = flags;
    HCCS_CUDA(ctx, hccs::launch_fused(a, stream, &ctx->launches));
    return HCCS_OK;
}

hccs_status_t hccs_attention_fused(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                   const int8_t *V, int32_t *O, const int32_t *requant_mult,
                                   int32_t requant_shift, int32_t B, int32_t H, int32_t L, int32_t d,
                                   uint32_t flags, void *cuda_stream) {
    return fused_common(ctx, Q, K, V, O, nullptr, nullptr, 0, nullptr, requant_mult, requant_shift, B, H, L, d, flags, cuda_stream);
}

hccs_status_t hccs_attention_fused_keylen(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                          const int8_t *V, int32_t *O, const int32_t *key_len,
                                          const int32_t *requant_mult, int32_t requant_shift,
                                          int32_t B, int32_t H, int32_t L, int32_t d,
                                          uint32_t flags, void *cuda_stream) {
    if (!key_len && (int64_t)B * H * L * d != 0) return HCCS_ERR_INVALID_ARG;
    return fused_common(ctx, Q, K, V, O, nullptr, nullptr, 0, key_len, requant_mult, requant_shift, B, H, L, d, flags, cuda_stream);
}

hccs_status_t hccs_attention_fused_f32(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                       const int8_t *V, float *O, const float *out_scale,
                                       const int32_t *requant_mult, int32_t requant_shift,
                                       int32_t B, int32_t H, int32_t L, int32_t d,
                                       uint32_t flags, void *cuda_stream) {
    if (!out_scale) return HCCS_ERR_INVALID_ARG;
    return fused_common(ctx, Q, K, V, O, out_scale, nullptr, 0, nullptr, requant_mult, requant_shift, B, H, L, d, flags, cuda_stream);
}

hccs_status_t hccs_attention_fused_i8(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                      const int8_t *V, int8_t *O, const int32_t *out_mult, int32_t out_shift,
                                      const int32_t *requant_mult, int32_t requant_shift,
                                      int32_t B, int32_t H, int32_t L, int32_t d,
                                      uint32_t flags, void *cuda_stream) {
    if (!out_mult) return HCCS_ERR_INVALID_ARG;
    return fused_common(ctx, Q, K, V, O, nullptr, out_mult, out_shift, nullptr, requant_mult, requant_shift, B, H, L, d, flags, cuda_stream);
}

hccs_status_t hccs_device_status(hccs_ctx_t *ctx, uint32_t *word, void *cuda_stream) {
    if (!ctx) return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    HCCS_CUDA(ctx, cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(uint32_t),
                                   cudaMemcpyDeviceToHost, stream));
    HCCS_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(uint32_t), stream));
    HCCS_CUDA(ctx, cudaStreamSynchronize(stream));
    const uint32_t w = *ctx->h_status;
    if (word) *word = w;
    return w ? HCCS_ERR_DEVICE_TIMEOUT : HCCS_OK;
}

hccs_status_t hccs_debug_wait_timeout(hccs_ctx_t *ctx, int32_t mode, int64_t limit_cycles, void *cuda_stream) {
    if (!ctx || (mode != 0 && mode != 1)) return HCCS_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > 10000000) return HCCS_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
    HCCS_CUDA(ctx, hccs::launch_wait_probe(ctx->d_status, mode, (long long)limit_cycles, (cudaStream_t)cuda_stream));
    ctx->launches += 1;
    return HCCS_OK;
}

int32_t hccs_last_cuda_error(const hccs_ctx_t *ctx) { return ctx ? ctx->last_cuda_error : 0; }

uint64_t hccs_launch_count(const hccs_ctx_t *ctx) { return ctx ? ctx->launches : 0; }

const char *hccs_status_string(hccs_status_t status) {
    switch (status) {
        case HCCS_OK: return "HCCS_OK";
        case HCCS_ERR_INVALID_ARG: return "HCCS_ERR_INVALID_ARG";
        case HCCS_ERR_CONSTRAINT: return "HCCS_ERR_CONSTRAINT";
        case HCCS_ERR_NOT_UPLOADED: return "HCCS_ERR_NOT_UPLOADED";
        case HCCS_ERR_UNSUPPORTED: return "HCCS_ERR_UNSUPPORTED";
        case HCCS_ERR_CUDA: return "HCCS_ERR_CUDA";
        case HCCS_ERR_DEVICE_TIMEOUT: return "HCCS_ERR_DEVICE_TIMEOUT";
    }
    return "HCCS_<unknown status>";
}

}  // extern "C"
