/*
 * hccs.h -- C ABI of libhccs: the inference step of the Head-Calibrated
 * Clipped-Linear Softmax (HCCS) on NVIDIA B200 (sm_100a).
 *
 * HCCS maps a row of int8 attention logits x to scaled integer probabilities
 * using only integer arithmetic (paper, Section III and Algorithm 1):
 *
 *   m       = max_j x_j                                   (Eq. 1)
 *   delta_j = min(m - x_j, Dmax_h)                        (Eq. 2)
 *   s_j     = B_h - S_h * delta_j            (>= 0)       (Eq. 3, Eq. 4)
 *   Z       = sum_j s_j                                   (Eq. 5)
 *   int16 output:  rho = floor(32767 / Z),      p_j = s_j * rho           (Eq. 6, 7)
 *   int8 output:   rho = floor(255 * 2^15 / Z), p_j = (s_j * rho) >> (15 + OUT_SHIFT)   (Eq. 8)
 *   leading-bit reciprocal (CLB): k = floor(log2 Z), rho = T' >> k        (Eq. 9)
 *
 * with one parameter triple theta_h = (B_h, S_h, Dmax_h) per attention head.
 *
 * Conventions for every entry point
 *   - Tensors are contiguous, row-major, innermost dimension last.
 *   - "device" pointers are CUDA device memory of the context's device, owned by
 *     the caller; "host" pointers are ordinary (preferably pinned) host memory.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the default stream) and the call returns without synchronising, unless
 *     stated otherwise.
 *   - Errors are return codes only.  On any error nothing is launched.
 *   - A context is not thread-safe: one host call at a time per context (different contexts, also
 *     on the same device, are independent).  On the GPU, hccs_forward, hccs_forward_keylen and
 *     hccs_forward_host calls of one context only read the context's parameter table and may
 *     overlap each other freely (different streams, back to back on one stream).  Calls that rewrite
 *     device memory the context owns do so on their own `cuda_stream`: hccs_params_upload (the
 *     parameter table) and the hccs_attention_fused* calls (a small per-head multiplier table,
 *     rewritten only when the multipliers, the shift or the output scales differ from the previous
 *     fused call's).  Order such a call against other work of the same context that may still be
 *     running on another stream yourself (an event, or one stream per context).
 *   - There is no CPU implementation behind this interface.
 */
#ifndef HCCS_H
#define HCCS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hccs_ctx hccs_ctx_t;   /* opaque; owns the device parameter table and a status word */

/* theta_h of the paper's Section "Offline Calibration": fixed at inference. */
typedef struct {
    int32_t B;      /* B_h    > 0  : score of the row maximum                     */
    int32_t S;      /* S_h    >= 0 : slope per unit of clamped distance           */
    int32_t Dmax;   /* Dmax_h in [1,127] : clamp bound of the distance (Eq. 2)    */
} hccs_head_params_t;

typedef enum {
    HCCS_OK = 0,
    HCCS_ERR_INVALID_ARG    = 1,  /* NULL pointer, negative size, unknown flag, wrong H          */
    HCCS_ERR_CONSTRAINT     = 2,  /* theta outside the admissible region, or Lk > n_design       */
    HCCS_ERR_NOT_UPLOADED   = 3,  /* hccs_forward before hccs_params_upload                      */
    HCCS_ERR_UNSUPPORTED    = 4,  /* shape the kernels cannot take (documented per call)         */
    HCCS_ERR_CUDA           = 5,  /* a CUDA runtime call failed; see hccs_last_cuda_error        */
    HCCS_ERR_DEVICE_TIMEOUT = 6   /* a bounded device-side wait gave up (hccs_device_status)     */
} hccs_status_t;

/* flags of hccs_forward / hccs_attention_fused (bitwise OR) */
enum {
    HCCS_OUT_U8    = 0,   /* uint8 probabilities, T = 255 (int8 output path, Eq. 8)             */
    HCCS_OUT_U16   = 1,   /* uint16 probabilities, T = 32767 (Eq. 6, 7)                         */
    HCCS_RECIP_DIV = 0,   /* exact integer divide                                               */
    HCCS_RECIP_CLB = 2,   /* leading-bit reciprocal (Eq. 9); uint8 results saturate at 255      */
    HCCS_CAUSAL    = 4    /* key j of query i takes part iff j <= i + (Lk - Lq); others give 0  */
};

/* Creates a context on CUDA device `device` (allocates a small parameter table lazily and a
 * 4-byte device status word).  *out receives the context.  Synchronous. */
hccs_status_t hccs_create(hccs_ctx_t **out, int device);

/* Frees the context's device memory.  The caller must have synchronised its streams. */
hccs_status_t hccs_destroy(hccs_ctx_t *ctx);

/*
 * Uploads the per-head parameter table (Section "Offline Calibration"; looked up per row by the
 * row's head, Section "Multi-tile scaling").
 *   params     host array of num_heads triples
 *   n_design   the row length n the table was calibrated for (1..32767)
 *   out_shift  OUT_SHIFT of the int8 output path (Eq. 8), 0..8; 0 unless you know better
 *   bad_head   may be NULL; receives the first offending head on HCCS_ERR_CONSTRAINT, else -1
 * Every item of the paper's Section "Integer Range Constraints" is checked on the host for
 * n = n_design:  Dmax <= 127;  S >= 0;  B - S*Dmax >= ceil(256/n);  n*B <= 32767 (hence
 * B <= 32767).  Two more bounds are this library's own additions, not the paper's: Dmax >= 1 (a
 * clamp bound of 0 would make every row uniform) and S <= 127 (the paper describes the score as a
 * single int8 multiply-accumulate, so S is kept an int8 operand).  On a violation nothing is
 * uploaded and the previous table stays in force.
 * The table is copied from an internal pinned staging buffer on `cuda_stream`; `params` may be
 * reused as soon as the call returns.  The first upload (or one with more heads than before)
 * allocates device memory and therefore synchronises the device.
 */
hccs_status_t hccs_params_upload(hccs_ctx_t *ctx, const hccs_head_params_t *params,
                                 int32_t num_heads, int32_t n_design, int32_t out_shift,
                                 int32_t *bad_head, void *cuda_stream);

/* The host-side admissibility check of hccs_params_upload on its own (no context, no CUDA call):
 * HCCS_OK, or HCCS_ERR_CONSTRAINT with *bad_head (may be NULL) = first offending head, or
 * HCCS_ERR_INVALID_ARG for a NULL table, num_heads < 1 or n_design outside 1..32767. */
hccs_status_t hccs_params_check(const hccs_head_params_t *params, int32_t num_heads,
                                int32_t n_design, int32_t *bad_head);

/*
 * HCCS over every row of a logit tensor (Algorithm 1 applied to B*H*Lq independent rows,
 * Section "Vectorization and Parallelism Across Rows").
 *   logits  device int8  [B, H, Lq, Lk]
 *   probs   device uint8 [B, H, Lq, Lk] (HCCS_OUT_U8) or uint16 (HCCS_OUT_U16); may equal
 *           `logits` for uint8 output (each row is read completely before it is written)
 *   H       must equal the uploaded num_heads; the head of flat row r is (r / Lq) mod H
 *   Lk      1..n_design (HCCS_ERR_CONSTRAINT beyond: the admissible band only narrows with n)
 * Rows shorter than n_design, and causal rows with few valid keys, are computed with the same
 * formulas in 32-bit integers (rho is not narrowed to int16).  Masked positions take no part in
 * the max or the sum and produce 0; a row without any valid key produces all zeros.
 * Any Lk and any pointer alignment is accepted; the fast kernels need Lk % 16 == 0 and
 * 16-byte-aligned pointers, everything else runs in a slower CUDA kernel.  Empty tensors
 * (B*H*Lq*Lk == 0) return HCCS_OK without a launch.  B*H*Lq must be below 2^31.
 */
hccs_status_t hccs_forward(hccs_ctx_t *ctx, const int8_t *logits, void *probs,
                           int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                           uint32_t flags, void *cuda_stream);

/*
 * hccs_forward with a padding mask: key j of batch entry b takes part iff j < key_len[b] (and,
 * with HCCS_CAUSAL, iff the causal rule holds as well).  This is the mask of the paper's encoder
 * workloads, whose sequences are padded to 64 or 128 tokens (Section "Models and tasks"); the
 * paper itself does not define masking: masked keys are left out of the max (Eq. 1) and the sum
 * (Eq. 5) and produce 0, a row without valid keys produces zeros.
 *   key_len  device int32 [B]; values are clamped to [0, Lk]
 * Everything else as hccs_forward.
 */
hccs_status_t hccs_forward_keylen(hccs_ctx_t *ctx, const int8_t *logits, void *probs,
                                  const int32_t *key_len, int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                                  uint32_t flags, void *cuda_stream);

/*
 * The same operation for HOST tensors: copies `logits_host` to `logits_staging`, runs
 * hccs_forward, copies the result back to `probs_host`, all on `cuda_stream`, in pieces so that
 * the two copy directions and the kernel overlap.  The caller provides both device staging
 * buffers (same sizes as the tensors; the library allocates nothing here).  Host buffers should
 * be pinned (cudaHostAlloc / torch pin_memory), otherwise the copies serialise.  The result is
 * complete once `cuda_stream` has been synchronised.
 */
hccs_status_t hccs_forward_host(hccs_ctx_t *ctx, const int8_t *logits_host, void *probs_host,
                                int8_t *logits_staging, void *probs_staging,
                                int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                                uint32_t flags, void *cuda_stream);

/*
 * Fused integer attention (not in the paper, which only notes that the integer outputs stay
 * compatible with fixed-point attention pipelines): per (b, h)
 *   acc_ij = sum_c Q[i,c] * K[j,c]                         (int32)
 *   x_ij   = clamp((acc_ij * requant_mult[h] + 2^(requant_shift-1)) >> requant_shift, -128, 127)
 *   P_i.   = HCCS(x_i.) with theta_h, uint8 output         (Algorithm 1, Eq. 8)
 *   O[i,:] = sum_j P_ij * V[j,:]                           (int32)
 *   Q, K, V       device int8  [B, H, L, d]
 *   O             device int32 [B, H, L, d]
 *   requant_mult  HOST int32 [H], each in [0, 2^13) and below 2^(requant_shift-1); requant_shift in 1..31
 *   flags         HCCS_RECIP_CLB and HCCS_CAUSAL are honoured; HCCS_OUT_U16 is HCCS_ERR_UNSUPPORTED
 * Supported shapes: d == 64 or d == 128 with 1 <= L <= 1024 (the 128 x L probability panel stays in
 * one SM's shared memory; for d == 128 beyond 512 keys K and V stream through a ring of buffers
 * beside it); L <= n_design, pointers 16-byte aligned; anything else returns HCCS_ERR_UNSUPPORTED.
 * The logits and probabilities never leave the chip.
 */
hccs_status_t hccs_attention_fused(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                   const int8_t *V, int32_t *O, const int32_t *requant_mult,
                                   int32_t requant_shift, int32_t B, int32_t H, int32_t L, int32_t d,
                                   uint32_t flags, void *cuda_stream);

/*
 * hccs_attention_fused with a key-padding mask: key_len is a DEVICE int32 [B] array; keys at and
 * beyond key_len[b] (clamped to 0..L) of batch entry b are padding: like causally masked keys they
 * take no part in the row maximum and the row sum and get probability 0, so O is the attention over
 * the first key_len[b] keys alone; a batch entry with key length 0 gets O = 0.  Key blocks that
 * hold padding only are not computed at all.  Combines with HCCS_CAUSAL.  Everything else as hccs_attention_fused.  (Masking is not in the paper, whose
 * encoder workloads are padded to a fixed length, Section "Models and tasks".)
 */
hccs_status_t hccs_attention_fused_keylen(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                          const int8_t *V, int32_t *O, const int32_t *key_len,
                                          const int32_t *requant_mult, int32_t requant_shift,
                                          int32_t B, int32_t H, int32_t L, int32_t d,
                                          uint32_t flags, void *cuda_stream);

/*
 * hccs_attention_fused with a dequantised fp32 output: O[b,h,i,:] = float(int32 accumulator) *
 * out_scale[h] (HOST float [H]; e.g. the V quantisation step divided by 255).  The integer result
 * is exact; the two fp32 roundings keep the relative error below 2^-23.  O is device float
 * [B, H, L, d]; everything else as hccs_attention_fused.  (Not in the paper.)
 */
hccs_status_t hccs_attention_fused_f32(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                       const int8_t *V, float *O, const float *out_scale,
                                       const int32_t *requant_mult, int32_t requant_shift,
                                       int32_t B, int32_t H, int32_t L, int32_t d,
                                       uint32_t flags, void *cuda_stream);

/*
 * hccs_attention_fused with an int8 output, for pipelines that stay in int8 after the attention:
 * O[b,h,i,c] = clamp((acc * out_mult[h] + 2^(out_shift-1)) >> out_shift, -128, 127), acc the int32
 * accumulator of P.V, i.e. the rounding rule of the logit requantisation applied to the output
 * (round half up, arithmetic shift, then clamp; exact: computed in 64 bits).
 *   O          device int8 [B, H, L, d]
 *   out_mult   HOST int32 [H], each in [0, 2^13);  out_shift in 1..31
 * Everything else as hccs_attention_fused.  (Not in the paper.)
 */
hccs_status_t hccs_attention_fused_i8(hccs_ctx_t *ctx, const int8_t *Q, const int8_t *K,
                                      const int8_t *V, int8_t *O, const int32_t *out_mult, int32_t out_shift,
                                      const int32_t *requant_mult, int32_t requant_shift,
                                      int32_t B, int32_t H, int32_t L, int32_t d,
                                      uint32_t flags, void *cuda_stream);

/* A bounded grid of candidates for hccs_calibrate: D = D_lo, D_lo + D_step, ... <= D_hi (clipped to
 * 1..127), S likewise (clipped to 0..127), and for each (D, S) the values B = S*D + ceil(256/n),
 * + B_step, ... <= floor(32767/n): every candidate lies in the admissible band (Eq. 11). */
typedef struct {
    int32_t D_lo, D_hi, D_step;
    int32_t S_lo, S_hi, S_step;
    int32_t B_step;
} hccs_calib_grid_t;

/*
 * Offline per-head calibration (Section "Offline Calibration", Eq. 10): scans the grid and returns,
 * for each head, the theta that minimises the mean over the head's rows of
 * KL( softmax(alpha * x) || q ), q the int16-path HCCS row renormalised to sum one (the paper
 * recommends the int16 space; the renormalisation and the logit scale alpha are readings).
 *   logits   device int8 [B, H, Lq, Lk], the calibration rows; n_design = Lk
 *   best     HOST array of H triples (output);  best_kl  HOST double [H] (output, may be NULL)
 * Ties go to the smallest (Dmax, S, B).  Needs no context.  Offline tooling: allocates and frees
 * its work space (128 * B * H * Lq * 4 bytes plus small tables) and synchronises `cuda_stream`.
 * fp64 throughout.  HCCS_ERR_CONSTRAINT when the grid holds no admissible candidate.
 */
hccs_status_t hccs_calibrate(const int8_t *logits, int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                             double alpha, const hccs_calib_grid_t *grid, hccs_head_params_t *best,
                             double *best_kl, void *cuda_stream);

/* Reads (and clears) the device status word: 0 = no kernel gave up a bounded wait.  Synchronises
 * `cuda_stream`.  Returns HCCS_ERR_DEVICE_TIMEOUT when the word was non-zero; *word (may be NULL)
 * receives it. */
hccs_status_t hccs_device_status(hccs_ctx_t *ctx, uint32_t *word, void *cuda_stream);

/*
 * Self-test of the device-side wait limits.  (The paper has no counterpart.)  Every wait of the
 * TMA-staged kernels (on a bulk copy, on a tensor-core commit) gives up after a limit of SM clock
 * cycles -- about a second in production -- sets a bit of the status word and lets the kernel return
 * instead of hanging the GPU.  This call runs that give-up path on purpose and harmlessly: one small
 * CTA waits, through the same wait routines, on a barrier that nothing will ever complete, with the
 * limit given here.
 *   mode          0: the wait of the long-row kernel (sets bit 0 of the status word);
 *                 1: the abort-flag wait of the fused kernel (sets bit 1; a second thread gives up
 *                    because it sees the flag, not because its own, longer limit ran out)
 *   limit_cycles  1 .. 10 000 000
 * Afterwards hccs_device_status returns HCCS_ERR_DEVICE_TIMEOUT once and clears the word.
 */
hccs_status_t hccs_debug_wait_timeout(hccs_ctx_t *ctx, int32_t mode, int64_t limit_cycles, void *cuda_stream);

/* The cudaError_t of the last failing CUDA call made through this context (0 = none). */
int32_t hccs_last_cuda_error(const hccs_ctx_t *ctx);

/* Static, human-readable name of a status code. */
const char *hccs_status_string(hccs_status_t status);

/* Number of kernels launched through this context since creation (for launch accounting). */
uint64_t hccs_launch_count(const hccs_ctx_t *ctx);

/*
 * hccs_forward for callers that are not allowed to allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a memory pool's or a
 * framework's allocator callback, in a process whose device memory was handed out in full at
 * start-up (a serving engine that pre-claims the whole GPU), or in a latency-critical loop where
 * an allocation (which may synchronise the whole device) cannot be tolerated.  Such a caller
 * cannot create an hccs_ctx_t, because the context allocates its parameter table.
 *
 * What it does: the same result as hccs_forward, computed by the shared-memory-staged
 * one-CTA-per-row kernel, with all of the library's working memory (the parameter table and the
 * status word that device-side waits report to) in one fixed 4.25 KB array that is part of the
 * loaded library image on every GPU.  No context, no cudaMalloc/cudaFree, no allocating library
 * call, no host-to-device copy; the tensors are the caller's.
 *   params, num_heads, n_design, out_shift   HOST table, checked exactly as hccs_params_upload
 *        does; it travels to the GPU as a kernel argument, so it may be reused or freed as soon as
 *        the call returns.  num_heads above 256 does not fit the fixed array: HCCS_ERR_UNSUPPORTED
 *   logits, probs, B, H, Lq, Lk, flags       as hccs_forward, on the CURRENT device; this entry
 *        point needs Lk % 16 == 0 and 16-byte aligned pointers (else HCCS_ERR_UNSUPPORTED)
 *   timed_out   NULL: two kernels are enqueued on `cuda_stream` (one that fills the array, then the
 *        row kernel) and the call returns without waiting for them.  Non-NULL (host): the call
 *        also synchronises `cuda_stream` and stores the status word there; non-zero returns
 *        HCCS_ERR_DEVICE_TIMEOUT as well.
 * The first call on each device looks up the device address of the fixed array
 * (cudaGetSymbolAddress); make that first call before any stream capture begins.  All calls on a
 * device share the array and it keeps the previous call's contents: each call rewrites the table
 * and clears the status word on `cuda_stream` before its row kernel.  Two calls whose work
 * overlaps on the GPU (different streams, no dependency between them) therefore race on it --
 * serialise them.
 */
hccs_status_t hccs_forward_static_scratch(const hccs_head_params_t *params, int32_t num_heads,
                                          int32_t n_design, int32_t out_shift,
                                          const int8_t *logits, void *probs,
                                          int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                                          uint32_t flags, uint32_t *timed_out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* HCCS_H */
