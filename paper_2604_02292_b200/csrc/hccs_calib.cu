// Offline per-head calibration (paper Section "Offline Calibration", Eq. 10): grid scan of
// theta = (B, S, Dmax) inside the admissible band, minimising the mean KL divergence between
// softmax(alpha * x) and the HCCS distribution of the int16 output path over a set of rows.
//
// Readings (the paper fixes neither): the integer row is renormalised to sum one, so the
// reciprocal cancels and q_j = s_j / Z exactly; the softmax is taken of alpha * x.  Then
//     KL = sum_j sm_j log sm_j  -  sum_j sm_j log s_j  +  log Z,
// and because s depends on a logit only through its distance delta = m - x_j (Eq. 2, Eq. 3), a
// row enters the scan only through
//     w[delta]  = softmax mass at distance delta   (256 bins, summed over the rows of a head),
//     T(D)      = sum_j min(delta_j, D)             (one integer per row and clamp bound D),
// since Z = n*B - S*T(D).  Kernel 1 makes these once; kernel 2 evaluates every candidate from
// them in fp64: 256 logs for the middle term and one log per row for the last.
// The scan is deterministic up to the order of the fp64 atomic adds in kernel 1.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <vector>

#include "hccs.h"
#include "hccs_internal.h"

namespace hccs {

namespace {

constexpr int kMaxD = 127;

// ---- kernel 1: one warp per row
__global__ void __launch_bounds__(256) calib_rows_kernel(const int8_t *__restrict__ x_all, int rows, int H, int Lq,
                                                         int Lk, double alpha, double *W /* [H][256] */,
                                                         double *negH /* [H] */, int32_t *T /* [H][128][rows_h] */,
                                                         int rows_h) {
    __shared__ double w_hist[8][256];
    __shared__ int c_hist[8][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = blockIdx.x * 8 + warp; r < rows; r += gridDim.x * 8) {
        const int bh = r / Lq, i = r - bh * Lq, b = bh / H, h = bh - b * H;
        const int rh = b * Lq + i;                                   // index of the row inside its head
        const int8_t *x = x_all + (int64_t)r * Lk;
        for (int d = lane; d < 256; d += 32) { w_hist[warp][d] = 0.0; c_hist[warp][d] = 0; }
        int m = -128;
        for (int j = lane; j < Lk; j += 32) m = max(m, (int)x[j]);
        for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        double se = 0.0;
        for (int j = lane; j < Lk; j += 32) se += exp(alpha * (double)((int)x[j] - m));
        for (int o = 16; o; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const double lse = log(se);
        __syncwarp();
        double nh = 0.0;
        for (int j = lane; j < Lk; j += 32) {
            const int delta = m - (int)x[j];
            const double lg = -alpha * (double)delta - lse;          // log softmax_j
            const double sm = exp(lg);
            nh += sm * lg;
            atomicAdd(&w_hist[warp][delta], sm);
            atomicAdd(&c_hist[warp][delta], 1);
        }
        for (int o = 16; o; o >>= 1) nh += __shfl_xor_sync(0xffffffffu, nh, o);
        __syncwarp();
        if (lane == 0) atomicAdd(&negH[h], nh);
        for (int d = lane; d < 256; d += 32)
            if (c_hist[warp][d]) atomicAdd(&W[h * 256 + d], w_hist[warp][d]);
        // T(D) = sum_delta count[delta] * min(delta, D)
        for (int D = 1 + lane; D <= kMaxD; D += 32) {
            int t = 0;
            for (int d = 1; d < 256; ++d) t += c_hist[warp][d] * min(d, D);
            T[((int64_t)h * 128 + D) * rows_h + rh] = t;
        }
        __syncwarp();
    }
}

struct Pair { int32_t D, S, B0, nB; };   // candidates B0, B0 + step, ... (nB of them) for one (D, S)

// ---- kernel 2: one CTA per (pair, head)
__global__ void __launch_bounds__(256) calib_scan_kernel(const Pair *pairs, const double *W, const double *negH,
                                                         const int32_t *T, int rows_h, int n, int B_step,
                                                         double *best_val /* [H][pairs] */,
                                                         int32_t *best_B /* [H][pairs] */) {
    __shared__ double red[8];
    __shared__ double w_sh[256];
    const Pair pr = pairs[blockIdx.x];
    const int h = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    w_sh[tid] = W[h * 256 + tid];
    __syncthreads();
    const int32_t *Trow = T + ((int64_t)h * 128 + pr.D) * rows_h;
    const double w_mine = w_sh[tid];
    const int dmin = min(tid, pr.D);
    double bestv = INFINITY;
    int bestb = -1;
    for (int k = 0; k < pr.nB; ++k) {
        const int B = pr.B0 + k * B_step;
        double acc = 0.0;
        if (w_mine != 0.0) acc -= w_mine * log((double)(B - pr.S * dmin));
        for (int r = tid; r < rows_h; r += 256) acc += log((double)(n * B - pr.S * Trow[r]));
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        __syncthreads();
        if (lane == 0) red[warp] = acc;
        __syncthreads();
        if (tid == 0) {
            double tot = negH[h];
            for (int w = 0; w < 8; ++w) tot += red[w];
            tot /= (double)rows_h;
            if (tot < bestv) { bestv = tot; bestb = B; }
        }
    }
    if (tid == 0) {
        best_val[(int64_t)h * gridDim.x + blockIdx.x] = bestv;
        best_B[(int64_t)h * gridDim.x + blockIdx.x] = bestb;
    }
}

}  // namespace

}  // namespace hccs

extern "C" hccs_status_t hccs_calibrate(const int8_t *logits, int32_t B, int32_t H, int32_t Lq, int32_t Lk,
                                        double alpha, const hccs_calib_grid_t *grid, hccs_head_params_t *best,
                                        double *best_kl, void *cuda_stream) {
    using namespace hccs;
    if (!logits || !grid || !best || B < 1 || H < 1 || Lq < 1 || Lk < 1) return HCCS_ERR_INVALID_ARG;
    if (Lk > 32767 || !(alpha > 0.0)) return HCCS_ERR_INVALID_ARG;
    if (grid->D_step < 1 || grid->S_step < 1 || grid->B_step < 1) return HCCS_ERR_INVALID_ARG;
    const int64_t rows = (int64_t)B * H * Lq;
    if (rows >= (1ll << 31)) return HCCS_ERR_UNSUPPORTED;
    const int n = Lk, f = (256 + n - 1) / n, bmax = 32767 / n;
    // the (D, S) pairs of the grid, lexicographic; B runs inside the scan kernel
    std::vector<Pair> pairs;
    for (int D = grid->D_lo < 1 ? 1 : grid->D_lo; D <= (grid->D_hi > kMaxD ? kMaxD : grid->D_hi); D += grid->D_step)
        for (int S = grid->S_lo < 0 ? 0 : grid->S_lo; S <= (grid->S_hi > 127 ? 127 : grid->S_hi); S += grid->S_step) {
            const int B0 = S * D + f;
            if (B0 > bmax) continue;
            pairs.push_back(Pair{D, S, B0, (bmax - B0) / grid->B_step + 1});
        }
    if (pairs.empty()) return HCCS_ERR_CONSTRAINT;             // no admissible candidate in the grid
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int rows_h = B * Lq;
    const size_t nP = pairs.size();
    double *dW = nullptr, *dNegH = nullptr, *dBestV = nullptr;
    int32_t *dT = nullptr, *dBestB = nullptr;
    Pair *dPairs = nullptr;
    cudaError_t e = cudaMalloc(&dW, sizeof(double) * 256 * H);
    if (e == cudaSuccess) e = cudaMalloc(&dNegH, sizeof(double) * H);
    if (e == cudaSuccess) e = cudaMalloc(&dT, sizeof(int32_t) * 128 * (size_t)H * rows_h);
    if (e == cudaSuccess) e = cudaMalloc(&dPairs, sizeof(Pair) * nP);
    if (e == cudaSuccess) e = cudaMalloc(&dBestV, sizeof(double) * nP * H);
    if (e == cudaSuccess) e = cudaMalloc(&dBestB, sizeof(int32_t) * nP * H);
    std::vector<double> hV(nP * H);
    std::vector<int32_t> hB(nP * H);
    if (e == cudaSuccess) e = cudaMemsetAsync(dW, 0, sizeof(double) * 256 * H, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(dNegH, 0, sizeof(double) * H, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dPairs, pairs.data(), sizeof(Pair) * nP, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        int blocks = (int)((rows + 7) / 8);
        if (blocks > 148 * 16) blocks = 148 * 16;
        calib_rows_kernel<<<blocks, 256, 0, st>>>(logits, (int)rows, H, Lq, Lk, alpha, dW, dNegH, dT, rows_h);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) {
        calib_scan_kernel<<<dim3((unsigned)nP, (unsigned)H), 256, 0, st>>>(dPairs, dW, dNegH, dT, rows_h, n, grid->B_step,
                                                                         dBestV, dBestB);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(hV.data(), dBestV, sizeof(double) * nP * H, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(hB.data(), dBestB, sizeof(int32_t) * nP * H, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(dW); cudaFree(dNegH); cudaFree(dT); cudaFree(dPairs); cudaFree(dBestV); cudaFree(dBestB);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return HCCS_ERR_CUDA; }
    for (int h = 0; h < H; ++h) {
        size_t arg = 0;
        for (size_t p = 1; p < nP; ++p)
            if (hV[h * nP + p] < hV[h * nP + arg]) arg = p;          // first minimum: smallest (D, S, B)
        best[h].B = hB[h * nP + arg];
        best[h].S = pairs[arg].S;
        best[h].Dmax = pairs[arg].D;
        if (best_kl) best_kl[h] = hV[h * nP + arg];
    }
    return HCCS_OK;
}
