// mosaic_act_norms: per-input-channel sum of squares of the calibration
// activations, accumulated in fp64, and the fp32 l2 norm (the ||A||_2 term of
// Eq. 5).
#include "colreduce.cuh"

namespace mosaic {

// Stage 2: add the split partials of each column to the caller's accumulator, and optionally
// finalise norm = (float) sqrt(sumsq).  A CTA covers 32 columns with 8 lanes of threads per
// column: lane g adds the partials g, g+8, ... in that order (all its loads in flight at once),
// then the 8 lane sums are added in lane order.  The order is fixed, so the result does not
// depend on the launch.
constexpr int kFinCols = 32, kFinLanes = 8;
__global__ void __launch_bounds__(kFinCols * kFinLanes) act_finish_kernel(const double* __restrict__ partial, int splits,
                                                                            int64_t cols, double* __restrict__ sumsq,
                                                                            float* __restrict__ norms_out, int reset) {
    __shared__ double sm[kFinLanes][kFinCols + 1];
    const int cl = threadIdx.x % kFinCols, g = threadIdx.x / kFinCols;
    const int64_t c = (int64_t)blockIdx.x * kFinCols + cl;
    double s = 0.0;
    if (c < cols) {
#pragma unroll 8
        for (int p = g; p < splits; p += kFinLanes) s += partial[(int64_t)p * cols + c];
    }
    sm[g][cl] = s;
    __syncthreads();
    if (g == 0 && c < cols) {
        double t = reset ? 0.0 : sumsq[c];
#pragma unroll
        for (int r = 0; r < kFinLanes; ++r) t += sm[r][cl];
        sumsq[c] = t;
        if (norms_out) norms_out[c] = (float)sqrt(t);
    }
}

}  // namespace mosaic

using namespace mosaic;

extern "C" size_t mosaic_act_norms_workspace_bytes(int64_t tokens, int64_t cols) {
    if (tokens <= 0 || cols <= 0) return 256;
    const ColSplit p = col_split_plan(tokens, cols);
    return align_up((size_t)p.splits * (size_t)cols * sizeof(double), 256);
}

extern "C" int mosaic_act_norms(const void* X, int64_t tokens, int64_t cols, int64_t ldx, int dtype,
                                double* sumsq_accum, float* norms_out, int flags, void* ws, size_t ws_bytes,
                                void* stream) {
    if (dtype != MOSAIC_F32 && dtype != MOSAIC_BF16) return MOSAIC_ERR_BAD_DTYPE;
    if (tokens < 0 || cols <= 0 || (flags & ~MOSAIC_RESET_ACCUM)) return MOSAIC_ERR_INVALID_ARG;
    if (sumsq_accum == nullptr) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(sumsq_accum) & 7u) || (reinterpret_cast<uintptr_t>(norms_out) & 3u))
        return MOSAIC_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int splits = 0;
    if (tokens > 0) {
        int rc = check_matrix(X, tokens, cols, ldx, dtype);
        if (rc != MOSAIC_OK) return rc;
        if (ws == nullptr) return MOSAIC_ERR_NULL_PTR;
        if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
        if (ws_bytes < mosaic_act_norms_workspace_bytes(tokens, cols)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
        const ColSplit p = col_split_plan(tokens, cols);
        splits = p.splits;
        dim3 grid((unsigned)((cols + kColTile - 1) / kColTile), (unsigned)p.splits);
        if (dtype == MOSAIC_BF16)
            col_partial_kernel<MOSAIC_BF16><<<grid, kColTile, 0, st>>>(X, tokens, cols, ldx, p.rows_per_split,
                                                                       static_cast<double*>(ws));
        else
            col_partial_kernel<MOSAIC_F32><<<grid, kColTile, 0, st>>>(X, tokens, cols, ldx, p.rows_per_split,
                                                                      static_cast<double*>(ws));
        MOSAIC_LAUNCH_CHECK();
    }
    act_finish_kernel<<<(unsigned)((cols + kFinCols - 1) / kFinCols), kFinCols * kFinLanes, 0, st>>>(
        static_cast<const double*>(ws), splits, cols, sumsq_accum, norms_out, (flags & MOSAIC_RESET_ACCUM) ? 1 : 0);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}
