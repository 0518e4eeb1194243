// Column-wise fp64 reduction over the rows of a row-major matrix, in two
// deterministic stages:
//   stage 1: grid (column tiles of 256) x (row splits).  A CTA is 32 column
//            lanes x 8 row lanes; a thread owns 8 adjacent columns (one 16-byte
//            load of bf16) and walks its rows in order, 4 loads in flight.
//            The 8 row lanes are combined in shared memory in lane order and
//            one fp64 partial per (split, column) is written.
//   stage 2: the caller adds the partials of a column in split order.
// The value reduced is x^2 (activation norms, Eq. 5's ||A||_2 term).
#pragma once
#include "common.cuh"

namespace mosaic {

constexpr int kColTile = 256;   // columns per CTA
constexpr int kRowLanes = 8;    // row lanes per CTA
constexpr int kColUnroll = 4;   // rows in flight per thread

struct ColSplit {
    int splits;          // number of row splits (gridDim.y)
    int rows_per_split;  // multiple of kRowLanes * kColUnroll
};

inline ColSplit col_split_plan(int64_t rows, int64_t cols) {
    const int64_t tiles = (cols + kColTile - 1) / kColTile;
    const int64_t target = (int64_t)sm_count() * 16;
    const int64_t quantum = kRowLanes * kColUnroll;
    int64_t splits = target / tiles;
    if (splits < 1) splits = 1;
    const int64_t max_splits = (rows + 2 * quantum - 1) / (2 * quantum);  // >= 64 rows per split
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    if (splits > 65535) splits = 65535;
    int64_t rps = (rows + splits - 1) / splits;
    rps = (rps + quantum - 1) / quantum * quantum;
    if (rps < quantum) rps = quantum;
    ColSplit p;
    p.rows_per_split = (int)rps;
    p.splits = (int)((rows + rps - 1) / rps);
    if (p.splits < 1) p.splits = 1;
    return p;
}

#ifdef __CUDACC__

template <int DT>
__device__ __forceinline__ void col_accumulate(double (&acc)[kVec], const Raw8<DT>& r) {
#pragma unroll
    for (int e = 0; e < kVec; ++e) {
        const double x = (double)r.f32(e);
        acc[e] = fma(x, x, acc[e]);           // exact product, one rounding in the add
    }
}

template <int DT>
__global__ void __launch_bounds__(kColTile) col_partial_kernel(const void* __restrict__ M, int64_t rows, int64_t cols,
                                                                int64_t ld, int rows_per_split,
                                                                double* __restrict__ partial) {
    __shared__ double sm[kRowLanes][kColTile + 2];
    const int cl = threadIdx.x & 31, rl = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kColTile + cl * kVec;
    const int64_t t0 = (int64_t)blockIdx.y * rows_per_split;
    const int64_t t1 = (t0 + rows_per_split < rows) ? t0 + rows_per_split : rows;

    double acc[kVec];
#pragma unroll
    for (int e = 0; e < kVec; ++e) acc[e] = 0.0;

    if (c0 < cols) {
        int64_t t = t0 + rl;
        for (; t + (kColUnroll - 1) * kRowLanes < t1; t += kColUnroll * kRowLanes) {
            Raw8<DT> r[kColUnroll];
#pragma unroll
            for (int u = 0; u < kColUnroll; ++u) load_vec<DT, true>(r[u], M, (t + u * kRowLanes) * ld, c0, cols);
#pragma unroll
            for (int u = 0; u < kColUnroll; ++u) col_accumulate<DT>(acc, r[u]);
        }
        for (; t < t1; t += kRowLanes) {
            Raw8<DT> r;
            load_vec<DT, true>(r, M, t * ld, c0, cols);
            col_accumulate<DT>(acc, r);
        }
    }
#pragma unroll
    for (int e = 0; e < kVec; ++e) sm[rl][cl * kVec + e] = acc[e];
    __syncthreads();
    const int64_t c = (int64_t)blockIdx.x * kColTile + threadIdx.x;
    if (c < cols) {
        double s = 0.0;
#pragma unroll
        for (int r = 0; r < kRowLanes; ++r) s += sm[r][threadIdx.x];
        partial[(int64_t)blockIdx.y * cols + c] = s;
    }
}

#endif  // __CUDACC__
}  // namespace mosaic
