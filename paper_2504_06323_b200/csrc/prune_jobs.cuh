// Job descriptors shared by the per-row pruning kernels (mosaic_prune_unstructured[_batch];
// Section 4.1.3, unstructured projection pruning) and the launcher of the warp-per-row kernel.
#pragma once
#include "common.cuh"

namespace mosaic {

// One matrix to prune, as the kernels see it.  A launch works through a list of them, all with
// the same number of columns; rows are numbered across the list (row0 = first global row).
struct PruneJob {
    const uint16_t* W_in;
    uint16_t* W_out;        // or nullptr: only the keep bitmask is written
    const float* norms;
    uint8_t* mask;          // keep bitmask as bytes, or nullptr
    int64_t rows, ldw, row0;
    int k, mask_row_bytes;
};
template <int NJ>
struct PruneJobList {
    int n;
    PruneJob job[NJ];
};
constexpr int kBatchJobs = 256;   // jobs per launch of the batched kernels (the list travels as a kernel parameter)

// Row-group kernel (prune_warp.cu): bf16 rows of kWarpMinCols..kWarpMaxCols columns, cols % 8 == 0,
// 0 < k < cols for every job.  Enqueues one launch; returns a mosaic_status.
constexpr int kWarpMinCols = 2048, kWarpMaxCols = 16384;
bool prune_warp_takes(int64_t cols);   // true iff a launch shape exists for rows of this length
int launch_prune_warp(const PruneJobList<1>& jobs, int64_t total_rows, int cols, cudaStream_t st);
int launch_prune_warp(const PruneJobList<kBatchJobs>& jobs, int64_t total_rows, int cols, cudaStream_t st);

}  // namespace mosaic
