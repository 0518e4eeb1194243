// mosaic_prune_structured_compact / mosaic_rank_units: structured projection
// pruning (Section 4.1.3; Section 2.3) - unit scores, exact ranking of units,
// dense compaction.
//
//   scores : one sweep over W in tiles of 256 columns x 256 rows.  A lane owns 8
//            adjacent columns: it adds every score to its column accumulators
//            and to the row's partial sum (fp64); a row's partial over a chunk
//            is combined by a fixed butterfly, the chunks of a row in chunk
//            order, the warps' and the bands' column partials in index order.  One fp64 sum per unit over its rows / columns in
//            index order follows, rounded once to fp32.
//   rank   : one CTA per dimension; 4 x 8-bit radix select on the fp32 score
//            bits finds the threshold key and tie quota; an ordered block scan
//            then emits the ascending keep list (ties: lowest index removed
//            first).
//   compact: one CTA per output row: the source row is staged in shared memory
//            with coalesced 16-byte loads, every thread then gathers 8 output
//            elements from it through the kept-column list and stores 16 bytes.
#include "common.cuh"

namespace mosaic {

constexpr int kRankThreads = 1024;

constexpr int kSTileCols = 256;    // columns per tile: one warp row of 32 lanes x 8 columns
constexpr int kSTileRows = 256;    // rows per tile, dealt round-robin to the CTA's warps
constexpr int kSThreads = 128;
constexpr int kSWarps = kSThreads / 32;

struct StructWs {  // carve-up of the caller's workspace
    double* row_partial;  // [chunks, rows]
    double* col_partial;  // [bands, cols]
    float* scores;        // [n_ru + n_cu]
    int chunks, bands;
    size_t bytes;
};

static StructWs struct_ws(void* base, int64_t rows, int64_t cols) {
    StructWs w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.chunks = (int)((cols + kSTileCols - 1) / kSTileCols);
    w.bands = (int)((rows + kSTileRows - 1) / kSTileRows);
    w.row_partial = reinterpret_cast<double*>(p + off);
    off += align_up(sizeof(double) * (size_t)w.chunks * (size_t)rows, 256);
    w.col_partial = reinterpret_cast<double*>(p + off);
    off += align_up(sizeof(double) * (size_t)w.bands * (size_t)cols, 256);
    w.scores = reinterpret_cast<float*>(p + off);
    off += align_up(sizeof(float) * (size_t)(rows + cols), 256);
    w.bytes = off;
    return w;
}

// One tile per CTA (blockIdx.x = column chunk of 256, blockIdx.y = row band of 256).  Every warp
// covers the chunk's 256 columns (a lane owns 8 adjacent ones) and takes every fourth row of the
// band: the row's partial sum over the chunk is one butterfly away, and the lane's column
// accumulators are combined over the four warps in warp order at the end.  All sums in fp64.
template <int DT>
__global__ void __launch_bounds__(kSThreads) unit_partial_kernel(const void* __restrict__ W, int64_t rows, int64_t cols,
                                                                  int64_t ldw, const float* __restrict__ norms,
                                                                  double* __restrict__ row_partial,
                                                                  double* __restrict__ col_partial) {
    __shared__ double cp[kSWarps][kSTileCols + 2];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int64_t c0 = (int64_t)blockIdx.x * kSTileCols + lane * kVec;
    const int64_t r0 = (int64_t)blockIdx.y * kSTileRows;
    const int64_t r1 = (r0 + kSTileRows < rows) ? r0 + kSTileRows : rows;
    float nrm[kVec];
    double acc[kVec];
#pragma unroll
    for (int e = 0; e < kVec; ++e) {
        acc[e] = 0.0;
        nrm[e] = (c0 + e < cols) ? (norms ? norms[c0 + e] : 1.0f) : 0.0f;
    }
    constexpr int U = 4;   // rows in flight per warp
    for (int64_t r = r0 + wid; r < r1; r += U * kSWarps) {
        Raw8<DT> v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t rr = r + u * kSWarps;
            if (rr < r1 && c0 < cols) load_vec<DT, true>(v[u], W, rr * ldw, c0, cols);
            else v[u].clear();
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t rr = r + u * kSWarps;
            double p = 0.0;
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                const double s = (double)__fmul_rn(nrm[e], v[u].abs_f32(e));
                acc[e] += s;
                p += s;
            }
            p = warp_sum(p);
            if (lane == 0 && rr < r1) row_partial[(int64_t)blockIdx.x * rows + rr] = p;
        }
    }
#pragma unroll
    for (int e = 0; e < kVec; ++e) cp[wid][lane * kVec + e] = acc[e];
    __syncthreads();
    for (int i = threadIdx.x; i < kSTileCols; i += kSThreads) {
        const int64_t c = (int64_t)blockIdx.x * kSTileCols + i;
        if (c < cols) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < kSWarps; ++w) s += cp[w][i];
            col_partial[(int64_t)blockIdx.y * cols + c] = s;
        }
    }
}

// Unit score = fp64 sum over the unit's rows (chunk partials in chunk order) or columns (band
// partials in band order), in index order, rounded once to fp32.
__global__ void unit_score_kernel(const double* __restrict__ row_partial, int chunks, int64_t rows, int64_t n_ru,
                                  int64_t row_group, const double* __restrict__ col_partial, int bands, int64_t cols,
                                  int64_t n_cu, int64_t col_group, float* __restrict__ out, int accumulate) {
    const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= n_ru + n_cu) return;
    double s = 0.0;
    if (u < n_ru) {
        for (int64_t i = u * row_group; i < (u + 1) * row_group; ++i) {
            double rs = 0.0;
#pragma unroll 8
            for (int p = 0; p < chunks; ++p) rs += row_partial[(int64_t)p * rows + i];
            s += rs;
        }
    } else {
        const int64_t v = u - n_ru;
        for (int64_t c = v * col_group; c < (v + 1) * col_group; ++c) {
            double cs = 0.0;
#pragma unroll 16
            for (int p = 0; p < bands; ++p) cs += col_partial[(int64_t)p * cols + c];   // loads batched, adds in order
            s += cs;
        }
    }
    const float f = (float)s;
    out[u] = accumulate ? __fadd_rn(out[u], f) : f;
}

__global__ void sum_scores_kernel(float* __restrict__ dst, const float* __restrict__ src, int64_t n) {
    const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u < n) dst[u] = __fadd_rn(dst[u], src[u]);
}

__device__ __forceinline__ uint32_t unit_key(float s) { return (s != s) ? 0xFFFFFFFFu : __float_as_uint(s); }

// Keep list of one dimension: remove the (n - keep) units first under (score, index).
__device__ void rank_units_block(const float* __restrict__ scores, int64_t n, int64_t keep, int32_t* __restrict__ keep_out) {
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_tot[2][32];
    __shared__ uint32_t sel_bin, sel_rank, sel_cnt;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int64_t remove = n - keep;
    uint32_t T = 0u;
    int64_t q = 0, n_eq = 0;  // q of the n_eq units with key == T are removed
    if (remove > 0) {
        uint32_t prefix = 0u, pmask = 0u;
        int64_t rank = remove;
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (tid < 256) hist[tid] = 0u;
            __syncthreads();
            for (int64_t u = tid; u < n; u += kRankThreads) {
                const uint32_t key = unit_key(scores[u]);
                if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFFu], 1u);
            }
            __syncthreads();
            if (wid == 0) {   // warp 0: 8 bins per lane, prefix over the lanes, then inside the lane that holds the rank
                uint32_t c[8], sum = 0u;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    c[i] = hist[lane * 8 + i];
                    sum += c[i];
                }
                uint32_t incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += n;
                }
                int64_t cum = (int64_t)(incl - sum);
                if (cum < rank && rank <= cum + (int64_t)sum) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (cum < rank && rank <= cum + (int64_t)c[i]) {
                            sel_bin = (uint32_t)(lane * 8 + i);
                            sel_rank = (uint32_t)(rank - cum);
                            sel_cnt = c[i];
                        }
                        cum += c[i];
                    }
                }
            }
            __syncthreads();
            prefix |= sel_bin << shift;
            pmask |= 0xFFu << shift;
            rank = sel_rank;
            n_eq = sel_cnt;
            __syncthreads();
        }
        T = prefix;
        q = rank;
    }
    // ordered emission, 1024 units per step
    int64_t eq_before = 0, kept_before = 0;
    for (int64_t base = 0; base < n; base += kRankThreads) {
        const int64_t u = base + tid;
        uint32_t is_eq = 0u, key = 0u;
        if (u < n) {
            key = unit_key(scores[u]);
            is_eq = (remove > 0 && key == T) ? 1u : 0u;
        }
        // scan of the tie indicator
        uint32_t incl = is_eq;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_tot[0][wid] = incl;
        __syncthreads();
        uint32_t eq_excl = incl - is_eq, eq_total = 0u;
        for (int w = 0; w < kRankThreads / 32; ++w) {
            const uint32_t t = warp_tot[0][w];
            if (w < wid) eq_excl += t;
            eq_total += t;
        }
        uint32_t kept = 0u;
        if (u < n) {
            if (remove == 0) kept = 1u;
            else if (key > T) kept = 1u;
            else if (key == T) kept = (eq_before + (int64_t)eq_excl >= q) ? 1u : 0u;
        }
        uint32_t kincl = kept;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, kincl, o);
            if (lane >= o) kincl += v;
        }
        if (lane == 31) warp_tot[1][wid] = kincl;
        __syncthreads();
        uint32_t k_excl = kincl - kept, k_total = 0u;
        for (int w = 0; w < kRankThreads / 32; ++w) {
            const uint32_t t = warp_tot[1][w];
            if (w < wid) k_excl += t;
            k_total += t;
        }
        if (kept) {
            const int64_t pos = kept_before + (int64_t)k_excl;
            if (pos < keep) keep_out[pos] = (int32_t)u;
        }
        eq_before += eq_total;
        kept_before += k_total;
        __syncthreads();
    }
    (void)n_eq;
}

// blockIdx.x == 0 ranks the row units, 1 the column units (either may be skipped).
__global__ void __launch_bounds__(kRankThreads) rank_kernel(const float* row_scores, int64_t n_ru, int64_t row_keep,
                                                             int32_t* row_out, const float* col_scores, int64_t n_cu,
                                                             int64_t col_keep, int32_t* col_out) {
    if (blockIdx.x == 0) {
        if (row_out) rank_units_block(row_scores, n_ru, row_keep, row_out);
    } else {
        if (col_out) rank_units_block(col_scores, n_cu, col_keep, col_out);
    }
}

// Dense gather.  grid.x = output rows.  The source row is staged in shared memory (dynamic,
// cols elements) with 16-byte loads; threads then walk output vectors of 8 elements.
template <int DT>
__global__ void __launch_bounds__(256) compact_kernel(const void* __restrict__ W, int64_t cols, int64_t ldw,
                                                       const int32_t* __restrict__ row_keep, int64_t n_ru, int64_t row_group,
                                                       const int32_t* __restrict__ col_keep, int64_t n_cu, int64_t col_group,
                                                       int64_t out_cols, void* __restrict__ out) {
    extern __shared__ __align__(16) unsigned char srow[];
    constexpr int esz = (DT == MOSAIC_F32) ? 4 : 2;
    const int64_t a = blockIdx.x;
    int64_t ru = row_keep[a / row_group];
    ru = ru < 0 ? 0 : (ru >= n_ru ? n_ru - 1 : ru);
    const int64_t src_row = ru * row_group + a % row_group;
    const int64_t in_vec = (cols + kVec - 1) / kVec;
    for (int64_t v = threadIdx.x; v < in_vec; v += blockDim.x) {
        Raw8<DT> r;
        load_vec<DT, true>(r, W, src_row * ldw, v * kVec, cols);
        uint4* dst = reinterpret_cast<uint4*>(srow + v * kVec * esz);
        dst[0] = make_uint4(r.w[0], r.w[1], r.w[2], r.w[3]);
        if (DT == MOSAIC_F32) dst[1] = make_uint4(r.w[4 % (Raw8<DT>::kBytes / 4)], r.w[5 % (Raw8<DT>::kBytes / 4)],
                                                  r.w[6 % (Raw8<DT>::kBytes / 4)], r.w[7 % (Raw8<DT>::kBytes / 4)]);
    }
    __syncthreads();
    const int64_t nvec = (out_cols + kVec - 1) / kVec;
    const bool vec_ok = (out_cols % kVec) == 0;   // every output row then starts 16-byte aligned
    for (int64_t v = threadIdx.x; v < nvec; v += blockDim.x) {
        Raw8<DT> r;
        r.clear();
        const int64_t b0 = v * kVec;
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const int64_t b = b0 + e;
            if (b < out_cols) {
                int64_t cu = (col_group == 1) ? (int64_t)col_keep[b] : (int64_t)col_keep[b / col_group];
                cu = cu < 0 ? 0 : (cu >= n_cu ? n_cu - 1 : cu);
                const int64_t j = (col_group == 1) ? cu : cu * col_group + b % col_group;
                r.set_scalar(e, srow, j);
            }
        }
        if (vec_ok) {
            r.store((char*)out + (a * out_cols + b0) * esz);
        } else {
#pragma unroll
            for (int e = 0; e < kVec; ++e)
                if (b0 + e < out_cols) r.put_scalar(e, out, a * out_cols + b0 + e);
        }
    }
}

}  // namespace mosaic

using namespace mosaic;

extern "C" size_t mosaic_prune_structured_compact_workspace_bytes(int64_t rows, int64_t cols) {
    if (rows <= 0 || cols <= 0) return 256;
    return struct_ws(nullptr, rows, cols).bytes;
}

extern "C" int mosaic_rank_units(const float* scores, int64_t n_units, int64_t keep, int32_t* keep_out, void* stream) {
    if (!scores || (!keep_out && keep > 0)) return MOSAIC_ERR_NULL_PTR;
    if (n_units <= 0 || keep < 0 || keep > n_units || n_units > 0x7FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
    if (keep == 0) return MOSAIC_OK;
    rank_kernel<<<1, kRankThreads, 0, static_cast<cudaStream_t>(stream)>>>(scores, n_units, keep, keep_out, nullptr, 0, 0,
                                                                          nullptr);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

extern "C" int mosaic_sum_unit_scores(float* dst, const float* src, int64_t n_units, void* stream) {
    if (!dst || !src) return MOSAIC_ERR_NULL_PTR;
    if (n_units < 0) return MOSAIC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dst) & 3u) || (reinterpret_cast<uintptr_t>(src) & 3u)) return MOSAIC_ERR_MISALIGNED;
    if (dst != src && dst < src + n_units && src < dst + n_units) return MOSAIC_ERR_ALIASING;
    if (n_units == 0) return MOSAIC_OK;
    sum_scores_kernel<<<(unsigned)((n_units + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(dst, src, n_units);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

extern "C" int mosaic_prune_structured_compact(const void* W_in, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                               const float* norms, int64_t row_group, int64_t col_group,
                                               int64_t row_units_keep, int64_t col_units_keep, int32_t* row_keep_units,
                                               int32_t* col_keep_units, int flags, void* W_out, float* unit_scores_out,
                                               void* ws, size_t ws_bytes, void* stream) {
    int rc = check_matrix(W_in, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    const int known = MOSAIC_ROWS_GIVEN | MOSAIC_COLS_GIVEN | MOSAIC_RANK_ONLY | MOSAIC_SCORES_ONLY | MOSAIC_SCORES_ACCUM;
    if (rows == 0 || (flags & ~known) || row_group <= 0 || col_group <= 0 || rows % row_group || cols % col_group)
        return MOSAIC_ERR_INVALID_ARG;
    if (rows > 0x7FFFFFFF || cols > 0x7FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
    const int64_t n_ru = rows / row_group, n_cu = cols / col_group;
    const bool scores_only = flags & MOSAIC_SCORES_ONLY;
    const bool rank_only = flags & MOSAIC_RANK_ONLY;
    const bool rows_given = flags & MOSAIC_ROWS_GIVEN, cols_given = flags & MOSAIC_COLS_GIVEN;
    if ((flags & MOSAIC_SCORES_ACCUM) && !unit_scores_out) return MOSAIC_ERR_NULL_PTR;
    if (scores_only && !unit_scores_out) return MOSAIC_ERR_NULL_PTR;
    if (!scores_only) {
        if (row_units_keep < 1 || row_units_keep > n_ru || col_units_keep < 1 || col_units_keep > n_cu)
            return MOSAIC_ERR_INVALID_ARG;
        if (!row_keep_units || !col_keep_units) return MOSAIC_ERR_NULL_PTR;
        if ((reinterpret_cast<uintptr_t>(row_keep_units) & 3u) || (reinterpret_cast<uintptr_t>(col_keep_units) & 3u))
            return MOSAIC_ERR_MISALIGNED;
    }
    const bool need_scores = scores_only || unit_scores_out || !(rows_given && cols_given);
    const int64_t out_rows = row_units_keep * row_group, out_cols = col_units_keep * col_group;
    if (!scores_only && !rank_only) {
        if (!W_out) return MOSAIC_ERR_NULL_PTR;
        if (reinterpret_cast<uintptr_t>(W_out) & 15u) return MOSAIC_ERR_MISALIGNED;
        const size_t in_span = ((size_t)(rows - 1) * (size_t)ldw + (size_t)cols) * elem_size(dtype);
        const size_t out_span = (size_t)out_rows * (size_t)out_cols * elem_size(dtype);
        const char *a = static_cast<const char*>(W_in), *b = static_cast<const char*>(W_out);
        if (a < b + out_span && b < a + in_span) return MOSAIC_ERR_ALIASING;
    }
    if ((reinterpret_cast<uintptr_t>(norms) & 3u) || (reinterpret_cast<uintptr_t>(unit_scores_out) & 3u))
        return MOSAIC_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    StructWs w{};
    if (need_scores) {
        if (!ws) return MOSAIC_ERR_NULL_PTR;
        if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
        if (ws_bytes < mosaic_prune_structured_compact_workspace_bytes(rows, cols)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
        w = struct_ws(ws, rows, cols);
        dim3 grid((unsigned)w.chunks, (unsigned)w.bands);
        if (dtype == MOSAIC_BF16)
            unit_partial_kernel<MOSAIC_BF16><<<grid, kSThreads, 0, st>>>(W_in, rows, cols, ldw, norms, w.row_partial, w.col_partial);
        else
            unit_partial_kernel<MOSAIC_F32><<<grid, kSThreads, 0, st>>>(W_in, rows, cols, ldw, norms, w.row_partial, w.col_partial);
        MOSAIC_LAUNCH_CHECK();
        // with SCORES_ACCUM the running totals live in the caller's array; ranking then uses those
        float* dst = (flags & MOSAIC_SCORES_ACCUM) ? unit_scores_out : w.scores;
        const int64_t nu = n_ru + n_cu;
        unit_score_kernel<<<(unsigned)((nu + 127) / 128), 128, 0, st>>>(w.row_partial, w.chunks, rows, n_ru, row_group,
                                                                       w.col_partial, w.bands, cols, n_cu, col_group, dst,
                                                                       (flags & MOSAIC_SCORES_ACCUM) ? 1 : 0);
        MOSAIC_LAUNCH_CHECK();
        if (unit_scores_out && dst != unit_scores_out)
            MOSAIC_CUDA_TRY(cudaMemcpyAsync(unit_scores_out, dst, sizeof(float) * (size_t)nu, cudaMemcpyDeviceToDevice, st));
        w.scores = dst;
    }
    if (scores_only) return MOSAIC_OK;

    if (!(rows_given && cols_given)) {
        rank_kernel<<<2, kRankThreads, 0, st>>>(w.scores, n_ru, row_units_keep, rows_given ? nullptr : row_keep_units,
                                                w.scores + n_ru, n_cu, col_units_keep, cols_given ? nullptr : col_keep_units);
        MOSAIC_LAUNCH_CHECK();
    }
    if (rank_only) return MOSAIC_OK;

    const size_t row_smem = align_up((size_t)((cols + kVec - 1) / kVec * kVec) * elem_size(dtype), 16);
    if (row_smem > 200 * 1024) return MOSAIC_ERR_INVALID_ARG;   // a source row must fit in shared memory (cols <= 51200 fp32)
    static DeviceCache attr_set[2];   // the opt-in belongs to one device's copy of the kernel
    const int opted = attr_set[dtype == MOSAIC_BF16].get([&]() -> int {
        const cudaError_t e = (dtype == MOSAIC_BF16)
            ? cudaFuncSetAttribute(compact_kernel<MOSAIC_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
            : cudaFuncSetAttribute(compact_kernel<MOSAIC_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) (void)cudaGetLastError();
        return e == cudaSuccess ? 1 : -1;
    });
    if (opted < 0) return MOSAIC_ERR_CUDA;
    if (dtype == MOSAIC_BF16)
        compact_kernel<MOSAIC_BF16><<<(unsigned)out_rows, 256, row_smem, st>>>(W_in, cols, ldw, row_keep_units, n_ru, row_group,
                                                                              col_keep_units, n_cu, col_group, out_cols, W_out);
    else
        compact_kernel<MOSAIC_F32><<<(unsigned)out_rows, 256, row_smem, st>>>(W_in, cols, ldw, row_keep_units, n_ru, row_group,
                                                                             col_keep_units, n_cu, col_group, out_cols, W_out);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}
