// Structured projection pruning (Section 4.1.3: remove the lowest-magnitude heads and channels;
// Section 2.3: structured pruning leaves smaller dense matrices): unit scores, exact ranking of
// units, dense compaction - as single calls and as batched calls that take a host list of
// matrices and do each step for all of them in one launch (a model has N*M projections; one
// launch chain per projection is bound by launch latency and by the host).
//
//   scores : one sweep over W in tiles of 256 columns x 256 rows.  A warp covers the tile's 256
//            columns (a lane owns 8 adjacent ones) and takes every fourth row: every score goes to
//            the lane's column accumulators and to the row's partial sum (fp64); a row's partial
//            over the tile is the lanes' sums added in lane order (through shared memory), the tiles
//            of a row in column order, the warps' and the row bands' column partials in index order
//            (one thread per row / column).  One fp64 sum per unit over its rows / columns in
//            index order follows, rounded once to fp32.  Nothing depends on the launch shape.
//   rank   : one CTA per list of units; 4 x 8-bit radix select on the fp32 score bits finds the
//            threshold key and tie quota; an ordered block scan then emits the ascending keep
//            list (ties: lowest index removed first).
//   compact: CTAs walk the output rows of all matrices.  Kept columns that come in whole 16-byte
//            vectors (every column kept, or column units of a multiple of 8 columns) are copied
//            vector by vector straight from global memory; otherwise the source row is staged in
//            shared memory and gathered through the kept-column list.
#include <memory>
#include <new>

#include "common.cuh"

namespace mosaic {

constexpr int kRankThreads = 1024;
constexpr int kSTileCols = 256;    // columns per tile: a warp row of 32 lanes x 8 columns
constexpr int kSTileRows = 256;    // rows per tile, dealt round-robin to the CTA's warps
constexpr int kSSubRows = 64;      // rows whose lane sums wait in shared memory for the per-row addition
constexpr int kSThreads = 128;
constexpr int kSWarps = kSThreads / 32;
constexpr int kStructBatch = 128;  // matrices per launch (the list travels as a kernel parameter)

struct ScoreJob {
    const void* W;
    const float* norms;    // or nullptr: norm = 1
    double* row_partial;   // [chunks, rows]
    double* col_partial;   // [bands, cols]
    float* row_out;        // [rows / row_group] or nullptr
    float* col_out;        // [cols / col_group] or nullptr
    int64_t rows, cols, ldw, row_group, col_group;
    int64_t unit0;         // first global unit (row units, then column units)
    int64_t line0;         // first global line (rows, then columns)
    int tile0, chunks, bands, accumulate;
};
template <int NJ>
struct ScoreJobList {
    int n;
    ScoreJob job[NJ];
};
struct RankJob {
    const float* scores;
    int32_t* keep_out;
    int64_t n_units, keep;
};
template <int NJ>
struct RankJobList {
    int n;
    RankJob job[NJ];
};
struct AddJob {
    float* dst;
    const float* a;
    const float* b;
    int64_t n, item0;
};
template <int NJ>
struct AddJobList {
    int n;
    AddJob job[NJ];
};
struct CompactJob {
    const void* W_in;
    void* W_out;
    const int32_t* row_keep;
    const int32_t* col_keep;
    int64_t cols, ldw, n_ru, row_group, n_cu, col_group, out_rows, out_cols, out_row0;
};
template <int NJ>
struct CompactJobList {
    int n;
    CompactJob job[NJ];
};

static void score_shape(int64_t rows, int64_t cols, int* chunks, int* bands) {
    *chunks = (int)((cols + kSTileCols - 1) / kSTileCols);
    *bands = (int)((rows + kSTileRows - 1) / kSTileRows);
}
// Scratch of one matrix: row partials [chunks, rows], column partials [bands, cols], 256-byte aligned.
static size_t score_ws_bytes(int64_t rows, int64_t cols) {
    int chunks, bands;
    score_shape(rows, cols, &chunks, &bands);
    return align_up(sizeof(double) * (size_t)chunks * (size_t)rows, 256) + align_up(sizeof(double) * (size_t)bands * (size_t)cols, 256);
}

// Index of the job whose [first, next first) range holds x: first(i) is ascending.
template <class F>
__device__ __forceinline__ int find_job(int n, int64_t x, F first) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (first(mid) <= x) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

// One tile per CTA.  All sums in fp64.  The tile's rows are worked through in sub-tiles of 64: a
// lane adds the 8 scores of its vector of a row into its column accumulators and leaves their sum
// in shared memory; after the sub-tile one thread per row adds the 32 lane sums in lane order.
template <int DT, int NJ>
__global__ void __launch_bounds__(kSThreads, 6) unit_partial_kernel(const __grid_constant__ ScoreJobList<NJ> jobs) {
    __shared__ double cp[kSWarps][kSTileCols + 2];
    __shared__ double rowbuf[32][kSSubRows + 1];   // [lane][row of the sub-tile]
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int tile = blockIdx.x;
    const ScoreJob& J = jobs.job[find_job(jobs.n, tile, [&](int i) { return (int64_t)jobs.job[i].tile0; })];
    const int local = tile - J.tile0;
    const int chunk = local % J.chunks, band = local / J.chunks;
    const int64_t rows = J.rows, cols = J.cols, ldw = J.ldw;
    const int64_t c0 = (int64_t)chunk * kSTileCols + lane * kVec;
    const int64_t r0 = (int64_t)band * kSTileRows;
    const int64_t r1 = (r0 + kSTileRows < rows) ? r0 + kSTileRows : rows;
    float nrm[kVec];
    double acc[kVec];
#pragma unroll
    for (int e = 0; e < kVec; ++e) {
        acc[e] = 0.0;
        nrm[e] = (c0 + e < cols) ? (J.norms ? J.norms[c0 + e] : 1.0f) : 0.0f;
    }
    constexpr int U = 4;   // rows in flight per warp
    // bf16 rows of whole vectors: the same sums in the same order with plain pointer stepping
    const bool lean = DT == MOSAIC_BF16 && (cols % kVec) == 0;
    for (int64_t rs = r0; rs < r1; rs += kSSubRows) {
        if (lean) {
            const int n_sub = (int)(r1 - rs < kSSubRows ? r1 - rs : kSSubRows);
            const bool lane_in = c0 < cols;
            const size_t stride = (size_t)ldw * 2u;
            const char* base = static_cast<const char*>(J.W) + ((size_t)rs * (size_t)ldw + (size_t)(lane_in ? c0 : 0)) * 2u;
#pragma unroll 1
            for (int i = wid; i < kSSubRows; i += U * kSWarps) {
                uint4 v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = i + u * kSWarps;
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (lane_in && r < n_sub) v[u] = ld_stream16_ro(base + (size_t)r * stride);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    double p = 0.0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const double s0 = (double)__fmul_rn(nrm[2 * q], fabsf(__uint_as_float(w[q] << 16)));
                        acc[2 * q] += s0;
                        p += s0;
                        const double s1 = (double)__fmul_rn(nrm[2 * q + 1], fabsf(__uint_as_float(w[q] & 0xFFFF0000u)));
                        acc[2 * q + 1] += s1;
                        p += s1;
                    }
                    rowbuf[lane][i + u * kSWarps] = p;
                }
            }
        } else
#pragma unroll 1
        for (int i = wid; i < kSSubRows; i += U * kSWarps) {
            Raw8<DT> v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t rr = rs + i + u * kSWarps;
                if (rr < r1 && c0 < cols) load_vec<DT, true>(v[u], J.W, rr * ldw, c0, cols);
                else v[u].clear();
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                double p = 0.0;
#pragma unroll
                for (int e = 0; e < kVec; ++e) {
                    const double s = (double)__fmul_rn(nrm[e], v[u].abs_f32(e));
                    acc[e] += s;
                    p += s;
                }
                rowbuf[lane][i + u * kSWarps] = p;
            }
        }
        __syncthreads();
        if (threadIdx.x < kSSubRows && rs + threadIdx.x < r1) {
            double s = 0.0;
#pragma unroll
            for (int l = 0; l < 32; ++l) s += rowbuf[l][threadIdx.x];
            J.row_partial[(int64_t)chunk * rows + rs + threadIdx.x] = s;
        }
        __syncthreads();
    }
#pragma unroll
    for (int e = 0; e < kVec; ++e) cp[wid][lane * kVec + e] = acc[e];
    __syncthreads();
    for (int i = threadIdx.x; i < kSTileCols; i += kSThreads) {
        const int64_t c = (int64_t)chunk * kSTileCols + i;
        if (c < cols) {
            double s = 0.0;
#pragma unroll
            for (int w = 0; w < kSWarps; ++w) s += cp[w][i];
            J.col_partial[(int64_t)band * cols + c] = s;
        }
    }
}

// Line sums: for every row the fp64 sum of its tile partials in column order, for every column
// the sum of its band partials in band order, written over the first partial of the line.  One
// thread per line (row lines first, then column lines) of the list.
template <int NJ>
__global__ void line_sum_kernel(const __grid_constant__ ScoreJobList<NJ> jobs, int64_t total_lines) {
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total_lines) return;
    const ScoreJob& J = jobs.job[find_job(jobs.n, g, [&](int i) { return jobs.job[i].line0; })];
    const int64_t l = g - J.line0;
    if (l < J.rows) {
        if (J.row_out == nullptr) return;
        double rs = 0.0;
#pragma unroll 8
        for (int p = 0; p < J.chunks; ++p) rs += J.row_partial[(int64_t)p * J.rows + l];
        J.row_partial[l] = rs;
    } else {
        if (J.col_out == nullptr) return;
        const int64_t c = l - J.rows;
        double cs = 0.0;
#pragma unroll 16
        for (int p = 0; p < J.bands; ++p) cs += J.col_partial[(int64_t)p * J.cols + c];   // loads batched, adds in order
        J.col_partial[c] = cs;
    }
}

// Unit score = fp64 sum of the unit's line sums in index order, rounded once to fp32.  One thread
// per unit of the list.
template <int NJ>
__global__ void unit_score_kernel(const __grid_constant__ ScoreJobList<NJ> jobs, int64_t total_units) {
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total_units) return;
    const ScoreJob& J = jobs.job[find_job(jobs.n, g, [&](int i) { return jobs.job[i].unit0; })];
    const int64_t u = g - J.unit0, n_ru = J.rows / J.row_group;
    double s = 0.0;
    float* out;
    if (u < n_ru) {
        if (J.row_out == nullptr) return;
#pragma unroll 8
        for (int64_t i = u * J.row_group; i < (u + 1) * J.row_group; ++i) s += J.row_partial[i];
        out = J.row_out + u;
    } else {
        if (J.col_out == nullptr) return;
        const int64_t v = u - n_ru;
#pragma unroll 8
        for (int64_t c = v * J.col_group; c < (v + 1) * J.col_group; ++c) s += J.col_partial[c];
        out = J.col_out + v;
    }
    const float f = (float)s;
    *out = J.accumulate ? __fadd_rn(*out, f) : f;
}

// dst[u] = fl32(a[u] + b[u]) for every item of the list (items must not write what another reads).
template <int NJ>
__global__ void add_scores_kernel(const __grid_constant__ AddJobList<NJ> jobs, int64_t total) {
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= total) return;
    const AddJob& J = jobs.job[find_job(jobs.n, g, [&](int i) { return jobs.job[i].item0; })];
    const int64_t u = g - J.item0;
    J.dst[u] = __fadd_rn(J.a[u], J.b[u]);
}

__device__ __forceinline__ uint32_t unit_key(float s) { return (s != s) ? 0xFFFFFFFFu : __float_as_uint(s); }

// Keep list of one dimension: remove the (n - keep) units first under (score, index).
__device__ void rank_units_block(const float* __restrict__ scores, int64_t n, int64_t keep, int32_t* __restrict__ keep_out) {
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_tot[2][32];
    __shared__ uint32_t sel_bin, sel_rank;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int64_t remove = n - keep;
    uint32_t T = 0u;
    int64_t q = 0;   // q of the units with key == T are removed
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
                    const uint32_t nn = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += nn;
                }
                int64_t cum = (int64_t)(incl - sum);
                if (cum < rank && rank <= cum + (int64_t)sum) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (cum < rank && rank <= cum + (int64_t)c[i]) {
                            sel_bin = (uint32_t)(lane * 8 + i);
                            sel_rank = (uint32_t)(rank - cum);
                        }
                        cum += c[i];
                    }
                }
            }
            __syncthreads();
            prefix |= sel_bin << shift;
            pmask |= 0xFFu << shift;
            rank = sel_rank;
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
        uint32_t incl = is_eq;   // scan of the tie indicator
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
}

// One CTA per list.
template <int NJ>
__global__ void __launch_bounds__(kRankThreads) rank_kernel(const __grid_constant__ RankJobList<NJ> jobs) {
    const RankJob& J = jobs.job[blockIdx.x];
    if (J.keep_out != nullptr && J.keep > 0) rank_units_block(J.scores, J.n_units, J.keep, J.keep_out);
}

__device__ __forceinline__ int64_t clamp_unit(int64_t u, int64_t n) { return u < 0 ? 0 : (u >= n ? n - 1 : u); }

// Dense gather.  CTAs walk the output rows of all jobs (grid-stride).  Dynamic shared memory: one
// source row of the widest job that needs staging (0 if none does).
template <int DT, int NJ>
__global__ void __launch_bounds__(256) compact_kernel(const __grid_constant__ CompactJobList<NJ> jobs, int64_t total_out_rows) {
    extern __shared__ __align__(16) unsigned char srow[];
    constexpr int esz = (DT == MOSAIC_F32) ? 4 : 2;
    int job = 0;   // a CTA's rows ascend, so its job index only moves forward
    for (int64_t g = blockIdx.x; g < total_out_rows; g += gridDim.x) {
        while (job + 1 < jobs.n && jobs.job[job + 1].out_row0 <= g) ++job;
        const CompactJob& J = jobs.job[job];
        const int64_t a = g - J.out_row0;
        // (rows < 2^31: 32-bit division, and none at all for single rows)
        const uint32_t rg = (uint32_t)J.row_group, a_unit = rg == 1u ? (uint32_t)a : (uint32_t)a / rg, a_in = rg == 1u ? 0u : (uint32_t)a % rg;
        const int64_t src_row = clamp_unit(J.row_keep[a_unit], J.n_ru) * J.row_group + a_in;
        const int64_t cols = J.cols, out_cols = J.out_cols, col_group = J.col_group;
        const char* src = static_cast<const char*>(J.W_in) + (size_t)src_row * (size_t)J.ldw * esz;
        char* dst = static_cast<char*>(J.W_out) + (size_t)a * (size_t)out_cols * esz;
        const bool vec_units = (col_group % kVec) == 0 || (J.out_cols == cols && col_group == 1);   // (block-uniform)
        if (vec_units) {
            // every output vector of 8 elements is 8 adjacent source columns inside one kept unit
            // (all columns kept: the keep list is 0, 1, 2, ... and the row is copied as it is)
            const int64_t nvec = out_cols / kVec;
            const bool dst_aligned = (out_cols % kVec) == 0;   // else only a whole-row copy with a ragged width gets here
            if (dst_aligned) {
                const uint32_t cg = (uint32_t)col_group;   // (columns < 2^31: 32-bit division)
                for (int v = threadIdx.x; v < (int)nvec; v += blockDim.x) {
                    const uint32_t b0 = (uint32_t)v * kVec;
                    const int64_t j0 = (cg == 1u) ? (int64_t)b0 : clamp_unit(J.col_keep[b0 / cg], J.n_cu) * col_group + b0 % cg;
                    Raw8<DT> r;
                    r.template load<true>(src + j0 * esz);
                    r.store(dst + (size_t)b0 * esz);
                }
            } else {
                for (int64_t b = threadIdx.x; b < out_cols; b += blockDim.x) {
                    Raw8<DT> r;
                    r.set_scalar(0, src, b);
                    r.put_scalar(0, dst, b);
                }
            }
            continue;
        }
        __syncthreads();   // the previous row's gather is done with the staging buffer
        const int64_t in_vec = (cols + kVec - 1) / kVec;
        for (int64_t v = threadIdx.x; v < in_vec; v += blockDim.x) {
            Raw8<DT> r;
            load_vec<DT, true>(r, src, 0, v * kVec, cols);
            uint4* d = reinterpret_cast<uint4*>(srow + v * kVec * esz);
            d[0] = make_uint4(r.w[0], r.w[1], r.w[2], r.w[3]);
            if (DT == MOSAIC_F32) d[1] = make_uint4(r.w[4 % (Raw8<DT>::kBytes / 4)], r.w[5 % (Raw8<DT>::kBytes / 4)],
                                                    r.w[6 % (Raw8<DT>::kBytes / 4)], r.w[7 % (Raw8<DT>::kBytes / 4)]);
        }
        __syncthreads();
        const int n_out = (int)out_cols, ng = (int)col_group;
        if (ng == 1) {
            // Single columns: one 32-bit word of the output per lane, so that a warp reads 32
            // neighbouring entries of the keep list and writes 128 adjacent bytes per step.
            const int n_cu_m1 = (int)J.n_cu - 1;
            auto col = [&](int b) -> int { return min(max(__ldg(J.col_keep + b), 0), n_cu_m1); };
            if (DT == MOSAIC_F32) {
                const uint32_t* s32 = reinterpret_cast<const uint32_t*>(srow);
                uint32_t* d32 = reinterpret_cast<uint32_t*>(dst);
                for (int e = threadIdx.x; e < n_out; e += blockDim.x) __stcs(d32 + e, s32[col(e)]);
            } else {
                // the output matrix is dense: an odd row of odd width starts on the upper half of a word
                const uint16_t* s16 = reinterpret_cast<const uint16_t*>(srow);
                uint16_t* d16 = reinterpret_cast<uint16_t*>(dst);
                const int head = (int)(a & out_cols & 1);   // parity of a * out_cols
                const int pairs = (n_out - head) / 2;
                uint32_t* d32 = reinterpret_cast<uint32_t*>(d16 + head);
                for (int q = threadIdx.x; q < pairs; q += blockDim.x) {
                    const int j0 = col(head + 2 * q), j1 = col(head + 2 * q + 1);
                    __stcs(d32 + q, __byte_perm((uint32_t)s16[j0], (uint32_t)s16[j1], 0x5410));
                }
                if (threadIdx.x == 0 && head) d16[0] = s16[col(0)];
                if (threadIdx.x == 32 % blockDim.x && head + 2 * pairs < n_out) d16[n_out - 1] = s16[col(n_out - 1)];
            }
            continue;
        }
        // Units of several columns that are not whole vectors.  This row's elements
        // [head, head + 8*body) start on a 16-byte boundary whatever out_cols is and go out as whole
        // vectors; the up to 7 elements before and after them are stored one by one.
        const int head_full = (int)((kVec - (a * out_cols) % kVec) % kVec);
        const int head = head_full < n_out ? head_full : n_out;
        const int body = (n_out - head) / kVec;
        auto source_col = [&](int b) -> int {   // column of the staged row that output column b takes
            return (int)clamp_unit((int64_t)J.col_keep[b / ng], J.n_cu) * ng + b % ng;
        };
        for (int v = threadIdx.x; v < body; v += blockDim.x) {
            Raw8<DT> r;
            const int b0 = head + v * kVec;
#pragma unroll
            for (int e = 0; e < kVec; ++e) r.set_scalar(e, srow, source_col(b0 + e));
            r.store(dst + (size_t)b0 * esz);
        }
        const int tail0 = head + body * kVec;
        for (int t = threadIdx.x; t < head + (n_out - tail0); t += blockDim.x) {
            const int bb = t < head ? t : tail0 + (t - head);
            Raw8<DT> r;
            r.set_scalar(0, srow, source_col(bb));
            r.put_scalar(0, dst, bb);
        }
    }
}

// ---------------------------------------------------------------- host side: argument checks and launches
static int check_score_job(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype, const float* norms,
                           int64_t row_group, int64_t col_group) {
    const int rc = check_matrix(W, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (rows == 0 || row_group <= 0 || col_group <= 0 || rows % row_group || cols % col_group) return MOSAIC_ERR_INVALID_ARG;
    if (rows > 0x7FFFFFFF || cols > 0x7FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(norms) & 3u) return MOSAIC_ERR_MISALIGNED;
    return MOSAIC_OK;
}

template <int NJ>
static int launch_scores(const ScoreJobList<NJ>& list, int64_t tiles, int64_t units, int64_t lines, int dtype, cudaStream_t st) {
    if (dtype == MOSAIC_BF16) unit_partial_kernel<MOSAIC_BF16, NJ><<<(unsigned)tiles, kSThreads, 0, st>>>(list);
    else unit_partial_kernel<MOSAIC_F32, NJ><<<(unsigned)tiles, kSThreads, 0, st>>>(list);
    MOSAIC_LAUNCH_CHECK();
    line_sum_kernel<NJ><<<(unsigned)((lines + 127) / 128), 128, 0, st>>>(list, lines);
    MOSAIC_LAUNCH_CHECK();
    unit_score_kernel<NJ><<<(unsigned)((units + 127) / 128), 128, 0, st>>>(list, units);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

// True iff the kept columns come in whole 16-byte vectors (no staging of the source row needed).
static bool compact_by_vectors(int64_t cols, int64_t col_group, int64_t col_units_keep) {
    return (col_group % kVec) == 0 || (col_group == 1 && col_units_keep == cols);
}

static size_t staged_row_bytes(int64_t cols, int dtype) {
    return align_up((size_t)((cols + kVec - 1) / kVec * kVec) * elem_size(dtype), 16);
}

static int check_compact_job(const void* W_in, int64_t rows, int64_t cols, int64_t ldw, int dtype, const int32_t* row_keep,
                             int64_t row_units_keep, int64_t row_group, const int32_t* col_keep, int64_t col_units_keep,
                             int64_t col_group, const void* W_out) {
    const int rc = check_matrix(W_in, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (rows == 0 || row_group <= 0 || col_group <= 0 || rows % row_group || cols % col_group) return MOSAIC_ERR_INVALID_ARG;
    if (rows > 0x7FFFFFFF || cols > 0x7FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
    const int64_t n_ru = rows / row_group, n_cu = cols / col_group;
    if (row_units_keep < 1 || row_units_keep > n_ru || col_units_keep < 1 || col_units_keep > n_cu) return MOSAIC_ERR_INVALID_ARG;
    if (!row_keep || !col_keep || !W_out) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(row_keep) & 3u) || (reinterpret_cast<uintptr_t>(col_keep) & 3u) ||
        (reinterpret_cast<uintptr_t>(W_out) & 15u))
        return MOSAIC_ERR_MISALIGNED;
    const size_t in_span = ((size_t)(rows - 1) * (size_t)ldw + (size_t)cols) * elem_size(dtype);
    const size_t out_span = (size_t)(row_units_keep * row_group) * (size_t)(col_units_keep * col_group) * elem_size(dtype);
    const char *a = static_cast<const char*>(W_in), *b = static_cast<const char*>(W_out);
    if (a < b + out_span && b < a + in_span) return MOSAIC_ERR_ALIASING;
    // a source row that has to be staged must fit in shared memory (cols <= 51200 fp32)
    if (!compact_by_vectors(cols, col_group, col_units_keep) &&
        staged_row_bytes(cols, dtype) > 200 * 1024)
        return MOSAIC_ERR_INVALID_ARG;
    return MOSAIC_OK;
}

static CompactJob make_compact_job(const void* W_in, int64_t rows, int64_t cols, int64_t ldw, const int32_t* row_keep,
                                   int64_t row_units_keep, int64_t row_group, const int32_t* col_keep, int64_t col_units_keep,
                                   int64_t col_group, void* W_out, int64_t out_row0) {
    return CompactJob{W_in, W_out, row_keep, col_keep, cols, ldw, rows / row_group, row_group, cols / col_group, col_group,
                      row_units_keep * row_group, col_units_keep * col_group, out_row0};
}

template <int NJ>
static int launch_compact(const CompactJobList<NJ>& list, int64_t total_out_rows, int dtype, cudaStream_t st) {
    size_t smem = 0;
    for (int i = 0; i < list.n; ++i) {
        const CompactJob& J = list.job[i];
        if (!compact_by_vectors(J.cols, J.col_group, J.out_cols / J.col_group)) {
            const size_t need = staged_row_bytes(J.cols, dtype);
            if (need > smem) smem = need;
        }
    }
    static DeviceCache attr_set[2];   // the opt-in belongs to one device's copy of the kernel
    const int opted = attr_set[dtype == MOSAIC_BF16].get([&]() -> int {
        const cudaError_t e = (dtype == MOSAIC_BF16)
            ? cudaFuncSetAttribute(compact_kernel<MOSAIC_BF16, NJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
            : cudaFuncSetAttribute(compact_kernel<MOSAIC_F32, NJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) (void)cudaGetLastError();
        return e == cudaSuccess ? 1 : -1;
    });
    if (opted < 0) return MOSAIC_ERR_CUDA;
    // Resident CTAs: bounded by the staging buffer and by 2048 threads per SM.  What has to be in
    // flight to keep HBM busy is rows, not threads: short rows get CTAs of 128 threads, 16 per SM.
    const int by_smem = smem == 0 ? 16 : (int)((216 * 1024) / (smem + 1024));
    const int threads = by_smem >= 16 ? 128 : 256;
    int per_sm = by_smem < 1 ? 1 : (by_smem > 2048 / threads ? 2048 / threads : by_smem);
    int64_t grid = (int64_t)sm_count() * per_sm;
    if (grid > total_out_rows) grid = total_out_rows;
    if (dtype == MOSAIC_BF16) compact_kernel<MOSAIC_BF16, NJ><<<(unsigned)grid, threads, smem, st>>>(list, total_out_rows);
    else compact_kernel<MOSAIC_F32, NJ><<<(unsigned)grid, threads, smem, st>>>(list, total_out_rows);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

}  // namespace mosaic

using namespace mosaic;

// ---------------------------------------------------------------- batched calls
extern "C" size_t mosaic_unit_scores_batch_workspace_bytes(const mosaic_unit_score_job* jobs, int64_t n_jobs) {
    size_t total = 256;
    if (jobs == nullptr) return total;
    for (int64_t i = 0; i < n_jobs; ++i)
        if (jobs[i].rows > 0 && jobs[i].cols > 0) total += score_ws_bytes(jobs[i].rows, jobs[i].cols);
    return total;
}

extern "C" int mosaic_unit_scores_batch(const mosaic_unit_score_job* jobs, int64_t n_jobs, int dtype, void* ws, size_t ws_bytes,
                                        void* stream) {
    if (n_jobs < 0) return MOSAIC_ERR_INVALID_ARG;
    if (n_jobs == 0) return MOSAIC_OK;
    if (jobs == nullptr || ws == nullptr) return MOSAIC_ERR_NULL_PTR;
    for (int64_t i = 0; i < n_jobs; ++i) {
        const mosaic_unit_score_job& j = jobs[i];
        const int rc = check_score_job(j.W, j.rows, j.cols, j.ldw, dtype, j.norms, j.row_group, j.col_group);
        if (rc != MOSAIC_OK) return rc;
        if ((reinterpret_cast<uintptr_t>(j.row_scores_out) & 3u) || (reinterpret_cast<uintptr_t>(j.col_scores_out) & 3u))
            return MOSAIC_ERR_MISALIGNED;
    }
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
    if (ws_bytes < mosaic_unit_scores_batch_workspace_bytes(jobs, n_jobs)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::unique_ptr<ScoreJobList<kStructBatch>> mem(new (std::nothrow) ScoreJobList<kStructBatch>);
    if (!mem) return MOSAIC_ERR_INVALID_ARG;
    ScoreJobList<kStructBatch>& list = *mem;
    char* wsp = static_cast<char*>(ws);
    int64_t i = 0;
    while (i < n_jobs) {
        list.n = 0;
        int64_t tiles = 0, units = 0, lines = 0;
        while (i < n_jobs && list.n < kStructBatch) {
            const mosaic_unit_score_job& j = jobs[i];
            int chunks, bands;
            score_shape(j.rows, j.cols, &chunks, &bands);
            if (tiles + (int64_t)chunks * bands > 0x3FFFFFFF) break;
            double* rp = reinterpret_cast<double*>(wsp);
            double* cpart = reinterpret_cast<double*>(wsp + align_up(sizeof(double) * (size_t)chunks * (size_t)j.rows, 256));
            list.job[list.n++] = ScoreJob{j.W, j.norms, rp, cpart, j.row_scores_out, j.col_scores_out, j.rows, j.cols, j.ldw,
                                          j.row_group, j.col_group, units, lines, (int)tiles, chunks, bands, 0};
            wsp += score_ws_bytes(j.rows, j.cols);
            tiles += (int64_t)chunks * bands;
            units += j.rows / j.row_group + j.cols / j.col_group;
            lines += j.rows + j.cols;
            ++i;
        }
        if (list.n == 0) return MOSAIC_ERR_INVALID_ARG;
        const int rc = launch_scores<kStructBatch>(list, tiles, units, lines, dtype, st);
        if (rc != MOSAIC_OK) return rc;
    }
    return MOSAIC_OK;
}

extern "C" int mosaic_rank_units_batch(const mosaic_rank_job* jobs, int64_t n_jobs, void* stream) {
    if (n_jobs < 0) return MOSAIC_ERR_INVALID_ARG;
    if (n_jobs == 0) return MOSAIC_OK;
    if (jobs == nullptr) return MOSAIC_ERR_NULL_PTR;
    for (int64_t i = 0; i < n_jobs; ++i) {
        const mosaic_rank_job& j = jobs[i];
        if (!j.scores || (!j.keep_out && j.keep > 0)) return MOSAIC_ERR_NULL_PTR;
        if (j.n_units <= 0 || j.keep < 0 || j.keep > j.n_units || j.n_units > 0x7FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(j.scores) & 3u) || (reinterpret_cast<uintptr_t>(j.keep_out) & 3u)) return MOSAIC_ERR_MISALIGNED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    constexpr int NJ = 4 * kStructBatch;
    std::unique_ptr<RankJobList<NJ>> mem(new (std::nothrow) RankJobList<NJ>);
    if (!mem) return MOSAIC_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n_jobs; i += NJ) {
        mem->n = (int)(n_jobs - i < NJ ? n_jobs - i : NJ);
        for (int m = 0; m < mem->n; ++m) mem->job[m] = RankJob{jobs[i + m].scores, jobs[i + m].keep_out, jobs[i + m].n_units, jobs[i + m].keep};
        rank_kernel<NJ><<<(unsigned)mem->n, kRankThreads, 0, st>>>(*mem);
        MOSAIC_LAUNCH_CHECK();
    }
    return MOSAIC_OK;
}

extern "C" int mosaic_add_unit_scores_batch(const mosaic_add_job* jobs, int64_t n_jobs, void* stream) {
    if (n_jobs < 0) return MOSAIC_ERR_INVALID_ARG;
    if (n_jobs == 0) return MOSAIC_OK;
    if (jobs == nullptr) return MOSAIC_ERR_NULL_PTR;
    for (int64_t i = 0; i < n_jobs; ++i) {
        const mosaic_add_job& j = jobs[i];
        if (j.n < 0) return MOSAIC_ERR_INVALID_ARG;
        if (j.n > 0 && (!j.dst || !j.a || !j.b)) return MOSAIC_ERR_NULL_PTR;
        if ((reinterpret_cast<uintptr_t>(j.dst) & 3u) || (reinterpret_cast<uintptr_t>(j.a) & 3u) || (reinterpret_cast<uintptr_t>(j.b) & 3u))
            return MOSAIC_ERR_MISALIGNED;
        // dst may be a or b exactly; any partial overlap is refused
        for (const float* s : {j.a, j.b})
            if (j.n > 0 && j.dst != s && j.dst < s + j.n && s < j.dst + j.n) return MOSAIC_ERR_ALIASING;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    constexpr int NJ = 4 * kStructBatch;
    std::unique_ptr<AddJobList<NJ>> mem(new (std::nothrow) AddJobList<NJ>);
    if (!mem) return MOSAIC_ERR_INVALID_ARG;
    int64_t i = 0;
    while (i < n_jobs) {
        mem->n = 0;
        int64_t total = 0;
        for (; i < n_jobs && mem->n < NJ; ++i) {
            if (jobs[i].n == 0) continue;
            mem->job[mem->n++] = AddJob{jobs[i].dst, jobs[i].a, jobs[i].b, jobs[i].n, total};
            total += jobs[i].n;
        }
        if (mem->n == 0) break;
        add_scores_kernel<NJ><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(*mem, total);
        MOSAIC_LAUNCH_CHECK();
    }
    return MOSAIC_OK;
}

extern "C" int mosaic_compact_batch(const mosaic_compact_job* jobs, int64_t n_jobs, int dtype, void* stream) {
    if (n_jobs < 0) return MOSAIC_ERR_INVALID_ARG;
    if (n_jobs == 0) return MOSAIC_OK;
    if (jobs == nullptr) return MOSAIC_ERR_NULL_PTR;
    for (int64_t i = 0; i < n_jobs; ++i) {
        const mosaic_compact_job& j = jobs[i];
        const int rc = check_compact_job(j.W_in, j.rows, j.cols, j.ldw, dtype, j.row_keep_units, j.row_units_keep, j.row_group,
                                         j.col_keep_units, j.col_units_keep, j.col_group, j.W_out);
        if (rc != MOSAIC_OK) return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::unique_ptr<CompactJobList<kStructBatch>> mem(new (std::nothrow) CompactJobList<kStructBatch>);
    if (!mem) return MOSAIC_ERR_INVALID_ARG;
    // One launch per class of staged row length (steps of 8 KB; class 0 = no staging), so that the
    // shared memory of a CTA, and with it the number of rows in flight per SM, fits the rows it serves.
    auto row_class = [&](const mosaic_compact_job& j) -> int {
        if (compact_by_vectors(j.cols, j.col_group, j.col_units_keep)) return 0;
        return (int)((staged_row_bytes(j.cols, dtype) + 8191) / 8192);
    };
    constexpr int kClasses = 200 * 1024 / 8192 + 1;
    bool present[kClasses] = {};
    for (int64_t i = 0; i < n_jobs; ++i) present[row_class(jobs[i])] = true;
    for (int c = 0; c < kClasses; ++c) {
        if (!present[c]) continue;
        int64_t i = 0;
        while (i < n_jobs) {
            mem->n = 0;
            int64_t total = 0;
            for (; i < n_jobs && mem->n < kStructBatch; ++i) {
                const mosaic_compact_job& j = jobs[i];
                if (row_class(j) != c) continue;
                mem->job[mem->n++] = make_compact_job(j.W_in, j.rows, j.cols, j.ldw, j.row_keep_units, j.row_units_keep, j.row_group,
                                                      j.col_keep_units, j.col_units_keep, j.col_group, j.W_out, total);
                total += j.row_units_keep * j.row_group;
            }
            if (mem->n == 0) break;
            const int rc = launch_compact<kStructBatch>(*mem, total, dtype, st);
            if (rc != MOSAIC_OK) return rc;
        }
    }
    return MOSAIC_OK;
}

// ---------------------------------------------------------------- single calls
extern "C" size_t mosaic_prune_structured_compact_workspace_bytes(int64_t rows, int64_t cols) {
    if (rows <= 0 || cols <= 0) return 256;
    return score_ws_bytes(rows, cols) + align_up(sizeof(float) * (size_t)(rows + cols), 256);
}

extern "C" int mosaic_rank_units(const float* scores, int64_t n_units, int64_t keep, int32_t* keep_out, void* stream) {
    const mosaic_rank_job one{scores, n_units, keep, keep_out};
    return mosaic_rank_units_batch(&one, 1, stream);
}

extern "C" int mosaic_sum_unit_scores(float* dst, const float* src, int64_t n_units, void* stream) {
    if (!dst || !src) return MOSAIC_ERR_NULL_PTR;
    const mosaic_add_job one{dst, dst, src, n_units};
    return mosaic_add_unit_scores_batch(&one, 1, stream);
}

extern "C" int mosaic_prune_structured_compact(const void* W_in, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                               const float* norms, int64_t row_group, int64_t col_group,
                                               int64_t row_units_keep, int64_t col_units_keep, int32_t* row_keep_units,
                                               int32_t* col_keep_units, int flags, void* W_out, float* unit_scores_out,
                                               void* ws, size_t ws_bytes, void* stream) {
    int rc = check_score_job(W_in, rows, cols, ldw, dtype, norms, row_group, col_group);
    if (rc != MOSAIC_OK) return rc;
    const int known = MOSAIC_ROWS_GIVEN | MOSAIC_COLS_GIVEN | MOSAIC_RANK_ONLY | MOSAIC_SCORES_ONLY | MOSAIC_SCORES_ACCUM;
    if (flags & ~known) return MOSAIC_ERR_INVALID_ARG;
    const int64_t n_ru = rows / row_group, n_cu = cols / col_group;
    const bool scores_only = flags & MOSAIC_SCORES_ONLY;
    const bool rank_only = flags & MOSAIC_RANK_ONLY;
    const bool rows_given = flags & MOSAIC_ROWS_GIVEN, cols_given = flags & MOSAIC_COLS_GIVEN;
    if ((flags & MOSAIC_SCORES_ACCUM) && !unit_scores_out) return MOSAIC_ERR_NULL_PTR;
    if (scores_only && !unit_scores_out) return MOSAIC_ERR_NULL_PTR;
    if (reinterpret_cast<uintptr_t>(unit_scores_out) & 3u) return MOSAIC_ERR_MISALIGNED;
    if (!scores_only) {
        if (row_units_keep < 1 || row_units_keep > n_ru || col_units_keep < 1 || col_units_keep > n_cu)
            return MOSAIC_ERR_INVALID_ARG;
        if (!row_keep_units || !col_keep_units) return MOSAIC_ERR_NULL_PTR;
        if ((reinterpret_cast<uintptr_t>(row_keep_units) & 3u) || (reinterpret_cast<uintptr_t>(col_keep_units) & 3u))
            return MOSAIC_ERR_MISALIGNED;
        if (!rank_only) {
            rc = check_compact_job(W_in, rows, cols, ldw, dtype, row_keep_units, row_units_keep, row_group, col_keep_units,
                                   col_units_keep, col_group, W_out);
            if (rc != MOSAIC_OK) return rc;
        }
    }
    const bool need_scores = scores_only || unit_scores_out || !(rows_given && cols_given);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    float* scores = nullptr;   // [row units, column units]
    if (need_scores) {
        if (!ws) return MOSAIC_ERR_NULL_PTR;
        if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
        if (ws_bytes < mosaic_prune_structured_compact_workspace_bytes(rows, cols)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
        int chunks, bands;
        score_shape(rows, cols, &chunks, &bands);
        char* wsp = static_cast<char*>(ws);
        double* rp = reinterpret_cast<double*>(wsp);
        double* cpart = reinterpret_cast<double*>(wsp + align_up(sizeof(double) * (size_t)chunks * (size_t)rows, 256));
        float* ws_scores = reinterpret_cast<float*>(wsp + score_ws_bytes(rows, cols));
        // with SCORES_ACCUM the running totals live in the caller's array; ranking then uses those
        scores = (flags & MOSAIC_SCORES_ACCUM) ? unit_scores_out : ws_scores;
        ScoreJobList<1> one;
        one.n = 1;
        one.job[0] = ScoreJob{W_in, norms, rp, cpart, scores, scores + n_ru, rows, cols, ldw, row_group, col_group, 0, 0, 0,
                              chunks, bands, (flags & MOSAIC_SCORES_ACCUM) ? 1 : 0};
        rc = launch_scores<1>(one, (int64_t)chunks * bands, n_ru + n_cu, rows + cols, dtype, st);
        if (rc != MOSAIC_OK) return rc;
        if (unit_scores_out && scores != unit_scores_out)
            MOSAIC_CUDA_TRY(cudaMemcpyAsync(unit_scores_out, scores, sizeof(float) * (size_t)(n_ru + n_cu), cudaMemcpyDeviceToDevice, st));
    }
    if (scores_only) return MOSAIC_OK;

    if (!(rows_given && cols_given)) {
        RankJobList<2> two;
        two.n = 2;
        two.job[0] = RankJob{scores, rows_given ? nullptr : row_keep_units, n_ru, rows_given ? 0 : row_units_keep};
        two.job[1] = RankJob{scores + n_ru, cols_given ? nullptr : col_keep_units, n_cu, cols_given ? 0 : col_units_keep};
        rank_kernel<2><<<2, kRankThreads, 0, st>>>(two);
        MOSAIC_LAUNCH_CHECK();
    }
    if (rank_only) return MOSAIC_OK;

    CompactJobList<1> one;
    one.n = 1;
    one.job[0] = make_compact_job(W_in, rows, cols, ldw, row_keep_units, row_units_keep, row_group, col_keep_units,
                                  col_units_keep, col_group, W_out, 0);
    return launch_compact<1>(one, row_units_keep * row_group, dtype, st);
}
