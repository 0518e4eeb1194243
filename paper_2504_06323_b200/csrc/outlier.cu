// mosaic_score (Eq. 5 materialised) and mosaic_outlier_ratio (Eq. 6 /
// the outlier-count step of Algorithm 1): fp64 sum of the weight metric over a projection,
// threshold tau = alpha * mean, strict outlier count.
//
// Every matrix is cut into tiles of 1024 columns (a thread owns 8 adjacent
// columns, whose norms stay in registers) by 64 rows; 8 row loads are in flight
// per thread.  A launch works through the tiles of a whole list of matrices
// with resident CTAs, each taking a contiguous range of tiles, so a model's
// worth of projections costs two launches, not two per projection.
//   sweep 1  writes one fp64 partial per tile.
//   sweep 2  on entering a matrix adds that matrix's partials in tile order (so
//            the sum depends neither on scheduling nor on the grid), forms tau,
//            and counts in fp32 against tau rounded toward -inf: for an fp32
//            score s, (double)s > tau  <=>  s > fl32_down(tau).  It walks the
//            tiles in reverse, starting on what sweep 1 touched last.
//
// bf16 matrices whose rows are whole 16-byte vectors (cols % 8 == 0: every projection of a
// model) take two leaner kernels with the same partial sums and the same results:
//   score_sum_bf16_kernel     the sweep above without the ragged-edge handling, 4 loads in flight
//                             and few enough registers for 32+ resident warps per SM;
//   outlier_count_bf16_kernel counts without forming a score: for a fixed column the predicate
//                             fl32(norm_j * |w|) > tau is monotone in the 15 magnitude bits of
//                             w, so per column there is one bf16 pattern A_j - found exactly, by
//                             bisection on that very predicate - with  score > tau  <=>  |w| >= A_j,
//                             and a row is counted two weights per integer subtract:
//                             (w | 0x8000) - A_j has bit 15 set iff the magnitude is >= A_j.
// The batched call reads such matrices only once: score_sum_ladder_kernel is the first sweep with a
// ladder of bf16 patterns per column around an estimated threshold, from which the exact count
// follows when the sum is known (see "Single sweep" below); the second sweep remains as the
// fallback for matrices whose threshold falls off a ladder.
#include <atomic>
#include <memory>
#include <new>

#include "common.cuh"

namespace mosaic {

constexpr int kOutThreads = 128;
constexpr int kOutChunk = kOutThreads * kVec;  // 1024 columns
constexpr int kOutUnroll = 8;
constexpr int kOutTileRows = 64;
constexpr int kOutBatch = 256;                 // matrices per launch (the list travels as a kernel parameter)

// Single-sweep bookkeeping of one matrix (batched bf16 path): the estimate of its score sum from a
// sample of rows, the count of its sure outliers, and whether the ladder settled its count.
struct OutlierCtrl {
    double est_sum;
    unsigned long long sure;        // weights above their column's ladder
    unsigned long long lad_count;   // ladder entries at or above the threshold, summed by the finishing CTAs
    int valid;                      // 1: count_out holds the count
    int invalid;                    // some column's threshold fell off its ladder
    int done;                       // finishing CTAs that have reported
};
constexpr int kLadder = 32;   // bf16 magnitude patterns per column that the single sweep keeps apart

struct OutlierJob {
    const void* W;
    const float* norms;
    unsigned long long* count_out;
    double* sum_out;       // or nullptr
    double* partial;       // [tiles of this matrix], in the workspace
    int64_t rows, cols, ldw;
    int tile0;             // first global tile
    int chunks;            // tiles per row band
    int ctile0;            // first global tile of the bf16 count sweep (taller tiles)
    int g_first, g_last;   // jobs of the launch that share this job's threshold (itself alone: Eq. 6; a layer: Eq. 3-4)
    OutlierCtrl* ctrl;     // single-sweep mode: bookkeeping and [cols][kLadder] counters in the workspace; else nullptr
    uint32_t* ladder;
};
template <int NJ>
struct OutlierJobList {
    int n;
    float alpha;
    OutlierJob job[NJ];
};

__host__ __device__ inline int64_t outlier_tiles(int64_t rows, int64_t cols) {
    return ((cols + kOutChunk - 1) / kOutChunk) * ((rows + kOutTileRows - 1) / kOutTileRows);
}

constexpr int kCntTileRows = 256;   // rows per tile of the bf16 count sweep: the per-column thresholds are found once per tile
__host__ __device__ inline int64_t outlier_count_tiles(int64_t rows, int64_t cols) {
    return ((cols + kOutChunk - 1) / kOutChunk) * ((rows + kCntTileRows - 1) / kCntTileRows);
}

// Tiles [t_begin, t_end) of this CTA: an equal share of the n_tiles, contiguous.
__device__ __forceinline__ void tile_share(int n_tiles, int* t_begin, int* t_end) {
    const int64_t g = gridDim.x, b = blockIdx.x;
    *t_begin = (int)((int64_t)n_tiles * b / g);
    *t_end = (int)((int64_t)n_tiles * (b + 1) / g);
}

template <int DT, int NJ>
__global__ void __launch_bounds__(kOutThreads) score_sum_kernel(const __grid_constant__ OutlierJobList<NJ> jobs, int n_tiles) {
    __shared__ double red[32];
    int t_begin, t_end;
    tile_share(n_tiles, &t_begin, &t_end);
    int j = 0;
    for (int tile = t_begin; tile < t_end; ++tile) {
        while (j + 1 < jobs.n && tile >= jobs.job[j + 1].tile0) ++j;
        const OutlierJob& J = jobs.job[j];
        const int local = tile - J.tile0;
        if (local == 0 && threadIdx.x == 0) *J.count_out = 0ull;   // sweep 2 is a later launch
        const int chunk = local % J.chunks, band = local / J.chunks;
        const int64_t rows = J.rows, cols = J.cols, ldw = J.ldw;
        const int64_t c0 = (int64_t)chunk * kOutChunk + threadIdx.x * kVec;
        const int64_t r0 = (int64_t)band * kOutTileRows;
        const int64_t r1 = (r0 + kOutTileRows < rows) ? r0 + kOutTileRows : rows;
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        if (c0 < cols) {
            float nrm[kVec];
#pragma unroll
            for (int e = 0; e < kVec; ++e) nrm[e] = (c0 + e < cols) ? J.norms[c0 + e] : 0.0f;
            int64_t r = r0;
            for (; r + kOutUnroll <= r1; r += kOutUnroll) {
                Raw8<DT> v[kOutUnroll];
#pragma unroll
                for (int u = 0; u < kOutUnroll; ++u) load_vec<DT, true>(v[u], J.W, (r + u) * ldw, c0, cols);
#pragma unroll
                for (int u = 0; u < kOutUnroll; ++u)
#pragma unroll
                    for (int e = 0; e < kVec; ++e) acc[u & 3] += (double)__fmul_rn(nrm[e], v[u].abs_f32(e));
            }
            for (; r < r1; ++r) {
                Raw8<DT> v;
                load_vec<DT, true>(v, J.W, r * ldw, c0, cols);
#pragma unroll
                for (int e = 0; e < kVec; ++e) acc[0] += (double)__fmul_rn(nrm[e], v.abs_f32(e));
            }
        }
        const double mine = (acc[0] + acc[1]) + (acc[2] + acc[3]);
        const double blk = block_sum(mine, red);
        if (threadIdx.x == 0) J.partial[local] = blk;
    }
}


// tau of job j, rounded toward -inf for the fp32 comparison: alpha * (S / C) over the jobs g_first..g_last
// that share it - each job's partial sums in tile order (thread-strided, then a fixed tree), the jobs in
// list order.  Block-wide; also writes the job's own sum if asked to.
template <int NJ>
__device__ float group_threshold(const OutlierJobList<NJ>& jobs, int j, bool write_sum, double* red, float* tau_sh) {
    const OutlierJob& J = jobs.job[j];
    double total = 0.0, numel = 0.0;
    for (int g = J.g_first; g <= J.g_last; ++g) {
        const OutlierJob& G = jobs.job[g];
        const int nt_g = (int)outlier_tiles(G.rows, G.cols);
        double s = 0.0;
        for (int i = threadIdx.x; i < nt_g; i += kOutThreads) s += __ldcg(&G.partial[i]);
        const double sg = block_sum(s, red);   // valid in thread 0
        total = total + sg;
        numel = numel + (double)(G.rows * G.cols);
        if (g == j && write_sum && threadIdx.x == 0 && J.sum_out) *J.sum_out = sg;
    }
    if (threadIdx.x == 0) {
        const double mean = total / numel;
        *tau_sh = __double2float_rd((double)jobs.alpha * mean);
    }
    __syncthreads();
    return *tau_sh;
}

template <int DT, int NJ>
__global__ void __launch_bounds__(kOutThreads) outlier_count_kernel(const __grid_constant__ OutlierJobList<NJ> jobs, int n_tiles) {
    __shared__ double red[32];
    __shared__ unsigned int cred[32];
    __shared__ float tau_sh;
    int t_begin, t_end;
    tile_share(n_tiles, &t_begin, &t_end);
    int j = jobs.n - 1, j_tau = -1;
    float tau = 0.0f;
    unsigned int cnt = 0;
    auto flush = [&](int job) {   // add this CTA's count for `job` (block-uniform call)
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
        const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
        __syncthreads();
        if (lane == 0) cred[wid] = cnt;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long tot = 0;
            for (int i = 0; i < kOutThreads / 32; ++i) tot += cred[i];
            if (tot) atomicAdd(jobs.job[job].count_out, tot);   // integer: exact in any order
        }
        cnt = 0;
    };
    for (int t2 = t_begin; t2 < t_end; ++t2) {
        const int tile = n_tiles - 1 - t2;   // reverse order of sweep 1
        while (tile < jobs.job[j].tile0) --j;
        const OutlierJob& J = jobs.job[j];
        const int64_t rows = J.rows, cols = J.cols, ldw = J.ldw;
        if (j != j_tau) {
            if (j_tau >= 0) flush(j_tau);
            const int nt_j = (int)outlier_tiles(rows, cols);
            tau = group_threshold<NJ>(jobs, j, tile == J.tile0 + nt_j - 1, red, &tau_sh);   // the sum: once, by the CTA that owns the last tile
            j_tau = j;
        }
        const int local = tile - J.tile0;
        const int chunk = local % J.chunks, band = local / J.chunks;
        const int64_t c0 = (int64_t)chunk * kOutChunk + threadIdx.x * kVec;
        const int64_t r0 = (int64_t)band * kOutTileRows;
        const int64_t r1 = (r0 + kOutTileRows < rows) ? r0 + kOutTileRows : rows;
        if (c0 < cols) {
            float nrm[kVec];
            bool valid[kVec];
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                valid[e] = (c0 + e < cols);
                nrm[e] = valid[e] ? J.norms[c0 + e] : 0.0f;
            }
            int64_t r = r1;
            for (; r - kOutUnroll >= r0; r -= kOutUnroll) {
                Raw8<DT> v[kOutUnroll];
#pragma unroll
                for (int u = 0; u < kOutUnroll; ++u) load_vec<DT, true>(v[u], J.W, (r - 1 - u) * ldw, c0, cols);
#pragma unroll
                for (int u = 0; u < kOutUnroll; ++u)
#pragma unroll
                    for (int e = 0; e < kVec; ++e)
                        cnt += (valid[e] && __fmul_rn(nrm[e], v[u].abs_f32(e)) > tau) ? 1u : 0u;
            }
            for (; r > r0; --r) {
                Raw8<DT> v;
                load_vec<DT, true>(v, J.W, (r - 1) * ldw, c0, cols);
#pragma unroll
                for (int e = 0; e < kVec; ++e) cnt += (valid[e] && __fmul_rn(nrm[e], v.abs_f32(e)) > tau) ? 1u : 0u;
            }
        }
    }
    if (j_tau >= 0) flush(j_tau);
}

// ------------------------------------------------------------------------------------------
// bf16, cols % 8 == 0
// ------------------------------------------------------------------------------------------
// The eight scores of one 16-byte vector added to four fp64 accumulators (element e to acc[e & 3]).
__device__ __forceinline__ void add_scores(const uint4& v, const float (&nrm)[kVec], double (&acc)[4]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
        acc[(2 * i) & 3] += (double)__fmul_rn(nrm[2 * i], fabsf(lo));
        acc[(2 * i + 1) & 3] += (double)__fmul_rn(nrm[2 * i + 1], fabsf(hi));
    }
}

template <int NJ>
__global__ void __launch_bounds__(kOutThreads, 8) score_sum_bf16_kernel(const __grid_constant__ OutlierJobList<NJ> jobs,
                                                                        int n_tiles) {
    __shared__ double red[32];
    int t_begin, t_end;
    tile_share(n_tiles, &t_begin, &t_end);
    int j = 0;
    for (int tile = t_begin; tile < t_end; ++tile) {
        while (j + 1 < jobs.n && tile >= jobs.job[j + 1].tile0) ++j;
        const OutlierJob& J = jobs.job[j];
        const int local = tile - J.tile0;
        if (local == 0 && threadIdx.x == 0) *J.count_out = 0ull;   // the count sweep is a later launch
        const int chunk = local % J.chunks, band = local / J.chunks;
        const int c0 = chunk * kOutChunk + (int)threadIdx.x * kVec;
        const int64_t r0 = (int64_t)band * kOutTileRows;
        const int n_rows = (int)((r0 + kOutTileRows < J.rows ? r0 + kOutTileRows : J.rows) - r0);
        double acc[4] = {0.0, 0.0, 0.0, 0.0};
        if (c0 < (int)J.cols) {
            float nrm[kVec];
#pragma unroll
            for (int e = 0; e < kVec; ++e) nrm[e] = __ldg(J.norms + c0 + e);
            const size_t stride = (size_t)J.ldw * 2u;
            const char* p = static_cast<const char*>(J.W) + ((size_t)r0 * (size_t)J.ldw + (size_t)c0) * 2u;
            int r = 0;
            for (; r + 4 <= n_rows; r += 4, p += 4 * stride) {
                const uint4 v0 = ld_stream16_ro(p), v1 = ld_stream16_ro(p + stride), v2 = ld_stream16_ro(p + 2 * stride),
                            v3 = ld_stream16_ro(p + 3 * stride);
                add_scores(v0, nrm, acc);
                add_scores(v1, nrm, acc);
                add_scores(v2, nrm, acc);
                add_scores(v3, nrm, acc);
            }
            for (; r < n_rows; ++r, p += stride) add_scores(ld_stream16_ro(p), nrm, acc);
        }
        const double blk = block_sum((acc[0] + acc[1]) + (acc[2] + acc[3]), red);
        if (threadIdx.x == 0) J.partial[local] = blk;
    }
}

// Smallest bf16 magnitude pattern a in [0, 0x7F80] with  fl32(n * value(a)) > tau  (0x8000 if there
// is none: n = 0, n or tau not a number, tau = +inf).  The predicate is evaluated exactly as the
// score is defined (one fp32 multiply, compared with tau already rounded toward -inf) and is
// monotone in a for n >= 0, so bisection finds the exact boundary; it starts from the bracket
// [g-2, g+2] around the pattern of tau / n, which holds it except in odd corners (subnormals,
// overflow), where the whole range is searched.
__device__ __forceinline__ uint32_t outlier_pattern(float n, float tau) {
    auto above = [&](uint32_t a) -> bool { return __fmul_rn(n, __uint_as_float(a << 16)) > tau; };
    if (!above(0x7F80u)) return 0x8000u;
    if (above(0u)) return 0u;
    uint32_t lo = 0u, hi = 0x7F80u;   // above(lo) false, above(hi) true
    const uint32_t g = __float_as_uint(__fdiv_rn(tau, n)) >> 16;   // tau >= 0 and n > 0 here
    if (g >= 2u && g + 2u <= 0x7F80u && !above(g - 2u) && above(g + 2u)) {
        lo = g - 2u;
        hi = g + 2u;
    }
    while (hi - lo > 1u) {
        const uint32_t mid = (lo + hi) >> 1;
        if (above(mid)) hi = mid;
        else lo = mid;
    }
    return hi;
}

// Flags of (magnitude >= threshold) of a vector's eight elements, counted.  See prune_warp.cu for
// the borrow-free subtraction: t = (w | 0x80008000) - A, thresholds A <= 0x8000 per 16-bit lane.
__device__ __forceinline__ uint32_t count_at_or_above(const uint4& v, const uint4& A) {
    const uint32_t t0 = (v.x | 0x80008000u) - A.x, t1 = (v.y | 0x80008000u) - A.y, t2 = (v.z | 0x80008000u) - A.z,
                   t3 = (v.w | 0x80008000u) - A.w;
    const uint32_t a = __byte_perm(t0, t1, 0x7531), b = __byte_perm(t2, t3, 0x7531);   // flag = top bit of every byte
    return (uint32_t)__popc(a & 0x80808080u) + (uint32_t)__popc(b & 0x80808080u);
}

template <int NJ>
__global__ void __launch_bounds__(kOutThreads, 8) outlier_count_bf16_kernel(const __grid_constant__ OutlierJobList<NJ> jobs,
                                                                            int n_tiles) {
    __shared__ double red[32];
    __shared__ unsigned int cred[32];
    __shared__ float tau_sh;
    int t_begin, t_end;
    tile_share(n_tiles, &t_begin, &t_end);
    int j = jobs.n - 1, j_tau = -1;
    float tau = 0.0f;
    unsigned int cnt = 0;
    bool settled = false;
    auto flush = [&](int job) {   // add this CTA's count for `job` (block-uniform call)
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
        const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
        __syncthreads();
        if (lane == 0) cred[wid] = cnt;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long tot = 0;
            for (int i = 0; i < kOutThreads / 32; ++i) tot += cred[i];
            if (tot) atomicAdd(jobs.job[job].count_out, tot);   // integer: exact in any order
        }
        cnt = 0;
    };
    for (int t2 = t_begin; t2 < t_end; ++t2) {
        const int tile = n_tiles - 1 - t2;   // reverse order of the sum sweep
        while (tile < jobs.job[j].ctile0) --j;
        const OutlierJob& J = jobs.job[j];
        if (j != j_tau) {
            if (j_tau >= 0 && !settled) flush(j_tau);
            settled = J.ctrl != nullptr && __ldcg(&J.ctrl->valid) != 0;   // the single sweep has this matrix's count already
            if (!settled) {
                const int last = J.ctile0 + (int)outlier_count_tiles(J.rows, J.cols) - 1;
                tau = group_threshold<NJ>(jobs, j, tile == last, red, &tau_sh);   // the sum: once, by the CTA that owns the matrix's last tile
            }
            j_tau = j;
        }
        if (settled) continue;
        const int local = tile - J.ctile0;
        const int chunk = local % J.chunks, band = local / J.chunks;
        const int c0 = chunk * kOutChunk + (int)threadIdx.x * kVec;
        const int64_t r0 = (int64_t)band * kCntTileRows;
        const int n_rows = (int)((r0 + kCntTileRows < J.rows ? r0 + kCntTileRows : J.rows) - r0);
        if (c0 < (int)J.cols) {
            uint32_t A[kVec];
#pragma unroll
            for (int e = 0; e < kVec; ++e) A[e] = outlier_pattern(__ldg(J.norms + c0 + e), tau);
            const uint4 A4 = make_uint4(A[0] | (A[1] << 16), A[2] | (A[3] << 16), A[4] | (A[5] << 16), A[6] | (A[7] << 16));
            const size_t stride = (size_t)J.ldw * 2u;
            const char* p = static_cast<const char*>(J.W) + ((size_t)r0 * (size_t)J.ldw + (size_t)c0) * 2u;
            int r = 0;
            for (; r + 8 <= n_rows; r += 8, p += 8 * stride) {
                uint4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = ld_stream16_ro(p + u * stride);
#pragma unroll
                for (int u = 0; u < 8; ++u) cnt += count_at_or_above(v[u], A4);
            }
            for (; r < n_rows; ++r, p += stride) cnt += count_at_or_above(ld_stream16_ro(p), A4);
        }
    }
    if (j_tau >= 0 && !settled) flush(j_tau);
}

// ------------------------------------------------------------------------------------------
// Single sweep (batched bf16 path).  The count needs the threshold tau = alpha * mean, and the mean
// needs the whole matrix - but for a fixed column the predicate score > tau is "magnitude pattern
// >= A_j(tau)", and bf16 has few patterns: an estimate tau^ of the threshold (from a sample of
// rows) is enough to know that A_j(tau) lies within kLadder patterns above A_j(0.97 tau^).  The
// sweep that sums the scores therefore also counts, per column, the weights on each of those
// kLadder patterns (a few per mille of all weights: one atomic each) and, in registers, the
// weights above them.  Once the sum is known the exact count is the sure ones plus the ladder
// entries from A_j(tau) up - the same number the count sweep would find, without a second read
// of the matrix.  A matrix whose tau falls outside some column's ladder (a poor estimate) keeps
// valid = 0 and is counted by the count sweep after all.
// ------------------------------------------------------------------------------------------

// est_sum of every matrix: the fp64 sum of the scores of about 256 evenly spaced rows, scaled to all
// rows.  kEstParts CTAs per matrix (128 column lanes of 8 columns x kEstRowLanes row lanes each) add
// their shares atomically: the estimate may differ in its last bits from run to run, which moves a
// ladder by a pattern at most and never the count.  The bookkeeping block was zeroed with the ladders.
constexpr int kEstRowLanes = 4, kEstParts = 8;
template <int NJ>
__global__ void __launch_bounds__(kOutThreads * kEstRowLanes) outlier_estimate_kernel(const __grid_constant__ OutlierJobList<NJ> jobs) {
    __shared__ double red[32];
    const OutlierJob& J = jobs.job[blockIdx.x];
    const int64_t step = J.rows / 256 > 0 ? J.rows / 256 : 1;
    const int64_t n_sampled = (J.rows - step / 2 + step - 1) / step;   // rows step/2, step/2 + step, ...
    const int cl = threadIdx.x % kOutThreads, rl = threadIdx.x / kOutThreads;
    const int lanes = kEstRowLanes * kEstParts, my = (int)blockIdx.y * kEstRowLanes + rl;
    const size_t stride = (size_t)J.ldw * 2u;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int c0 = cl * kVec; c0 < (int)J.cols; c0 += kOutChunk) {
        float nrm[kVec];
#pragma unroll
        for (int e = 0; e < kVec; ++e) nrm[e] = __ldg(J.norms + c0 + e);
        const char* base = static_cast<const char*>(J.W) + (size_t)c0 * 2u;
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {   // at most eight sampled rows per thread (256 rows over 32 lanes)
            const int64_t i = my + (int64_t)u * lanes;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (i < n_sampled) v[u] = ld_stream16_ro(base + (size_t)(step / 2 + i * step) * stride);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) add_scores(v[u], nrm, acc);
        for (int64_t i = my + 8ll * lanes; i < n_sampled; i += lanes)
            add_scores(ld_stream16_ro(base + (size_t)(step / 2 + i * step) * stride), nrm, acc);
    }
    const double s = block_sum((acc[0] + acc[1]) + (acc[2] + acc[3]), red);
    if (threadIdx.x == 0) {
        atomicAdd(&J.ctrl->est_sum, s * ((double)J.rows / (double)n_sampled));
        if (blockIdx.y == 0) *J.count_out = 0ull;
    }
}

// Lower edge of the ladders of job j: a little under the estimated threshold of the jobs that share it.
template <int NJ>
__device__ float ladder_floor(const OutlierJobList<NJ>& jobs, int j, float* sh) {
    if (threadIdx.x == 0) {
        const OutlierJob& J = jobs.job[j];
        double total = 0.0, numel = 0.0;
        for (int g = J.g_first; g <= J.g_last; ++g) {
            total = total + __ldcg(&jobs.job[g].ctrl->est_sum);
            numel = numel + (double)(jobs.job[g].rows * jobs.job[g].cols);
        }
        *sh = __double2float_rd((double)jobs.alpha * (total / numel) * 0.96875);
    }
    __syncthreads();
    const float v = *sh;
    __syncthreads();
    return v;
}

template <int NJ>
__global__ void __launch_bounds__(kOutThreads, 8) score_sum_ladder_kernel(const __grid_constant__ OutlierJobList<NJ> jobs,
                                                                          int n_ctiles) {
    __shared__ double red[32];
    __shared__ unsigned int cred[32];
    __shared__ float floor_sh;
    int t_begin, t_end;
    tile_share(n_ctiles, &t_begin, &t_end);
    int j = 0, j_floor = -1;
    float tau_lo = 0.0f;
    for (int tile = t_begin; tile < t_end; ++tile) {
        while (j + 1 < jobs.n && tile >= jobs.job[j + 1].ctile0) ++j;
        const OutlierJob& J = jobs.job[j];
        if (j != j_floor) {
            tau_lo = ladder_floor<NJ>(jobs, j, &floor_sh);
            j_floor = j;
        }
        const int local = tile - J.ctile0;
        const int chunk = local % J.chunks, band = local / J.chunks;
        const int c0 = chunk * kOutChunk + (int)threadIdx.x * kVec;
        const bool in_cols = c0 < (int)J.cols;
        float nrm[kVec];
        uint4 alo = make_uint4(0x80008000u, 0x80008000u, 0x80008000u, 0x80008000u), dep = make_uint4(0u, 0u, 0u, 0u);
        if (in_cols) {
            uint32_t a[kVec], d[kVec];
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                nrm[e] = __ldg(J.norms + c0 + e);
                a[e] = outlier_pattern(nrm[e], tau_lo);                                  // <= 0x8000
                d[e] = (a[e] + kLadder <= 0x8000u ? a[e] + kLadder : 0x8000u) - a[e];   // the ladder ends at 0x8000 at the latest
            }
            alo = make_uint4(a[0] | (a[1] << 16), a[2] | (a[3] << 16), a[4] | (a[5] << 16), a[6] | (a[7] << 16));
            dep = make_uint4(d[0] | (d[1] << 16), d[2] | (d[3] << 16), d[4] | (d[5] << 16), d[6] | (d[7] << 16));
        }
        uint32_t sure = 0u;
        uint32_t* lad = J.ladder + (size_t)c0 * kLadder;
        // One vector: its scores into the sum, its weights above the ladder counted, those on it noted.
        auto take = [&](const uint4& v, double (&acc)[4]) {
            add_scores(v, nrm, acc);
            const uint32_t t0 = (v.x | 0x80008000u) - alo.x, t1 = (v.y | 0x80008000u) - alo.y, t2 = (v.z | 0x80008000u) - alo.z,
                           t3 = (v.w | 0x80008000u) - alo.w;                         // bit 15 / 31: magnitude >= A_lo
            const uint32_t u0 = t0 - dep.x, u1 = t1 - dep.y, u2 = t2 - dep.z, u3 = t3 - dep.w;   // ... >= A_hi
            // flags of the eight elements on the top bits of the bytes of two words, merged into one for one popc
            const uint32_t ua = __byte_perm(u0, u1, 0x7531), ub = __byte_perm(u2, u3, 0x7531);
            sure += (uint32_t)__popc((ua & 0x80808080u) | ((ub >> 1) & 0x40404040u));
            // on the ladder: at or above A_lo but not above A_hi
            const uint32_t ta = __byte_perm(t0, t1, 0x7531), tb = __byte_perm(t2, t3, 0x7531);
            uint32_t hits = ((ta & ~ua) & 0x80808080u) | (((tb & ~ub) >> 1) & 0x40404040u);   // element e < 4 on bit 8e+7, e >= 4 on bit 8(e-4)+6
            while (hits != 0u) {   // a few per mille of the weights
                const int b = __ffs(hits) - 1;
                hits &= hits - 1u;
                const int e = (b >> 3) + ((b & 1) ? 0 : 4);
                const uint32_t tw = e < 2 ? t0 : (e < 4 ? t1 : (e < 6 ? t2 : t3));
                const uint32_t idx = ((e & 1) ? (tw >> 16) : tw) & 0x7FFFu;                   // magnitude - A_lo
                atomicAdd(&lad[e * kLadder + idx], 1u);
            }
        };
        const size_t stride = (size_t)J.ldw * 2u;
        // the tile's four bands of kOutTileRows rows give the same partial sums, in the same order, as the sum sweep
        for (int sub = 0; sub < kCntTileRows / kOutTileRows; ++sub) {
            const int64_t r0 = (int64_t)band * kCntTileRows + (int64_t)sub * kOutTileRows;
            if (r0 >= J.rows) break;   // (block-uniform)
            const int n_rows = (int)((r0 + kOutTileRows < J.rows ? r0 + kOutTileRows : J.rows) - r0);
            double acc[4] = {0.0, 0.0, 0.0, 0.0};
            if (in_cols) {
                const char* p = static_cast<const char*>(J.W) + ((size_t)r0 * (size_t)J.ldw + (size_t)c0) * 2u;
                int r = 0;
                for (; r + 4 <= n_rows; r += 4, p += 4 * stride) {
                    const uint4 v0 = ld_stream16_ro(p), v1 = ld_stream16_ro(p + stride), v2 = ld_stream16_ro(p + 2 * stride),
                                v3 = ld_stream16_ro(p + 3 * stride);
                    take(v0, acc);
                    take(v1, acc);
                    take(v2, acc);
                    take(v3, acc);
                }
                for (; r < n_rows; ++r, p += stride) take(ld_stream16_ro(p), acc);
            }
            const double blk = block_sum((acc[0] + acc[1]) + (acc[2] + acc[3]), red);
            if (threadIdx.x == 0) J.partial[(band * (kCntTileRows / kOutTileRows) + sub) * J.chunks + chunk] = blk;
        }
        // the tile's sure outliers
        sure = __reduce_add_sync(0xFFFFFFFFu, sure);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) cred[threadIdx.x >> 5] = sure;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long tot = 0;
            for (int i = 0; i < kOutThreads / 32; ++i) tot += cred[i];
            if (tot) atomicAdd(&J.ctrl->sure, tot);
        }
    }
}

// After the sweep, one CTA per matrix and chunk of kOutChunk columns: the threshold from the partial
// sums, then per column the ladder entries from A_j(tau) up.  The CTA that reports last writes the
// count and valid = 1 - iff tau lies on every column's ladder.
template <int NJ>
__global__ void __launch_bounds__(kOutThreads) outlier_finish_kernel(const __grid_constant__ OutlierJobList<NJ> jobs) {
    __shared__ double red[32];
    __shared__ float tau_sh, floor_sh;
    __shared__ unsigned long long total_sh;
    const int j = blockIdx.x, chunk = blockIdx.y;
    const OutlierJob& J = jobs.job[j];
    if (chunk >= J.chunks) return;
    const float tau = group_threshold<NJ>(jobs, j, chunk == 0, red, &tau_sh);
    const float tau_lo = ladder_floor<NJ>(jobs, j, &floor_sh);
    if (threadIdx.x == 0) total_sh = 0ull;
    __syncthreads();
    unsigned long long cnt = 0ull;
    bool ok = true;
    const int c_end = (chunk + 1) * kOutChunk < (int)J.cols ? (chunk + 1) * kOutChunk : (int)J.cols;
    for (int c = chunk * kOutChunk + (int)threadIdx.x; c < c_end; c += kOutThreads) {
        const float n = __ldg(J.norms + c);
        const uint32_t a_lo = outlier_pattern(n, tau_lo);
        const uint32_t a_hi = a_lo + kLadder <= 0x8000u ? a_lo + kLadder : 0x8000u;
        const uint32_t a_star = outlier_pattern(n, tau);
        if (a_star < a_lo || a_star > a_hi) {
            ok = false;
        } else {
            // the column's whole ladder in flight, then the entries from A(tau) up
            const uint4* lad4 = reinterpret_cast<const uint4*>(J.ladder + (size_t)c * kLadder);
            uint4 q[kLadder / 4];
#pragma unroll
            for (int i = 0; i < kLadder / 4; ++i) q[i] = __ldcg(&lad4[i]);
            const uint32_t first = a_star - a_lo, n_used = a_hi - a_lo;
#pragma unroll
            for (int i = 0; i < kLadder / 4; ++i) {
                const uint32_t w[4] = {q[i].x, q[i].y, q[i].z, q[i].w};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if ((uint32_t)(4 * i + e) >= first && (uint32_t)(4 * i + e) < n_used) cnt += w[e];
            }
        }
    }
    if (cnt) atomicAdd(&total_sh, cnt);
    const bool all_ok = __syncthreads_and(ok ? 1 : 0) != 0;
    if (threadIdx.x == 0) {
        if (total_sh) atomicAdd(&J.ctrl->lad_count, total_sh);
        if (!all_ok) atomicOr(&J.ctrl->invalid, 1);
        __threadfence();
        if (atomicAdd(&J.ctrl->done, 1) == J.chunks - 1) {   // every chunk has reported
            __threadfence();
            if (atomicOr(&J.ctrl->invalid, 0) == 0) {
                *J.count_out = __ldcg(&J.ctrl->sure) + atomicAdd(&J.ctrl->lad_count, 0ull);
                J.ctrl->valid = 1;
            }
        }
    }
}

template <int DT>
__global__ void score_kernel(const void* __restrict__ W, int64_t rows, int64_t cols, int64_t ldw,
                             const float* __restrict__ norms, float* __restrict__ out) {
    const int64_t nvec = (cols + kVec - 1) / kVec;
    const int64_t total = rows * nvec;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / nvec, c0 = (i % nvec) * kVec;
        Raw8<DT> v;
        load_vec<DT, true>(v, W, row * ldw, c0, cols);
#pragma unroll
        for (int e = 0; e < kVec; ++e)
            if (c0 + e < cols) out[row * cols + c0 + e] = __fmul_rn(norms[c0 + e], v.abs_f32(e));
    }
}

}  // namespace mosaic

using namespace mosaic;

extern "C" int mosaic_score(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype, const float* norms,
                            float* score_out, void* stream) {
    int rc = check_matrix(W, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (!norms || !score_out) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(norms) & 3u) || (reinterpret_cast<uintptr_t>(score_out) & 15u))
        return MOSAIC_ERR_MISALIGNED;
    if (rows == 0) return MOSAIC_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t total = rows * ((cols + kVec - 1) / kVec);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    if (dtype == MOSAIC_BF16)
        score_kernel<MOSAIC_BF16><<<(unsigned)blocks, 256, 0, st>>>(W, rows, cols, ldw, norms, score_out);
    else
        score_kernel<MOSAIC_F32><<<(unsigned)blocks, 256, 0, st>>>(W, rows, cols, ldw, norms, score_out);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

static int validate_outlier(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype, const float* norms,
                            const int64_t* outlier_count_out, const double* score_sum_out) {
    int rc = check_matrix(W, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (rows == 0) return MOSAIC_ERR_INVALID_ARG;
    if (!norms || !outlier_count_out) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(outlier_count_out) & 7u) || (reinterpret_cast<uintptr_t>(score_sum_out) & 7u) ||
        (reinterpret_cast<uintptr_t>(norms) & 3u))
        return MOSAIC_ERR_MISALIGNED;
    if (outlier_tiles(rows, cols) > 0x3FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
    return MOSAIC_OK;
}

// Resident CTAs per SM of a kernel, looked up once per device.
template <class K>
static int cached_occupancy(DeviceCache& cache, K kernel) {
    return cache.get([&]() -> int {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kOutThreads, 0) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = 4;
        }
        return n;
    });
}

// `lean`: every job is bf16 with cols % 8 == 0 (n_ctiles = tiles of the bf16 count sweep).
template <int NJ>
static int launch_outlier(const OutlierJobList<NJ>& list, int64_t n_tiles, int64_t n_ctiles, int dtype, bool lean,
                          cudaStream_t st) {
    static DeviceCache occ[7];   // occupancy is a property of one device's copy of a kernel
    int64_t g1, g2;
    if (lean && list.job[0].ctrl != nullptr) {
        // single sweep: estimates, the summing sweep with its ladders, the per-matrix finish; the count
        // sweep follows for the matrices the ladders did not settle (its CTAs skip the others at once)
        g1 = (int64_t)sm_count() * cached_occupancy(occ[6], score_sum_ladder_kernel<NJ>);
        g2 = (int64_t)sm_count() * cached_occupancy(occ[1], outlier_count_bf16_kernel<NJ>);
        if (g1 > n_ctiles) g1 = n_ctiles;
        if (g2 > n_ctiles) g2 = n_ctiles;
        outlier_estimate_kernel<NJ><<<dim3((unsigned)list.n, kEstParts), kOutThreads * kEstRowLanes, 0, st>>>(list);
        MOSAIC_LAUNCH_CHECK();
        score_sum_ladder_kernel<NJ><<<(unsigned)g1, kOutThreads, 0, st>>>(list, (int)n_ctiles);
        MOSAIC_LAUNCH_CHECK();
        int max_chunks = 1;
        for (int m = 0; m < list.n; ++m) max_chunks = list.job[m].chunks > max_chunks ? list.job[m].chunks : max_chunks;
        outlier_finish_kernel<NJ><<<dim3((unsigned)list.n, (unsigned)max_chunks), kOutThreads, 0, st>>>(list);
        MOSAIC_LAUNCH_CHECK();
        outlier_count_bf16_kernel<NJ><<<(unsigned)g2, kOutThreads, 0, st>>>(list, (int)n_ctiles);
    } else if (lean) {
        g1 = (int64_t)sm_count() * cached_occupancy(occ[0], score_sum_bf16_kernel<NJ>);
        g2 = (int64_t)sm_count() * cached_occupancy(occ[1], outlier_count_bf16_kernel<NJ>);
        if (g1 > n_tiles) g1 = n_tiles;
        if (g2 > n_ctiles) g2 = n_ctiles;
        score_sum_bf16_kernel<NJ><<<(unsigned)g1, kOutThreads, 0, st>>>(list, (int)n_tiles);
        MOSAIC_LAUNCH_CHECK();
        outlier_count_bf16_kernel<NJ><<<(unsigned)g2, kOutThreads, 0, st>>>(list, (int)n_ctiles);
    } else if (dtype == MOSAIC_BF16) {
        g1 = (int64_t)sm_count() * cached_occupancy(occ[2], score_sum_kernel<MOSAIC_BF16, NJ>);
        g2 = (int64_t)sm_count() * cached_occupancy(occ[3], outlier_count_kernel<MOSAIC_BF16, NJ>);
        if (g1 > n_tiles) g1 = n_tiles;
        if (g2 > n_tiles) g2 = n_tiles;
        score_sum_kernel<MOSAIC_BF16, NJ><<<(unsigned)g1, kOutThreads, 0, st>>>(list, (int)n_tiles);
        MOSAIC_LAUNCH_CHECK();
        outlier_count_kernel<MOSAIC_BF16, NJ><<<(unsigned)g2, kOutThreads, 0, st>>>(list, (int)n_tiles);
    } else {
        g1 = (int64_t)sm_count() * cached_occupancy(occ[4], score_sum_kernel<MOSAIC_F32, NJ>);
        g2 = (int64_t)sm_count() * cached_occupancy(occ[5], outlier_count_kernel<MOSAIC_F32, NJ>);
        if (g1 > n_tiles) g1 = n_tiles;
        if (g2 > n_tiles) g2 = n_tiles;
        score_sum_kernel<MOSAIC_F32, NJ><<<(unsigned)g1, kOutThreads, 0, st>>>(list, (int)n_tiles);
        MOSAIC_LAUNCH_CHECK();
        outlier_count_kernel<MOSAIC_F32, NJ><<<(unsigned)g2, kOutThreads, 0, st>>>(list, (int)n_tiles);
    }
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

extern "C" size_t mosaic_outlier_ratio_workspace_bytes(int64_t rows, int64_t cols) {
    if (rows <= 0 || cols <= 0) return 256;
    return align_up(sizeof(double) * (size_t)outlier_tiles(rows, cols), 256);
}

extern "C" int mosaic_outlier_ratio(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                    const float* norms, float alpha, int64_t* outlier_count_out, double* score_sum_out,
                                    void* ws, size_t ws_bytes, void* stream) {
    const int rc = validate_outlier(W, rows, cols, ldw, dtype, norms, outlier_count_out, score_sum_out);
    if (rc != MOSAIC_OK) return rc;
    if (!ws) return MOSAIC_ERR_NULL_PTR;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
    if (ws_bytes < mosaic_outlier_ratio_workspace_bytes(rows, cols)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    OutlierJobList<1> one;
    one.n = 1;
    one.alpha = alpha;
    one.job[0] = OutlierJob{W, norms, reinterpret_cast<unsigned long long*>(outlier_count_out), score_sum_out,
                            static_cast<double*>(ws), rows, cols, ldw, 0, (int)((cols + kOutChunk - 1) / kOutChunk), 0, 0, 0,
                            nullptr, nullptr};
    return launch_outlier<1>(one, outlier_tiles(rows, cols), outlier_count_tiles(rows, cols), dtype,
                             dtype == MOSAIC_BF16 && cols % kVec == 0, static_cast<cudaStream_t>(stream));
}

// Single-sweep scratch of one matrix: its bookkeeping block and kLadder counters per column.
static size_t ladder_bytes(int64_t cols) {
    return cols > 0 ? align_up(256 + sizeof(uint32_t) * (size_t)kLadder * (size_t)cols, 256) : 256;
}

extern "C" size_t mosaic_outlier_ratio_batch_workspace_bytes(const mosaic_outlier_job* jobs, int64_t n_jobs) {
    size_t total = 256;
    if (jobs == nullptr) return total;
    for (int64_t i = 0; i < n_jobs; ++i)
        total += mosaic_outlier_ratio_workspace_bytes(jobs[i].rows, jobs[i].cols) + ladder_bytes(jobs[i].cols);
    return total;
}

// The batched sweeps.  group_of == nullptr: every job has its own threshold (Eq. 6).  Otherwise adjacent
// jobs with equal group_of share one threshold (Eq. 3-4); a group never straddles two launches.
static int outlier_batch(const mosaic_outlier_job* jobs, const int32_t* group_of, int64_t n_jobs, int dtype, float alpha,
                         void* ws, size_t ws_bytes, void* stream) {
    if (n_jobs < 0) return MOSAIC_ERR_INVALID_ARG;
    if (n_jobs == 0) return MOSAIC_OK;
    if (jobs == nullptr || ws == nullptr) return MOSAIC_ERR_NULL_PTR;
    for (int64_t i = 0; i < n_jobs; ++i) {
        const mosaic_outlier_job& j = jobs[i];
        const int rc = validate_outlier(j.W, j.rows, j.cols, j.ldw, dtype, j.norms, j.outlier_count_out, j.score_sum_out);
        if (rc != MOSAIC_OK) return rc;
    }
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
    if (ws_bytes < mosaic_outlier_ratio_batch_workspace_bytes(jobs, n_jobs)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    auto group_end = [&](int64_t i) -> int64_t {   // one past the last job of the group that starts at i
        int64_t e = i + 1;
        if (group_of != nullptr)
            while (e < n_jobs && group_of[e] == group_of[i]) ++e;
        return e;
    };
    if (group_of != nullptr)
        for (int64_t i = 0; i < n_jobs; i = group_end(i))
            if (group_end(i) - i > kOutBatch) return MOSAIC_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // host staging of the kernel parameter (on the heap, one per call, so concurrent callers do not meet)
    std::unique_ptr<OutlierJobList<kOutBatch>> list_mem(new (std::nothrow) OutlierJobList<kOutBatch>);
    if (!list_mem) return MOSAIC_ERR_INVALID_ARG;
    OutlierJobList<kOutBatch>& list = *list_mem;
    char* wsp = static_cast<char*>(ws);
    bool lean = dtype == MOSAIC_BF16;
    for (int64_t m = 0; m < n_jobs; ++m) lean = lean && jobs[m].cols % kVec == 0;
    // the single-sweep scratch lies behind all partial sums
    char* lad = static_cast<char*>(ws);
    for (int64_t m = 0; m < n_jobs; ++m) lad += mosaic_outlier_ratio_workspace_bytes(jobs[m].rows, jobs[m].cols);
    int64_t i = 0;
    while (i < n_jobs) {
        list.n = 0;
        list.alpha = alpha;
        int64_t tiles = 0, ctiles = 0;
        char* lad_begin = lad;
        while (i < n_jobs) {
            const int64_t e = group_end(i);
            int64_t g_tiles = 0;
            for (int64_t m = i; m < e; ++m) g_tiles += outlier_tiles(jobs[m].rows, jobs[m].cols);
            if (list.n + (e - i) > kOutBatch || tiles + g_tiles > 0x3FFFFFFF) break;
            const int g_first = list.n, g_last = list.n + (int)(e - i) - 1;
            for (int64_t m = i; m < e; ++m) {
                const mosaic_outlier_job& j = jobs[m];
                list.job[list.n++] = OutlierJob{j.W, j.norms, reinterpret_cast<unsigned long long*>(j.outlier_count_out),
                                                j.score_sum_out, reinterpret_cast<double*>(wsp), j.rows, j.cols, j.ldw,
                                                (int)tiles, (int)((j.cols + kOutChunk - 1) / kOutChunk), (int)ctiles,
                                                g_first, g_last, lean ? reinterpret_cast<OutlierCtrl*>(lad) : nullptr,
                                                lean ? reinterpret_cast<uint32_t*>(lad + 256) : nullptr};
                lad += ladder_bytes(j.cols);
                wsp += mosaic_outlier_ratio_workspace_bytes(j.rows, j.cols);
                tiles += outlier_tiles(j.rows, j.cols);
                ctiles += outlier_count_tiles(j.rows, j.cols);
            }
            i = e;
        }
        if (list.n == 0) return MOSAIC_ERR_INVALID_ARG;   // a single group too large for one launch
        if (lean) MOSAIC_CUDA_TRY(cudaMemsetAsync(lad_begin, 0, (size_t)(lad - lad_begin), st));   // the ladders start at zero
        const int rc = launch_outlier<kOutBatch>(list, tiles, ctiles, dtype, lean, st);
        if (rc != MOSAIC_OK) return rc;
    }
    return MOSAIC_OK;
}

extern "C" int mosaic_outlier_ratio_batch(const mosaic_outlier_job* jobs, int64_t n_jobs, int dtype, float alpha, void* ws,
                                          size_t ws_bytes, void* stream) {
    return outlier_batch(jobs, nullptr, n_jobs, dtype, alpha, ws, ws_bytes, stream);
}

extern "C" int mosaic_outlier_ratio_grouped(const mosaic_outlier_job* jobs, const int32_t* group_of, int64_t n_jobs, int dtype,
                                            float alpha, void* ws, size_t ws_bytes, void* stream) {
    if (n_jobs > 0 && group_of == nullptr) return MOSAIC_ERR_NULL_PTR;
    return outlier_batch(jobs, group_of, n_jobs, dtype, alpha, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------
// mosaic_outlier_ratio_static: the same computation with the scratch memory built into the
// library, for callers that have no device allocator to take a workspace from.
// ------------------------------------------------------------------------------------------
namespace mosaic {

// Scratch of mosaic_outlier_ratio_static.  Every device that loads the library carries these
// 64 KiB until the process exits.  It holds one fp64 partial sum per tile (1024 columns by 64
// rows) of the first sweep: room for matrices of up to 8192 tiles, i.e. half a billion weights.
constexpr size_t kStaticScratchBytes = MOSAIC_OUTLIER_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_outlier_scratch[kStaticScratchBytes];

// Device address of g_outlier_scratch on the current device.  In host code the array's name is
// only a handle for the runtime, not something a kernel can dereference, so the address is asked
// for once per device (with that device current) and remembered.
static int static_scratch_address(void** out) {
    // One slot per device.  Two host threads that race on a device's first call both look the
    // address up and store the same value.  cudaDeviceReset() destroys the context the address
    // belongs to: a process that resets a device must not call this entry point on it afterwards.
    static std::atomic<void*> cached[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return MOSAIC_ERR_CUDA;
    if (dev < kMaxDevices) {
        void* hit = cached[dev].load(std::memory_order_acquire);
        if (hit != nullptr) {
            *out = hit;
            return MOSAIC_OK;
        }
    }
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_outlier_scratch) != cudaSuccess || p == nullptr) {
        (void)cudaGetLastError();
        return MOSAIC_ERR_CUDA;
    }
    if (dev < kMaxDevices) cached[dev].store(p, std::memory_order_release);
    *out = p;
    return MOSAIC_OK;
}

}  // namespace mosaic

extern "C" size_t mosaic_outlier_ratio_static_max_workspace_bytes(void) { return mosaic::kStaticScratchBytes; }

extern "C" int mosaic_outlier_ratio_static(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                           const float* norms, float alpha, int64_t* outlier_count_out,
                                           double* score_sum_out, void* stream) {
    // every argument error first, so that a bad call costs no CUDA work at all
    int rc = validate_outlier(W, rows, cols, ldw, dtype, norms, outlier_count_out, score_sum_out);
    if (rc != MOSAIC_OK) return rc;
    if (mosaic_outlier_ratio_workspace_bytes(rows, cols) > kStaticScratchBytes) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != MOSAIC_OK) return rc;
    // Nothing in the scratch has to start at zero: every partial sum is written by the first sweep
    // before the second reads it, so what an earlier call left behind is harmless.
    return mosaic_outlier_ratio(W, rows, cols, ldw, dtype, norms, alpha, outlier_count_out, score_sum_out, scratch,
                                kStaticScratchBytes, stream);
}
