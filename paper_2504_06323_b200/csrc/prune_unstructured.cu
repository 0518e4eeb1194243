// mosaic_prune_unstructured: per output row, exact selection of the k entries
// that come first under (weight metric ascending, column ascending), fused with
// the zeroing write and the keep-bitmask (Section 4.1.3, unstructured
// projection pruning; weight metric of Eq. 5).
//
// One CTA works on one row at a time and walks rows blockIdx.x, +gridDim.x, ...
// Thread t owns the vectors v*nt + t (8 adjacent columns each).  A row is read
// from HBM exactly once and the next row of the CTA is already in flight while
// the current one is selected.  Scores are >= +0, so the fp32 bit pattern of a
// score is an order preserving unsigned key.  The result of the selection is
// the exact k-th smallest key T of the row plus the tie quota q (how many
// entries equal to T are pruned, lowest column first).
//
// Rows of one projection share the norms and k, so their thresholds are close.
// Every kernel here therefore first tries a *window* [lo, lo + 2^w) of key
// space that should contain T: it counts the keys below lo, builds a histogram
// of the few keys inside, and only those take part in the selection.  A window
// comes from the previous rows of the CTA or, without one or after a miss,
// from the matching quantile of one key per thread.  The full radix select over
// all keys (digits of 11, 10 and 10 bits) remains as the exact fallback; all
// paths give the same bits.
//
// prune_rows_kernel here is the general kernel: any dtype, any shape, scores of all entries in
// fp32.  bf16 rows of 2048..16384 columns (cols % 8 == 0, 0 < k < cols) - the shapes of a model's
// projections - go to the row-group kernel of prune_warp.cu instead, which classifies weights in
// the bf16 domain and scores only the few near the threshold.
#include <memory>
#include <new>
#include <vector>

#include "prune_jobs.cuh"
#include "select.cuh"

namespace mosaic {

constexpr int kListCap = kBins1;  // candidate list shares the histogram's storage
constexpr int kTrackBits = 21;    // width (log2, in key units) of a window carried from row to row
constexpr int kSampleBits = 23;   // width of the window around a sampled quantile

struct RowSelect {   // hand-over between warp 0 and the CTA during a window attempt
    uint32_t ok, T, q, n_eq, lo, bin;
};

// V = vectors per thread, NT = threads per CTA; V*NT*8 >= cols.
template <int DT, int V, int NT, int MINB>
__global__ void __launch_bounds__(NT, MINB) prune_rows_kernel(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw,
                                                         const float* __restrict__ norms, int k,
                                                         uint8_t* __restrict__ mask_bytes, int mask_row_bytes) {
    __shared__ __align__(16) uint32_t buf[kBins1];    // candidate list of a window attempt, or histogram of the full select
    __shared__ __align__(16) uint32_t whist[256];     // warp 0's digit histogram
    __shared__ __align__(16) uint32_t hist_win[256];  // top 8 bits of a window; zero between attempts
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t red[64];
    __shared__ uint32_t n_list;
    __shared__ SelectResult sel3;
    __shared__ RowSelect sel;
    constexpr int kWarps = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int nvec = (cols + kVec - 1) / kVec;
    const uint32_t uk = (uint32_t)k;

    float nrm[V][kVec];
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const int c = (v * NT + tid) * kVec + e;
            nrm[v][e] = (c < cols) ? norms[c] : __int_as_float(0x7F800000);
        }
    if (tid == 0) n_list = 0u;
    for (int b = tid; b < 256; b += NT) hist_win[b] = 0u;
    __syncthreads();

    Raw8<DT> raw[V], nxt[V];
    auto load_row = [&](Raw8<DT>(&dst)[V], int64_t row) {
        const int64_t row_off = row * ldw;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vec = v * NT + tid;
            if (vec < nvec) load_vec<DT, false>(dst[v], W_in, row_off, (int64_t)vec * kVec, cols);
            else dst[v].clear();
        }
    };
    // Score key of element (v, e) of the current row.  Columns past the end hold zero bits and
    // an infinite norm: their product is the canonical NaN 0x7FFFFFFF, the largest key there is,
    // and they come after every real column in the tie order, so no rank <= cols reaches them.
    // (The sign bit is cleared: norms are >= +0 by contract, and a negative one must not index past
    // the histograms - its rows then come out in an unspecified but memory-safe way.)
    auto key_of = [&](int v, int e) -> uint32_t {
        return __float_as_uint(__fmul_rn(nrm[v][e], raw[v].abs_f32(e))) & 0x7FFFFFFFu;
    };

    uint32_t center = 0u;
    bool have_center = false;
    uint32_t T = 0u, q = 0u, n_eq = 0u;

    // One attempt on the window [lo, lo + 2^w), w >= 9.  Every thread counts its keys below lo and
    // adds its keys inside the window to a 256-bin histogram of the window's top 8 bits; warp 0
    // finds the bin that holds rank k.  The few keys of that bin are then collected and, unless
    // there is just one, ranked by warp 0.  Block-uniform result: true and (T, q, n_eq) set, or
    // false (the k-th key is outside the window, or its bin overflows the list).
    auto try_window = [&](uint32_t lo, int w) -> bool {
        const uint32_t width = 1u << w;
        const int shift = w - 8;
        uint32_t n_below = 0u;
        uint32_t inside[V];   // bit e: element (v, e) lies in the window
#pragma unroll
        for (int v = 0; v < V; ++v) {
            inside[v] = 0u;
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                const uint32_t d = key_of(v, e) - lo;   // key < lo wraps to >= 2^31 (key, lo < 2^31)
                n_below += d >> 31;
                if (d < width) {
                    inside[v] |= 1u << e;
                    atomicAdd(&hist_win[d >> shift], 1u);
                }
            }
        }
        n_below = __reduce_add_sync(0xFFFFFFFFu, n_below);
        if (lane == 0) red[wid] = n_below;
        __syncthreads();
        if (wid == 0) {
            const uint32_t below = __reduce_add_sync(0xFFFFFFFFu, (lane < kWarps) ? red[lane] : 0u);
            uint4* h4 = reinterpret_cast<uint4*>(hist_win);
            const uint4 a = h4[lane * 2], b = h4[lane * 2 + 1];
            h4[lane * 2] = make_uint4(0u, 0u, 0u, 0u);       // left clean for the next attempt
            h4[lane * 2 + 1] = make_uint4(0u, 0u, 0u, 0u);
            const uint32_t c[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            uint32_t sum = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) sum += c[i];
            uint32_t incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += n;
            }
            uint32_t base = below + incl - sum;
            const bool mine = base < uk && uk <= base + sum;   // false everywhere if k is outside the window
            const unsigned m = __ballot_sync(0xFFFFFFFFu, mine);
            if (mine) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (base < uk && uk <= base + c[i]) {
                        sel.bin = (uint32_t)(lane * 8 + i);
                        sel.q = uk - base;      // rank inside the bin
                        sel.n_eq = c[i];        // keys in the bin
                    }
                    base += c[i];
                }
            }
            if (lane == 0) {
                sel.ok = m != 0u ? 1u : 0u;
                n_list = 0u;
            }
        }
        __syncthreads();
        if (sel.ok == 0u) return false;
        const uint32_t bin = sel.bin, r_bin = sel.q, n_bin = sel.n_eq;   // sel.T is the only field written below
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < kVec; ++e)
                if (inside[v] & (1u << e)) {
                    const uint32_t key = key_of(v, e);
                    if (((key - lo) >> shift) == bin) {
                        if (n_bin == 1u) {
                            sel.T = key;
                        } else {
                            const uint32_t pos = atomicAdd(&n_list, 1u);
                            if (pos < (uint32_t)kListCap) buf[pos] = key;
                        }
                    }
                }
        __syncthreads();
        if (n_bin == 1u) {
            T = sel.T;
            q = 1u;
            n_eq = 1u;
            return true;
        }
        if (n_bin > (uint32_t)kListCap) return false;
        if (wid == 0) {
            uint32_t t = 0u, qq = 0u, ne = 0u;
            const bool ok = warp_select(buf, n_bin, lo + (bin << shift), shift, r_bin, whist, &t, &qq, &ne);
            if (lane == 0) {
                sel.ok = ok ? 1u : 0u;
                sel.T = t;
                sel.q = qq;
                sel.n_eq = ne;
            }
        }
        __syncthreads();
        if (sel.ok == 0u) return false;
        T = sel.T;
        q = sel.q;
        n_eq = sel.n_eq;
        return true;
    };

    int64_t row = blockIdx.x;
    if (row < rows) load_row(nxt, row);
    for (; row < rows; row += gridDim.x) {
#pragma unroll
        for (int v = 0; v < V; ++v) raw[v] = nxt[v];
        if (row + gridDim.x < rows) load_row(nxt, row + gridDim.x);
        const int64_t row_off = row * ldw;

        if (k > 0) {
            bool done = false;
            if (have_center) {
                const uint32_t half = 1u << (kTrackBits - 1);
                done = try_window(center > half ? center - half : 0u, kTrackBits);
            }
            if (!done) {
                // window around the matching quantile of one key per thread
                const uint32_t n_s = (uint32_t)(nvec < NT ? nvec : NT);
                if ((uint32_t)tid < n_s) buf[tid] = key_of(0, 0);
                __syncthreads();
                if (wid == 0) {
                    uint32_t r_s = (uint32_t)(((uint64_t)uk * n_s + (uint32_t)cols / 2u) / (uint32_t)cols);
                    r_s = r_s < 1u ? 1u : (r_s > n_s ? n_s : r_s);
                    uint32_t t = 0u, qq = 0u, ne = 0u;
                    const bool ok = warp_select(buf, n_s, 0u, 31, r_s, whist, &t, &qq, &ne);
                    const uint32_t half = 1u << (kSampleBits - 1);
                    if (lane == 0) {
                        sel.ok = ok ? 1u : 0u;
                        sel.lo = t > half ? t - half : 0u;
                    }
                }
                __syncthreads();
                if (sel.ok != 0u) {
                    const uint32_t lo = sel.lo;
                    done = try_window(lo, kSampleBits);
                }
            }
            if (!done) {
                for (int b = tid; b < kBins1; b += NT) buf[b] = 0u;   // the list may have left entries
                __syncthreads();
                radix_select_row<V>(key_of, uk, buf, warp_tot, &sel3, NT, &T, &q, &n_eq);
            }
            center = have_center ? (uint32_t)(((uint64_t)center + T) >> 1) : T;
            have_center = true;
        }

        uint32_t pruned[V];
#pragma unroll
        for (int v = 0; v < V; ++v) pruned[v] = 0u;
        if (k > 0) prune_flags<V>(key_of, T, q, n_eq, warp_tot, NT, pruned);
        store_row<DT, V>(raw, pruned, W_out, row_off, cols, nvec, NT, mask_bytes, row * mask_row_bytes, mask_row_bytes);
    }
}


// True iff the row-group kernel (prune_warp.cu) takes rows of this shape.
static bool warp_kernel_takes(int dtype, int64_t cols, int64_t k) {
    return dtype == MOSAIC_BF16 && k > 0 && k < cols && prune_warp_takes(cols);
}

template <int DT, int V, int NT, int MINB>
static int launch_prune(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw, const float* norms, int k,
                        uint32_t* mask, cudaStream_t st) {
    static DeviceCache occupancy;
    const int blocks_per_sm = occupancy.get([&]() -> int {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, prune_rows_kernel<DT, V, NT, MINB>, NT, 0) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = 1;
        }
        return n;
    });
    int64_t grid = (int64_t)sm_count() * blocks_per_sm;
    if (grid > rows) grid = rows;
    const int words = (cols + 31) / 32;
    prune_rows_kernel<DT, V, NT, MINB><<<(unsigned)grid, NT, 0, st>>>(W_in, W_out, rows, cols, ldw, norms, k,
                                                               reinterpret_cast<uint8_t*>(mask), words * 4);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

template <int DT>
static int dispatch_prune(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw, const float* norms, int k,
                          uint32_t* mask, cudaStream_t st) {
    const int nvec = (cols + kVec - 1) / kVec;
    // (vectors per thread, threads per CTA, CTAs per SM the register budget is set for)
#define MOSAIC_PRUNE_CASE(V, NT, MINB) \
    return launch_prune<DT, V, NT, MINB>(W_in, W_out, rows, cols, ldw, norms, k, mask, st)
    if (nvec <= 32) MOSAIC_PRUNE_CASE(1, 32, 16);
    if (nvec <= 64) MOSAIC_PRUNE_CASE(1, 64, 16);
    if (nvec <= 128) MOSAIC_PRUNE_CASE(1, 128, 8);
    if (nvec <= 256) MOSAIC_PRUNE_CASE(1, 256, 4);
    if (nvec <= 2 * 256) MOSAIC_PRUNE_CASE(2, 256, 3);
    if (nvec <= 3 * 256) MOSAIC_PRUNE_CASE(3, 256, 3);
    if (nvec <= 2 * 512) MOSAIC_PRUNE_CASE(2, 512, 2);
    if (nvec <= 3 * 512) MOSAIC_PRUNE_CASE(3, 512, 1);
    if (nvec <= 4 * 512) MOSAIC_PRUNE_CASE(4, 512, 1);
    if (nvec <= 3 * 1024) MOSAIC_PRUNE_CASE(3, 1024, 1);
    if (nvec <= 4 * 1024) MOSAIC_PRUNE_CASE(4, 1024, 1);
    if (nvec <= 6 * 1024) MOSAIC_PRUNE_CASE(6, 1024, 1);
    if (nvec <= 8 * 1024) MOSAIC_PRUNE_CASE(8, 1024, 1);
#undef MOSAIC_PRUNE_CASE
    return MOSAIC_ERR_INVALID_ARG;
}

}  // namespace mosaic

using namespace mosaic;

extern "C" size_t mosaic_prune_unstructured_workspace_bytes(int64_t, int64_t) { return 0; }

// Argument checks of one pruning job (shared by the single and the batched entry point).
static int validate_prune(const void* W_in, void* W_out, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                          const float* norms, int64_t k, uint32_t* mask_out) {
    int rc = check_matrix(W_in, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (W_out != nullptr) {   // W_out == NULL: mask-only mode, the keep bitmask is the only output
        rc = check_matrix(W_out, rows, cols, ldw, dtype);
        if (rc != MOSAIC_OK) return rc;
    } else if (mask_out == nullptr) {
        return MOSAIC_ERR_NULL_PTR;
    }
    if (!norms) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(norms) & 3u) || (reinterpret_cast<uintptr_t>(mask_out) & 3u)) return MOSAIC_ERR_MISALIGNED;
    if (k < 0 || k > cols || cols > 65536) return MOSAIC_ERR_INVALID_ARG;
    if (rows > 0 && W_out != nullptr && W_in != W_out) {
        const size_t span = ((size_t)(rows - 1) * (size_t)ldw + (size_t)cols) * elem_size(dtype);
        const char *a = static_cast<const char*>(W_in), *b = static_cast<const char*>(W_out);
        if (a < b + span && b < a + span) return MOSAIC_ERR_ALIASING;
    }
    return MOSAIC_OK;
}

extern "C" int mosaic_prune_unstructured(const void* W_in, void* W_out, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                         const float* norms, int64_t k, uint32_t* mask_out, void* ws, size_t ws_bytes,
                                         void* stream) {
    (void)ws;
    (void)ws_bytes;
    const int rc = validate_prune(W_in, W_out, rows, cols, ldw, dtype, norms, k, mask_out);
    if (rc != MOSAIC_OK) return rc;
    if (rows == 0) return MOSAIC_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (warp_kernel_takes(dtype, cols, k)) {
        PruneJobList<1> one;
        one.n = 1;
        one.job[0] = PruneJob{static_cast<const uint16_t*>(W_in), static_cast<uint16_t*>(W_out), norms,
                              reinterpret_cast<uint8_t*>(mask_out), rows, ldw, 0, (int)k,
                              (int)((cols + 31) / 32) * 4};
        return launch_prune_warp(one, rows, (int)cols, st);
    }
    if (dtype == MOSAIC_BF16)
        return dispatch_prune<MOSAIC_BF16>(W_in, W_out, rows, (int)cols, ldw, norms, (int)k, mask_out, st);
    return dispatch_prune<MOSAIC_F32>(W_in, W_out, rows, (int)cols, ldw, norms, (int)k, mask_out, st);
}

// The batched call needs no scratch: the row-group kernel finds its windows itself.
extern "C" size_t mosaic_prune_unstructured_batch_workspace_bytes(const mosaic_prune_job*, int64_t, int) { return 256; }

extern "C" int mosaic_prune_unstructured_batch(const mosaic_prune_job* jobs, int64_t n_jobs, int dtype, void* ws,
                                               size_t ws_bytes, void* stream) {
    if (n_jobs < 0) return MOSAIC_ERR_INVALID_ARG;
    if (n_jobs == 0) return MOSAIC_OK;
    if (jobs == nullptr) return MOSAIC_ERR_NULL_PTR;
    for (int64_t i = 0; i < n_jobs; ++i) {
        const mosaic_prune_job& j = jobs[i];
        const int rc = validate_prune(j.W_in, j.W_out, j.rows, j.cols, j.ldw, dtype, j.norms, j.k, j.mask_out);
        if (rc != MOSAIC_OK) return rc;
    }
    (void)ws;
    (void)ws_bytes;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // jobs for the row-group kernel are launched together, one launch per distinct row length and
    // per kBatchJobs jobs; everything else goes through the single call
    std::vector<char> done((size_t)n_jobs, 0);
    // host staging of the kernel parameter (18 KB: on the heap, one per call, so concurrent callers do not meet)
    std::unique_ptr<PruneJobList<kBatchJobs>> list_mem(new (std::nothrow) PruneJobList<kBatchJobs>);
    if (!list_mem) return MOSAIC_ERR_INVALID_ARG;
    PruneJobList<kBatchJobs>& list = *list_mem;
    for (int64_t i = 0; i < n_jobs; ++i) {
        if (done[(size_t)i]) continue;
        const mosaic_prune_job& lead = jobs[i];
        const bool by_warp = lead.rows > 0 && warp_kernel_takes(dtype, lead.cols, lead.k);
        if (by_warp) {   // all jobs of this row length that the row-group kernel takes, kBatchJobs per launch
            list.n = 0;
            int64_t total_rows = 0;
            for (int64_t m = i; m < n_jobs; ++m) {
                const mosaic_prune_job& j = jobs[m];
                if (done[(size_t)m] || j.cols != lead.cols || j.rows <= 0 || !warp_kernel_takes(dtype, j.cols, j.k)) continue;
                done[(size_t)m] = 1;
                list.job[list.n] = PruneJob{static_cast<const uint16_t*>(j.W_in), static_cast<uint16_t*>(j.W_out), j.norms,
                                            reinterpret_cast<uint8_t*>(j.mask_out), j.rows, j.ldw, total_rows,
                                            (int)j.k, (int)((j.cols + 31) / 32) * 4};
                total_rows += j.rows;
                if (++list.n == kBatchJobs) {
                    const int rc = launch_prune_warp(list, total_rows, (int)lead.cols, st);
                    if (rc != MOSAIC_OK) return rc;
                    list.n = 0;
                    total_rows = 0;
                }
            }
            if (list.n > 0) {
                const int rc = launch_prune_warp(list, total_rows, (int)lead.cols, st);
                if (rc != MOSAIC_OK) return rc;
            }
            continue;
        }
        // short or very long rows, fp32, k = 0 or k = cols: the general kernel, one launch per job
        done[(size_t)i] = 1;
        const int rc = mosaic_prune_unstructured(lead.W_in, lead.W_out, lead.rows, lead.cols, lead.ldw, dtype, lead.norms,
                                                 lead.k, lead.mask_out, nullptr, 0, stream);
        if (rc != MOSAIC_OK) return rc;
    }
    return MOSAIC_OK;
}
