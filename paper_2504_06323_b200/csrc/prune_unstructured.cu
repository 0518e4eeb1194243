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
// Two kernels:
//   prune_rows_bf16_kernel  bf16 rows of 2048..16384 columns.  For a fixed
//       window the test "score key below lo" is, per column j, a test of the
//       weight's 15 magnitude bits against a bf16 bit pattern A_lo[j], because
//       the score norm_j*|w| is monotone in |w|.  The thresholds of the thread's
//       columns live in registers (two 16-bit lanes per word), and a row is
//       classified two weights per integer subtract, without ever forming the
//       scores.  The thresholds are conservative (computed with an approximate
//       reciprocal and widened by two bf16 steps); the weights that fall
//       between A_lo[j] and A_hi[j] - a few percent of the row - are the
//       candidates, and only they get an exact fp32 score.
//   prune_rows_kernel       any dtype, any shape; scores of all entries in fp32.
#include "select.cuh"

#ifndef MOSAIC_PRUNE_MINB_2X256
#define MOSAIC_PRUNE_MINB_2X256 3
#endif
#ifndef MOSAIC_FAST_MAX_CTAS
#define MOSAIC_FAST_MAX_CTAS 8
#endif

namespace mosaic {

#ifdef MOSAIC_PRUNE_STATS   // development aid: how often each selection path ran
__device__ unsigned long long g_prune_stats[8];
#define MOSAIC_STAT(i) do { if (threadIdx.x == 0) atomicAdd(&g_prune_stats[i], 1ull); } while (0)
#define MOSAIC_STAT_ADD(i, n) do { if (threadIdx.x == 0) atomicAdd(&g_prune_stats[i], (unsigned long long)(n)); } while (0)
#else
#define MOSAIC_STAT(i) do { } while (0)
#define MOSAIC_STAT_ADD(i, n) do { } while (0)
#endif

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
    auto key_of = [&](int v, int e) -> uint32_t {
        return __float_as_uint(__fmul_rn(nrm[v][e], raw[v].abs_f32(e)));
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
        MOSAIC_STAT_ADD(7, n_bin);
        if (n_bin == 1u) {
            MOSAIC_STAT(6);
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
            MOSAIC_STAT(0);
            if (have_center) {
                const uint32_t half = 1u << (kTrackBits - 1);
                done = try_window(center > half ? center - half : 0u, kTrackBits);
                MOSAIC_STAT(1);
                if (done) MOSAIC_STAT(2);
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
                MOSAIC_STAT(3);
                if (sel.ok != 0u) {
                    const uint32_t lo = sel.lo;
                    done = try_window(lo, kSampleBits);
                    if (done) MOSAIC_STAT(4);
                }
            }
            if (!done) {
                MOSAIC_STAT(5);
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

template <int DT, int V, int NT, int MINB>
static int launch_prune(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw, const float* norms, int k,
                        uint32_t* mask, cudaStream_t st) {
    static int blocks_per_sm = 0;
    if (blocks_per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, prune_rows_kernel<DT, V, NT, MINB>, NT, 0) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = 1;
        }
        blocks_per_sm = n;
    }
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
    if (nvec <= 2 * 256) MOSAIC_PRUNE_CASE(2, 256, MOSAIC_PRUNE_MINB_2X256);
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

#ifdef MOSAIC_PRUNE_STATS
extern "C" int mosaic_debug_prune_stats(unsigned long long* host_out, int reset) {
    if (cudaMemcpyFromSymbol(host_out, g_prune_stats, sizeof(unsigned long long) * 8) != cudaSuccess) return MOSAIC_ERR_CUDA;
    if (reset) {
        unsigned long long z[8] = {0};
        if (cudaMemcpyToSymbol(g_prune_stats, z, sizeof(z)) != cudaSuccess) return MOSAIC_ERR_CUDA;
    }
    return MOSAIC_OK;
}
#endif

extern "C" size_t mosaic_prune_unstructured_workspace_bytes(int64_t, int64_t) { return 0; }

extern "C" int mosaic_prune_unstructured(const void* W_in, void* W_out, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                         const float* norms, int64_t k, uint32_t* mask_out, void* ws, size_t ws_bytes,
                                         void* stream) {
    (void)ws;
    (void)ws_bytes;
    int rc = check_matrix(W_in, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    rc = check_matrix(W_out, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (!norms) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(norms) & 3u) || (reinterpret_cast<uintptr_t>(mask_out) & 3u)) return MOSAIC_ERR_MISALIGNED;
    if (k < 0 || k > cols || cols > 65536) return MOSAIC_ERR_INVALID_ARG;
    if (rows == 0) return MOSAIC_OK;
    if (W_in != W_out) {
        const size_t span = ((size_t)(rows - 1) * (size_t)ldw + (size_t)cols) * elem_size(dtype);
        const char *a = static_cast<const char*>(W_in), *b = static_cast<const char*>(W_out);
        if (a < b + span && b < a + span) return MOSAIC_ERR_ALIASING;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == MOSAIC_BF16)
        return dispatch_prune<MOSAIC_BF16>(W_in, W_out, rows, (int)cols, ldw, norms, (int)k, mask_out, st);
    return dispatch_prune<MOSAIC_F32>(W_in, W_out, rows, (int)cols, ldw, norms, (int)k, mask_out, st);
}
