// mosaic_prune_unstructured: per output row, exact selection of the k entries
// that come first under (weight metric ascending, column ascending), fused with
// the zeroing write and the keep-bitmask (Section 4.1.3, unstructured
// projection pruning; weight metric of Eq. 5).
//
// One CTA works on one row at a time.  Thread t owns the vectors
// v*NT + t (8 adjacent columns each), so the norms of its columns live in
// registers for the whole kernel and the row is read from HBM exactly once:
// the raw weights and their 32-bit score keys stay in registers across the
// selection passes.  Scores are >= +0, so the fp32 bit pattern is an order
// preserving unsigned key.
//
// Selection = most-significant-digit radix select on the key with shared-memory
// histograms: digits of 11, 10 and 10 bits (bits 30..20, 19..10, 9..0; bit 31 is
// 0 for every valid key).  After each histogram a block-wide scan finds the bin
// that holds the k-th smallest key and the rank still to resolve inside it.
// After the third digit the threshold key T is exact; q = how many entries
// equal to T must still be pruned.  If q is all of them the row is finished
// with a plain compare; otherwise a block-wide ordered prefix count over the
// columns prunes the q lowest-indexed ties.
#include "common.cuh"

namespace mosaic {

constexpr int kBins1 = 2048;  // first digit: bits 30..20
constexpr int kBins23 = 1024; // second / third digit

struct SelectResult {
    uint32_t bin, rank, count;
};

// Block-wide: find the bin b with  cum(b-1) < rank <= cum(b)  in hist[0..NB), clear the
// histogram for the next pass, and return (b, rank - cum(b-1), hist[b]).
template <int NT, int NB>
__device__ __forceinline__ SelectResult find_bin(uint32_t* hist, uint32_t* warp_tot, SelectResult* sel, uint32_t rank) {
    constexpr int BPT = (NB + NT - 1) / NT;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t local[BPT];
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int b = tid * BPT + i;
        local[i] = (b < NB) ? hist[b] : 0u;
        if (b < NB) hist[b] = 0u;
        sum += local[i];
    }
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    uint32_t base = incl - sum;
    for (int w = 0; w < wid; ++w) base += warp_tot[w];
    if (base < rank && rank <= base + sum) {
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            if (rank <= base + local[i]) {
                sel->bin = (uint32_t)(tid * BPT + i);
                sel->rank = rank - base;
                sel->count = local[i];
                break;
            }
            base += local[i];
        }
    }
    __syncthreads();
    return *sel;
}

// Block-wide exclusive prefix of a per-thread count, in thread order.  Returns the
// exclusive prefix; *total receives the block total.
template <int NT>
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += n;
    }
    __syncthreads();
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    uint32_t base = incl - v, tot = 0;
    for (int w = 0; w < NT / 32; ++w) {
        const uint32_t t = warp_tot[w];
        if (w < wid) base += t;
        tot += t;
    }
    *total = tot;
    return base;
}

template <int DT, int V, int NT>
__global__ void __launch_bounds__(NT) prune_rows_kernel(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw,
                                                         const float* __restrict__ norms, int k,
                                                         uint8_t* __restrict__ mask_bytes, int mask_row_bytes) {
    __shared__ uint32_t hist[kBins1];
    __shared__ uint32_t warp_tot[32];
    __shared__ SelectResult sel;
    const int tid = threadIdx.x;
    const int nvec = (cols + kVec - 1) / kVec;

    float nrm[V][kVec];
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const int c = (v * NT + tid) * kVec + e;
            nrm[v][e] = (c < cols) ? norms[c] : 0.0f;
        }
    for (int b = tid; b < kBins1; b += NT) hist[b] = 0u;
    __syncthreads();

    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        Raw8<DT> raw[V];
        uint32_t key[V][kVec];
        const int64_t row_off = row * ldw;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vec = v * NT + tid;
            if (vec < nvec) load_vec<DT, false>(raw[v], W_in, row_off, (int64_t)vec * kVec, cols);
            else raw[v].clear();
        }
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                const int c = (v * NT + tid) * kVec + e;
                const uint32_t s = __float_as_uint(__fmul_rn(nrm[v][e], raw[v].abs_f32(e)));
                key[v][e] = (c < cols) ? s : 0xFFFFFFFFu;   // padding never selected (valid keys have bit 31 = 0)
            }

        uint32_t T = 0u, q = 0u, n_eq = 0u;
        if (k > 0) {
            // digit 1: bits 30..20
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int e = 0; e < kVec; ++e)
                    if (!(key[v][e] & 0x80000000u)) atomicAdd(&hist[key[v][e] >> 20], 1u);
            __syncthreads();
            SelectResult r = find_bin<NT, kBins1>(hist, warp_tot, &sel, (uint32_t)k);
            uint32_t prefix = r.bin << 20;
            // digit 2: bits 19..10 of the keys whose bits 31..20 match
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int e = 0; e < kVec; ++e)
                    if ((key[v][e] & 0xFFF00000u) == prefix) atomicAdd(&hist[(key[v][e] >> 10) & 0x3FFu], 1u);
            __syncthreads();
            r = find_bin<NT, kBins23>(hist, warp_tot, &sel, r.rank);
            prefix |= r.bin << 10;
            // digit 3: bits 9..0
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int e = 0; e < kVec; ++e)
                    if ((key[v][e] & 0xFFFFFC00u) == prefix) atomicAdd(&hist[key[v][e] & 0x3FFu], 1u);
            __syncthreads();
            r = find_bin<NT, kBins23>(hist, warp_tot, &sel, r.rank);
            T = prefix | r.bin;
            q = r.rank;      // entries equal to T that are pruned (1 <= q <= n_eq)
            n_eq = r.count;
        }

        // prune flags
        uint32_t pruned[V];
#pragma unroll
        for (int v = 0; v < V; ++v) {
            pruned[v] = 0u;
            if (k > 0) {
#pragma unroll
                for (int e = 0; e < kVec; ++e) pruned[v] |= (key[v][e] < T || (q == n_eq && key[v][e] == T)) ? (1u << e) : 0u;
            }
        }
        if (k > 0 && q != n_eq) {
            // ties at the threshold: prune the q lowest-indexed entries equal to T
            uint32_t before = 0u;  // ties in earlier vector slots (all threads)
#pragma unroll
            for (int v = 0; v < V; ++v) {
                uint32_t eq = 0u;
#pragma unroll
                for (int e = 0; e < kVec; ++e) eq |= (key[v][e] == T) ? (1u << e) : 0u;
                uint32_t total;
                uint32_t idx = before + block_excl_scan<NT>(__popc(eq), warp_tot, &total);
#pragma unroll
                for (int e = 0; e < kVec; ++e)
                    if (eq & (1u << e)) {
                        if (idx < q) pruned[v] |= (1u << e);
                        ++idx;
                    }
                before += total;
            }
        }

        // write W' and the keep bitmask
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vec = v * NT + tid;
            const int c0 = vec * kVec;
            if (vec < nvec) {
#pragma unroll
                for (int e = 0; e < kVec; ++e)
                    if (pruned[v] & (1u << e)) raw[v].zero(e);
                if (c0 + kVec <= cols) {
                    raw[v].store((char*)W_out + (row_off + c0) * (DT == MOSAIC_F32 ? 4 : 2));
                } else {
#pragma unroll
                    for (int e = 0; e < kVec; ++e)
                        if (c0 + e < cols) raw[v].put_scalar(e, W_out, row_off + c0 + e);
                }
            }
            if (mask_bytes != nullptr && vec < mask_row_bytes) {
                uint32_t keep = 0u;
                if (vec < nvec) {
                    const int nvalid = (cols - c0 < kVec) ? cols - c0 : kVec;
                    keep = ~pruned[v] & ((1u << nvalid) - 1u);
                }
                mask_bytes[row * mask_row_bytes + vec] = (uint8_t)keep;
            }
        }
    }
}

template <int DT, int V, int NT>
static int launch_prune(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw, const float* norms, int k,
                        uint32_t* mask, cudaStream_t st) {
    static int blocks_per_sm = 0;
    if (blocks_per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, prune_rows_kernel<DT, V, NT>, NT, 0) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = 1;
        }
        blocks_per_sm = n;
    }
    int64_t grid = (int64_t)sm_count() * blocks_per_sm;
    if (grid > rows) grid = rows;
    const int words = (cols + 31) / 32;
    prune_rows_kernel<DT, V, NT><<<(unsigned)grid, NT, 0, st>>>(W_in, W_out, rows, cols, ldw, norms, k,
                                                               reinterpret_cast<uint8_t*>(mask), words * 4);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

template <int DT>
static int dispatch_prune(const void* W_in, void* W_out, int64_t rows, int cols, int64_t ldw, const float* norms, int k,
                          uint32_t* mask, cudaStream_t st) {
    const int nvec = (cols + kVec - 1) / kVec;
#define MOSAIC_PRUNE_CASE(V, NT) return launch_prune<DT, V, NT>(W_in, W_out, rows, cols, ldw, norms, k, mask, st)
    if (nvec <= 32) MOSAIC_PRUNE_CASE(1, 32);
    if (nvec <= 64) MOSAIC_PRUNE_CASE(1, 64);
    if (nvec <= 128) MOSAIC_PRUNE_CASE(1, 128);
    if (nvec <= 256) MOSAIC_PRUNE_CASE(1, 256);
    if (nvec <= 2 * 256) MOSAIC_PRUNE_CASE(2, 256);
    if (nvec <= 3 * 256) MOSAIC_PRUNE_CASE(3, 256);
    if (nvec <= 4 * 256) MOSAIC_PRUNE_CASE(4, 256);
    if (nvec <= 5 * 256) MOSAIC_PRUNE_CASE(5, 256);
    if (nvec <= 6 * 256) MOSAIC_PRUNE_CASE(6, 256);
    if (nvec <= 7 * 256) MOSAIC_PRUNE_CASE(7, 256);
    if (nvec <= 8 * 256) MOSAIC_PRUNE_CASE(8, 256);
    if (nvec <= 5 * 512) MOSAIC_PRUNE_CASE(5, 512);
    if (nvec <= 6 * 512) MOSAIC_PRUNE_CASE(6, 512);
    if (nvec <= 7 * 512) MOSAIC_PRUNE_CASE(7, 512);
    if (nvec <= 8 * 512) MOSAIC_PRUNE_CASE(8, 512);
    if (nvec <= 5 * 1024) MOSAIC_PRUNE_CASE(5, 1024);
    if (nvec <= 6 * 1024) MOSAIC_PRUNE_CASE(6, 1024);
    if (nvec <= 7 * 1024) MOSAIC_PRUNE_CASE(7, 1024);
    if (nvec <= 8 * 1024) MOSAIC_PRUNE_CASE(8, 1024);
#undef MOSAIC_PRUNE_CASE
    return MOSAIC_ERR_INVALID_ARG;
}

}  // namespace mosaic

using namespace mosaic;

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
