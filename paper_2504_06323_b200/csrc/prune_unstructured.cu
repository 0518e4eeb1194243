// mosaic_prune_unstructured: per output row, exact selection of the k entries
// that come first under (weight metric ascending, column ascending), fused with
// the zeroing write and the keep-bitmask (Section 4.1.3, unstructured
// projection pruning; weight metric of Eq. 5).
//
// One CTA works on one row at a time and walks rows blockIdx.x, +gridDim.x, ...
// Thread t owns the vectors v*NT + t (8 adjacent columns each), so the norms of
// its columns live in registers for the whole kernel and the row is read from
// HBM exactly once: the raw weights stay in registers across the selection, and
// the next row of the CTA is already in flight (a second register set) while
// the current one is selected.  Scores are >= +0, so the fp32 bit pattern is an
// order preserving unsigned key.
//
// The result is the exact k-th smallest key T of the row plus the tie quota q
// (how many entries equal to T are pruned, lowest column first).  Three ways to
// get there, all exact, tried in order of cost:
//
//   1. tracked window.  Rows of one projection share the norms and k, so their
//      thresholds are close.  With a running estimate c of T the CTA counts the
//      keys below lo = c - 2^20 and collects the keys inside [lo, lo + 2^21) in
//      a shared-memory list (a few percent of the row).  If the k-th key lies in
//      the window, one warp finishes the selection on the list alone with an
//      8-bit-digit radix select.
//   2. sampled window.  Without an estimate (first row of a CTA) or after a
//      miss, the CTA selects the matching quantile of one key per thread and
//      opens a 2^23 window around it.
//   3. full radix select over all keys with shared-memory histograms: digits of
//      11, 10 and 10 bits (bits 30..20, 19..10, 9..0; bit 31 is 0 for every
//      valid key).  Always succeeds.
//
// If q is all of the ties the row is finished with a plain compare; otherwise a
// block-wide ordered prefix count over the columns prunes the q lowest-indexed
// ties.
#include "common.cuh"

#ifndef MOSAIC_PRUNE_MINB_2X256
#define MOSAIC_PRUNE_MINB_2X256 4
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

constexpr int kBins1 = 2048;      // first digit of the full select: bits 30..20
constexpr int kBins23 = 1024;     // second / third digit
constexpr int kListCap = kBins1;  // candidate list shares the histogram's storage
constexpr int kTrackBits = 21;    // width (log2, in key units) of the tracked window
constexpr int kSampleBits = 23;   // width of the window around a sampled quantile

struct SelectResult {
    uint32_t bin, rank, count;
};

struct RowSelect {   // hand-over between warp 0 and the CTA during a window attempt
    uint32_t ok, T, q, n_eq, lo, bin;
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

// One warp: the r-th smallest (1 <= r <= L) of list[0..L), whose entries all lie in
// [lo, lo + 2^w).  Radix select on d = key - lo with 8-bit digits from the top and a
// 256-bin histogram private to the warp.  Returns false if no bin holds the rank (a
// caller error, or keys outside the window); then nothing is written.
__device__ __forceinline__ bool warp_select(const uint32_t* list, uint32_t L, uint32_t lo, int w, uint32_t r,
                                            uint32_t* whist, uint32_t* T, uint32_t* q, uint32_t* n_eq) {
    const int lane = threadIdx.x & 31;
    uint32_t prefix = 0u, cnt = 0u;
    int top = w;   // low bits of d still undetermined
    while (top > 0) {
        const int nb = top >= 8 ? 8 : top;
        const int s = top - nb;
        const uint32_t dmask = (1u << nb) - 1u;
        uint4* wh4 = reinterpret_cast<uint4*>(whist);
        wh4[lane * 2] = make_uint4(0u, 0u, 0u, 0u);
        wh4[lane * 2 + 1] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
        for (uint32_t i = lane; i < L; i += 32) {
            const uint32_t d = list[i] - lo;
            if ((d >> top) == prefix) atomicAdd(&whist[(d >> s) & dmask], 1u);
        }
        __syncwarp();
        const uint4 a = wh4[lane * 2], b = wh4[lane * 2 + 1];
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
        uint32_t base = incl - sum;
        const bool mine = base < r && r <= base + sum;
        const unsigned m = __ballot_sync(0xFFFFFFFFu, mine);
        if (m == 0u) return false;
        uint32_t bin = 0u, rank = 0u, count = 0u;
        if (mine) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (count == 0u && r <= base + c[i]) {
                    bin = (uint32_t)(lane * 8 + i);
                    rank = r - base;
                    count = c[i];
                }
                base += c[i];
            }
        }
        const int src = __ffs(m) - 1;
        bin = __shfl_sync(0xFFFFFFFFu, bin, src);
        r = __shfl_sync(0xFFFFFFFFu, rank, src);
        cnt = __shfl_sync(0xFFFFFFFFu, count, src);
        prefix = (prefix << nb) | bin;
        top = s;
        __syncwarp();
    }
    *T = lo + prefix;
    *q = r;
    *n_eq = cnt;
    return true;
}

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
                // full radix select over all keys
                MOSAIC_STAT(5);
                for (int b = tid; b < kBins1; b += NT) buf[b] = 0u;
                __syncthreads();
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < kVec; ++e) {
                        atomicAdd(&buf[key_of(v, e) >> 20], 1u);
                    }
                __syncthreads();
                SelectResult r = find_bin<NT, kBins1>(buf, warp_tot, &sel3, uk);
                uint32_t prefix = r.bin << 20;
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < kVec; ++e) {
                        const uint32_t key = key_of(v, e);
                        if ((key & 0xFFF00000u) == prefix) atomicAdd(&buf[(key >> 10) & 0x3FFu], 1u);
                    }
                __syncthreads();
                r = find_bin<NT, kBins23>(buf, warp_tot, &sel3, r.rank);
                prefix |= r.bin << 10;
#pragma unroll
                for (int v = 0; v < V; ++v)
#pragma unroll
                    for (int e = 0; e < kVec; ++e) {
                        const uint32_t key = key_of(v, e);
                        if ((key & 0xFFFFFC00u) == prefix) atomicAdd(&buf[key & 0x3FFu], 1u);
                    }
                __syncthreads();
                r = find_bin<NT, kBins23>(buf, warp_tot, &sel3, r.rank);
                T = prefix | r.bin;
                q = r.rank;      // entries equal to T that are pruned (1 <= q <= n_eq)
                n_eq = r.count;
            }
            center = have_center ? (uint32_t)(((uint64_t)center + T) >> 1) : T;
            have_center = true;
        }

        // prune flags: key < T, and every key == T when all ties go
        uint32_t pruned[V];
        const uint32_t below = (q == n_eq) ? T + 1u : T;   // T < 2^31
#pragma unroll
        for (int v = 0; v < V; ++v) {
            pruned[v] = 0u;
            if (k > 0) {
#pragma unroll
                for (int e = 0; e < kVec; ++e) pruned[v] |= (key_of(v, e) < below) ? (1u << e) : 0u;
            }
        }
        if (k > 0 && q != n_eq) {
            // ties at the threshold: prune the q lowest-indexed entries equal to T
            uint32_t before = 0u;  // ties in earlier vector slots (all threads)
#pragma unroll
            for (int v = 0; v < V; ++v) {
                uint32_t eq = 0u;
#pragma unroll
                for (int e = 0; e < kVec; ++e) eq |= (key_of(v, e) == T) ? (1u << e) : 0u;
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
