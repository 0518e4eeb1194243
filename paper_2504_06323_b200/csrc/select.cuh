// Block- and warp-level building blocks of the per-row selection of
// mosaic_prune_unstructured: exact k-th smallest key of a row under
// (key ascending, column ascending), where a key is the fp32 bit pattern of a
// score >= +0 (weight metric of Eq. 5).
//
// A CTA of `nt` threads holds one row: thread t owns the vectors v*nt + t
// (8 adjacent columns each), v < V, and hands its keys out through a functor
// key_of(v, e).  Columns past the end of the row must yield 0x7FFFFFFF (the
// canonical NaN, the largest key): they come after every real column in the
// tie order, so no rank <= cols reaches them.
#pragma once
#include "common.cuh"

namespace mosaic {

constexpr int kBins1 = 2048;   // first digit of the full select: key bits 30..20
constexpr int kBins23 = 1024;  // second / third digit: bits 19..10, 9..0

struct SelectResult {
    uint32_t bin, rank, count;
};

// Block-wide over nt threads: the bin b with  cum(b-1) < rank <= cum(b)  in hist[0..NB),
// as (b, rank - cum(b-1), hist[b]).  The histogram is left cleared.
template <int NB>
__device__ __forceinline__ SelectResult find_bin(uint32_t* hist, uint32_t* warp_tot, SelectResult* sel, uint32_t rank,
                                                 int nt) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int bpt = (NB + nt - 1) / nt;
    const int b0 = tid * bpt;
    const int b1 = (b0 + bpt < NB) ? b0 + bpt : NB;
    uint32_t sum = 0u;
    for (int b = b0; b < b1; ++b) sum += hist[b];
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
        for (int b = b0; b < b1; ++b) {
            const uint32_t c = hist[b];
            if (rank <= base + c) {
                sel->bin = (uint32_t)b;
                sel->rank = rank - base;
                sel->count = c;
                break;
            }
            base += c;
        }
    }
    __syncthreads();
    for (int b = b0; b < b1; ++b) hist[b] = 0u;
    const SelectResult r = *sel;
    __syncthreads();   // histogram clean and *sel read before either is reused
    return r;
}

// Block-wide exclusive prefix of a per-thread count, in thread order.  Returns the
// exclusive prefix; *total receives the block total.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total, int nt) {
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
    uint32_t base = incl - v, tot = 0u;
    for (int w = 0; w < nt / 32; ++w) {
        const uint32_t t = warp_tot[w];
        if (w < wid) base += t;
        tot += t;
    }
    *total = tot;
    return base;
}

// One warp: the r-th smallest (1 <= r <= L) of list[0..L), whose entries all lie in
// [lo, lo + 2^w).  Radix select on d = key - lo with 8-bit digits from the top and a
// 256-bin histogram private to the warp.  T = the key, n_eq = how many entries equal
// it, q = the rank among those (1..n_eq).  Returns false if no bin holds the rank (a
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

// Full radix select over all keys of the row with shared-memory histograms: digits of
// 11, 10 and 10 bits.  hist[0..kBins1) must be zero on entry and is zero on exit.
// Always succeeds for 1 <= k <= cols.  T = k-th smallest key, n_eq = keys equal to T,
// q = how many of those are among the k smallest (1..n_eq).
template <int V, class KeyOf>
__device__ __forceinline__ void radix_select_row(KeyOf key_of, uint32_t k, uint32_t* hist, uint32_t* warp_tot,
                                                 SelectResult* sel, int nt, uint32_t* T, uint32_t* q, uint32_t* n_eq) {
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < kVec; ++e) atomicAdd(&hist[key_of(v, e) >> 20], 1u);
    __syncthreads();
    SelectResult r = find_bin<kBins1>(hist, warp_tot, sel, k, nt);
    uint32_t prefix = r.bin << 20;
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const uint32_t key = key_of(v, e);
            if ((key & 0xFFF00000u) == prefix) atomicAdd(&hist[(key >> 10) & 0x3FFu], 1u);
        }
    __syncthreads();
    r = find_bin<kBins23>(hist, warp_tot, sel, r.rank, nt);
    prefix |= r.bin << 10;
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const uint32_t key = key_of(v, e);
            if ((key & 0xFFFFFC00u) == prefix) atomicAdd(&hist[key & 0x3FFu], 1u);
        }
    __syncthreads();
    r = find_bin<kBins23>(hist, warp_tot, sel, r.rank, nt);
    *T = prefix | r.bin;
    *q = r.rank;
    *n_eq = r.count;
}

// Prune flags of the row for the threshold (T, q, n_eq): bit e of pruned[v] is set for
// every key < T and for the q lowest-column keys equal to T.
template <int V, class KeyOf>
__device__ __forceinline__ void prune_flags(KeyOf key_of, uint32_t T, uint32_t q, uint32_t n_eq, uint32_t* warp_tot, int nt,
                                            uint32_t (&pruned)[V]) {
    const uint32_t below = (q == n_eq) ? T + 1u : T;   // T < 2^31
#pragma unroll
    for (int v = 0; v < V; ++v) {
        pruned[v] = 0u;
#pragma unroll
        for (int e = 0; e < kVec; ++e) pruned[v] |= (key_of(v, e) < below) ? (1u << e) : 0u;
    }
    if (q != n_eq) {
        uint32_t before = 0u;   // ties in earlier vector slots (all threads)
#pragma unroll
        for (int v = 0; v < V; ++v) {
            uint32_t eq = 0u;
#pragma unroll
            for (int e = 0; e < kVec; ++e) eq |= (key_of(v, e) == T) ? (1u << e) : 0u;
            uint32_t total;
            uint32_t idx = before + block_excl_scan(__popc(eq), warp_tot, &total, nt);
#pragma unroll
            for (int e = 0; e < kVec; ++e)
                if (eq & (1u << e)) {
                    if (idx < q) pruned[v] |= (1u << e);
                    ++idx;
                }
            before += total;
        }
    }
}

// Write W' (pruned entries as +0, the others bit for bit; skipped when W_out is null) and the keep
// bitmask of one row.
template <int DT, int V>
__device__ __forceinline__ void store_row(Raw8<DT> (&raw)[V], const uint32_t (&pruned)[V], void* W_out, int64_t row_off,
                                          int cols, int nvec, int nt, uint8_t* mask_bytes, int64_t mask_off,
                                          int mask_row_bytes) {
    const int tid = threadIdx.x;
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vec = v * nt + tid;
        const int c0 = vec * kVec;
        if (vec < nvec && W_out != nullptr) {
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
            mask_bytes[mask_off + vec] = (uint8_t)keep;
        }
    }
}

}  // namespace mosaic
