// Per-row selection kernel of mosaic_prune_unstructured[_batch] for bf16 rows of 2048..16384
// columns (Section 4.1.3, unstructured projection pruning; weight metric of Eq. 5): per output
// row, the k entries first under (score ascending, column ascending) become +0, fused with the
// keep bitmask.
//
// One persistent CTA per SM.  A CTA takes a contiguous range of the launch's rows, so it changes
// matrix (job) only a few times; per job it keeps two tables in shared memory: the norms and, for
// a window [lo, hi) of score keys that should contain every row's threshold, per column the bf16
// magnitude pattern A_lo[j] such that a weight scores under lo iff its magnitude is below it, and
// the depth D[j] = A_hi[j] - A_lo[j] to the pattern from which a weight scores at least hi (the
// score norm_j * |w| is monotone in |w|).  Both patterns are exact: they are found by bisection on
// the very product that defines a score, so the candidates of a row are exactly its weights
// inside the window.  The window is centred on the median of one estimate per warp -
// the matching quantile of the exact scores of a quarter of one row of the job (rows spread
// evenly over the matrix), selected in registers - and made just wide enough, judged by the same
// samples, to hold the ranks a row's threshold can scatter over.
//
// A row is worked on by a group of G warps (G = 1 for short rows: a warp per row and no barrier at
// all on the row path; longer rows take 2, 4 or 8 warps so that 16 warps stay resident).  Every
// warp owns a fixed set of the row's 16-byte vectors from the copy into shared memory to the final
// store; the warps of a group only meet on the row's histogram:
//   1. the warp's vectors arrive in the group's row buffer by cp.async;
//   2. classification, two weights per integer subtract: (w | 0x8000) - A has bit 15 set iff the
//      magnitude is >= A.  Weights under A_lo are pruned for sure, weights from A_lo + D up are
//      kept for sure, the few per cent in between are the row's candidates; the keep bits of the
//      sure ones (candidates counted as kept) go to the row's keep bytes;
//   3. the warp queues its candidates (their columns), forms their exact fp32 score keys from the
//      row buffer and the norm table, adds them to the group's histogram of the window (up to 256
//      bins) and notes each one's bin beside its column;
//   4. (group barrier) every warp finds the bin that holds rank k and walks its queue once more:
//      a candidate of a lower bin loses its keep bit, the keys of the bin itself are collected
//      (group barrier) and ranked under (key, column), which is the oracle's total order, so ties
//      need no special case; those at or below the rank lose their keep bits too;
//   5. the store pass writes each vector under its keep byte; the row buffer is never modified.
// A row whose threshold falls outside the window, whose candidates overflow a queue, or whose bin
// holds more than 32 keys, and every row of a job whose window is unusable (norms that are not
// finite and >= 0, a threshold at zero or at overflow) takes slow_row(): a radix select by the
// group on exact (key, column) pairs.  All paths give the oracle's bits.
#include "prune_jobs.cuh"

namespace mosaic {

constexpr int kWMaxWarps = 16;
constexpr int kWBins = 256;
constexpr int kWBinList = 32;
constexpr uint32_t kWOverflow = 0xFFFFFFFFu;   // a warp's "my queue overflowed" in place of its count of sure-below weights

// Shared-memory carve-up for rows of `cols` columns worked on by groups of G warps (host and
// device agree on it).  Groups of several warps alternate between two histograms / bin lists /
// count slots from row to row, so that a warp may start the next row while another still reads.
struct WarpLayout {
    int nvec, nwords, qcap;   // qcap: candidates one warp may queue
    uint32_t off_alo, off_dep, off_nrm, off_misc, off_group0, per_group;             // bytes
    uint32_t o_queue, per_queue, o_qcol, o_qbin, per_qbin, o_hist, o_mbytes, o_bkey, o_bcol, o_ctl;   // bytes inside a group's block
};
__host__ __device__ inline WarpLayout warp_layout(int cols, int G) {
    WarpLayout L;
    const uint32_t sets = G == 1 ? 1u : 2u;
    L.nvec = cols >> 3;
    L.nwords = (cols + 31) >> 5;
    L.qcap = (((cols >> 3) + G - 1) / G + 31) & ~31;             // 1/8 of the warp's share of the row
    uint32_t o = 0;
    L.off_alo = o;   o += (uint32_t)L.nvec * 16u;
    L.off_dep = o;   o += (uint32_t)L.nvec * 16u;
    L.off_nrm = o;   o += (uint32_t)cols * 4u;
    L.off_misc = o;  o += 256u;
    L.off_group0 = o;
    uint32_t w = (uint32_t)L.nvec * 16u;               // the row
    L.o_queue = w;                                     // per warp: the columns of its candidates (2 B each)
    L.o_qcol = 0u;
    L.per_queue = (uint32_t)L.qcap * 2u;
    w += L.per_queue * (uint32_t)G;
    L.o_qbin = w;                                      // per warp: the window bin of each queued candidate (1 B each)
    L.per_qbin = (uint32_t)L.qcap;
    w += L.per_qbin * (uint32_t)G;
    w = (w + 15u) & ~15u;
    L.o_hist = w;    w += sets * kWBins * 4u;
    L.o_mbytes = w;  w += ((uint32_t)L.nwords * 4u + 15u) & ~15u;
    L.o_bkey = w;    w += sets * kWBinList * 4u;
    L.o_bcol = w;    w += sets * kWBinList * 4u;
    L.o_ctl = w;     w += G == 1 ? 16u : 256u;         // [p*16 + sub] sure-below counts, [32 + p] bin-list fill
    L.per_group = (w + 15u) & ~15u;
    return L;
}
constexpr uint32_t kWSmemBudget = 227u * 1024u - 256u;   // dynamic shared memory a CTA may use (static arrays need a little)

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem)), "l"(gmem)
                 : "memory");
}
// Barrier among the 32*G threads of a row group (G == 1: the warp).  Barrier 0 is the CTA's.
template <int G>
__device__ __forceinline__ void group_barrier(int gid) {
    if (G == 1) __syncwarp();
    else asm volatile("bar.sync %0, %1;" ::"r"(gid + 1), "r"(32 * G) : "memory");
}

// With x = word | 0x80008000 (each 16-bit lane = 0x8000 + magnitude) and A two 16-bit thresholds
// <= 0x8000, the lanes of t = x - A never borrow from each other and bit 15 / bit 31 of t is set
// iff magnitude >= threshold.  flags8 gathers those bits of a vector's four words into one word:
// element e < 4 lands on bit 8e+7, element e >= 4 on bit 8(e-4)+6.
__device__ __forceinline__ uint32_t flags8(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3) {
    const uint32_t a = __byte_perm(t0, t1, 0x7531);   // bytes: elements 0, 1, 2, 3 (flag = top bit)
    const uint32_t b = __byte_perm(t2, t3, 0x7531);   // elements 4, 5, 6, 7
    return (a & 0x80808080u) | ((b >> 1) & 0x40404040u);
}
// flags8 word -> byte with bit e = flag of element e.  (f & 0x80808080) holds elements 0..3 on bits
// 7, 15, 23, 31; the high word of its product with 2^25 + 2^18 + 2^11 + 2^4 has them on bits 0..3
// (no two partial products meet on a bit, so nothing carries).
__device__ __forceinline__ uint32_t byte_of_flags(uint32_t f) {
    const uint32_t lo = __umulhi(f & 0x80808080u, 0x02040810u) & 0xFu;
    const uint32_t hi = __umulhi((f << 1) & 0x80808080u, 0x02040810u) & 0xFu;
    return lo | (hi << 4);
}
// 0xFFFF over each 16-bit lane of t whose top bit is set (prmt replicates the sign of the selected byte).
__device__ __forceinline__ uint32_t lane_mask(uint32_t t) {
    uint32_t m;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(m) : "r"(t), "r"(0u), "r"(0xBB99u));
    return m;
}
__device__ __forceinline__ float mag_f32(uint32_t word, int half) {   // |element| widened exactly to fp32
    return __uint_as_float(half ? (word & 0x7FFF0000u) : ((word << 16) & 0x7FFFFFFFu));
}
__device__ __forceinline__ uint32_t word_of(const uint4& r, int i) { return i == 0 ? r.x : (i == 1 ? r.y : (i == 2 ? r.z : r.w)); }

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += n;
    }
    return v;
}

// The bin of hist[0..256) that holds rank `rank` (1-based) when `base0` entries come before bin 0.
// Warp-wide; CLEAR leaves the histogram zeroed.  Returns false if no bin holds the rank.
template <bool CLEAR>
__device__ __forceinline__ bool warp_find_bin(uint32_t* hist, uint32_t base0, uint32_t rank, int lane, uint32_t* bin,
                                              uint32_t* rank_in_bin, uint32_t* count) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
    const uint4 a = h4[lane * 2], b = h4[lane * 2 + 1];
    if (CLEAR) {
        h4[lane * 2] = make_uint4(0u, 0u, 0u, 0u);
        h4[lane * 2 + 1] = make_uint4(0u, 0u, 0u, 0u);
    }
    const uint32_t c[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t sum = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += c[i];
    const uint32_t incl = warp_incl_scan(sum, lane);
    uint32_t base = base0 + incl - sum;
    const unsigned m = __ballot_sync(0xFFFFFFFFu, base < rank && rank <= base + sum);
    if (m == 0u) return false;
    uint32_t bb = 0u, rr = 0u, cc = 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (cc == 0u && base < rank && rank <= base + c[i]) {
            bb = (uint32_t)(lane * 8 + i);
            rr = rank - base;
            cc = c[i];
        }
        base += c[i];
    }
    const int src = __ffs(m) - 1;
    *bin = __shfl_sync(0xFFFFFFFFu, bb, src);
    *rank_in_bin = __shfl_sync(0xFFFFFFFFu, rr, src);
    *count = __shfl_sync(0xFFFFFFFFu, cc, src);
    return true;
}
__device__ __forceinline__ void warp_clear_hist(uint32_t* hist, int lane) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
    h4[lane * 2] = make_uint4(0u, 0u, 0u, 0u);
    h4[lane * 2 + 1] = make_uint4(0u, 0u, 0u, 0u);
}

// Exact score key of element e of a vector (sign bit cleared: norms are >= +0 by contract, and a
// negative one must not index past a histogram).
__device__ __forceinline__ uint32_t exact_key(const uint4& r, const float* nrm8, int e) {
    return __float_as_uint(__fmul_rn(nrm8[e], mag_f32(word_of(r, e >> 1), e & 1))) & 0x7FFFFFFFu;
}

// The always-exact treatment of one row by its group: radix select (8-bit digits from the top) of
// the k-th smallest key T, then - if only q of the n_eq keys equal to T are among the k smallest -
// of the q-th smallest column among those; every entry at or below (T, column) is pruned.  Stores
// the warp's vectors and leaves their keep bits as bytes in mbytes.  `hist` may hold a failed
// attempt's counts on entry and is zero on exit.  Called by all warps of the group together.
template <int V, int G>
__device__ __noinline__ void slow_row(const uint4* row, const float* nrm, int nvec, uint32_t k, uint32_t* hist, uint8_t* mbytes,
                                      uint16_t* out_row, int gid, int sub) {
    const int lane = threadIdx.x & 31;
    const int gl = sub * 32 + lane;
    group_barrier<G>(gid);
    if (sub == 0) warp_clear_hist(hist, lane);
    group_barrier<G>(gid);
    uint32_t T = 0u, q = 0u, n_eq = 0u, colT = 0xFFFFu;
    // phase 0: the key, four digits; phase 1: the column among the keys equal to T, two digits
    for (int phase = 0; phase < 2; ++phase) {
        uint32_t prefix = 0u, pmask = 0u, rank = phase == 0 ? k : q, cnt = 0u;
        for (int shift = phase == 0 ? 24 : 8; shift >= 0; shift -= 8) {
#pragma unroll 2
            for (int v = 0; v < V; ++v) {
                const int vec = v * 32 * G + gl;
                if (vec < nvec) {
                    const uint4 r = row[vec];
                    const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                    const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint32_t key = exact_key(r, n8, e);
                        if (phase == 0) {
                            if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFFu], 1u);
                        } else {
                            const uint32_t col = (uint32_t)(vec * 8 + e);
                            if (key == T && (col & pmask) == prefix) atomicAdd(&hist[(col >> shift) & 0xFFu], 1u);
                        }
                    }
                }
            }
            group_barrier<G>(gid);
            uint32_t bin = 0u, rr = 0u, cc = 0u;
            warp_find_bin<false>(hist, 0u, rank, lane, &bin, &rr, &cc);   // always found: 1 <= rank <= matching entries
            group_barrier<G>(gid);
            if (sub == 0) warp_clear_hist(hist, lane);
            group_barrier<G>(gid);
            prefix |= bin << shift;
            pmask |= 0xFFu << shift;
            rank = rr;
            cnt = cc;
        }
        if (phase == 0) {
            T = prefix;
            q = rank;
            n_eq = cnt;
            if (q == n_eq) break;   // every key equal to T is pruned: colT stays above all columns
        } else {
            colT = prefix;
        }
    }
#pragma unroll 2
    for (int v = 0; v < V; ++v) {
        const int vec = v * 32 * G + gl;
        if (vec < nvec) {
            const uint4 r = row[vec];
            const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
            const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
            uint32_t pruned = 0u;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t key = exact_key(r, n8, e);
                if (key < T || (key == T && (uint32_t)(vec * 8 + e) <= colT)) pruned |= 1u << e;
            }
            uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (pruned & (1u << (2 * i))) w[i] &= 0xFFFF0000u;
                if (pruned & (2u << (2 * i))) w[i] &= 0x0000FFFFu;
            }
            if (out_row != nullptr) st_stream16(out_row + (int64_t)vec * kVec, make_uint4(w[0], w[1], w[2], w[3]));
            mbytes[vec] = (uint8_t)(~pruned & 0xFFu);
        }
    }
}

// Smallest bf16 magnitude pattern a in [0, 0x7F80] whose score key with norm n is >= key_t
// (1 <= key_t <= 0x7F800000; n >= 0 and finite).  The key of pattern a is the bit pattern of the one
// fp32 product that defines the score, which is monotone in a, so bisection finds the exact
// boundary:  magnitude < result  <=>  score key < key_t.  It starts from the bracket [g-2, g+2]
// around the pattern of t / n, which holds the boundary except in odd corners (subnormal or
// overflowing quotients), where the whole range is searched.  n = 0: every finite weight scores 0,
// the result is 0x7F80 (inf and NaN weights score NaN, the largest key).
__device__ __forceinline__ uint32_t pattern_at_key(float n, uint32_t key_t) {
    auto at_or_above = [&](uint32_t a) -> bool {
        return (__float_as_uint(__fmul_rn(n, __uint_as_float(a << 16))) & 0x7FFFFFFFu) >= key_t;
    };
    uint32_t lo = 0u, hi = 0x7F80u;   // at_or_above(0) is false (key 0 < key_t); at_or_above(0x7F80) is true (inf or NaN)
    const uint32_t g = __float_as_uint(__fdiv_rn(__uint_as_float(key_t), n)) >> 16;
    if (g >= 2u && g + 2u <= 0x7F80u && !at_or_above(g - 2u) && at_or_above(g + 2u)) {
        lo = g - 2u;
        hi = g + 2u;
    }
    while (hi - lo > 1u) {
        const uint32_t mid = (lo + hi) >> 1;
        if (at_or_above(mid)) hi = mid;
        else lo = mid;
    }
    return hi;
}

// A_lo of one vector of 8 columns for the window [lo, hi) of keys (packed like the row's words);
// returns the largest A_hi - A_lo of the vector.
__device__ __forceinline__ void thresholds_of_vector(const float* nrm8, uint32_t lo, uint32_t hi, uint4* alo, uint4* dep) {
    uint32_t al[8], d[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        al[e] = pattern_at_key(nrm8[e], lo);
        d[e] = pattern_at_key(nrm8[e], hi) - al[e];   // hi > lo: never negative
    }
    *alo = make_uint4(al[0] | (al[1] << 16), al[2] | (al[3] << 16), al[4] | (al[5] << 16), al[6] | (al[7] << 16));
    *dep = make_uint4(d[0] | (d[1] << 16), d[2] | (d[3] << 16), d[4] | (d[5] << 16), d[6] | (d[7] << 16));
}

// blockDim.x = 32 * G * groups; dynamic shared memory = off_group0 + groups * per_group of warp_layout(cols, G).
// Every job: cols % 8 == 0, cols <= V * 256 * G, 0 < k < cols.  FULL: cols == V * 256 * G, so every
// vector slot is inside the row and no bounds test is needed.
template <int V, int G, int NJ, bool FULL>
__global__ void __launch_bounds__(kWMaxWarps * 32, 1) prune_rows_warp_kernel(const __grid_constant__ PruneJobList<NJ> jobs,
                                                                             int64_t total_rows, int cols) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint16_t flagtab[32];   // bit of a packed candidate word -> (vector within its group of 4) * 256 * G + element
    constexpr int TG = 32 * G;         // threads of a row group
    constexpr int NW = (V + 3) / 4;    // packed candidate words per thread
    const WarpLayout L = warp_layout(cols, G);
    const int nvec = L.nvec, nwords = L.nwords;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = blockDim.x >> 5, nthreads = blockDim.x;
    const int gid = wid / G, sub = wid % G, ngroups = nwarps / G;
    const int gl = sub * 32 + lane;    // thread within the row group: owns the vectors v * TG + gl
    uint4* alo = reinterpret_cast<uint4*>(smem + L.off_alo);
    uint4* dep = reinterpret_cast<uint4*>(smem + L.off_dep);
    float* nrm = reinterpret_cast<float*>(smem + L.off_nrm);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + L.off_misc);   // [0..15] the warps' threshold estimates,
                                                                       // [17] samples taken, [32..63] samples by distance from the centre
    unsigned char* mine = smem + L.off_group0 + (size_t)gid * L.per_group;
    uint4* row = reinterpret_cast<uint4*>(mine);
    const uint16_t* row16 = reinterpret_cast<const uint16_t*>(mine);
    uint16_t* qcol = reinterpret_cast<uint16_t*>(mine + L.o_queue + (size_t)sub * L.per_queue);
    uint8_t* qbin = mine + L.o_qbin + (size_t)sub * L.per_qbin;
    uint32_t* hist0 = reinterpret_cast<uint32_t*>(mine + L.o_hist);
    uint8_t* mbytes = mine + L.o_mbytes;
    uint32_t* mwords = reinterpret_cast<uint32_t*>(mine + L.o_mbytes);
    uint32_t* bkey0 = reinterpret_cast<uint32_t*>(mine + L.o_bkey);
    uint32_t* bcol0 = reinterpret_cast<uint32_t*>(mine + L.o_bcol);
    uint32_t* ctl = reinterpret_cast<uint32_t*>(mine + L.o_ctl);

    if (tid < 32) {
        const int p = tid & 7, s = (7 - p) >> 1;
        const int e = (tid >> 3) + ((p & 1) ? 0 : 4);
        flagtab[tid] = (uint16_t)(s * 8 * TG + e);
    }
    if (sub == 0) {
        for (int b = lane; b < (G == 1 ? 1 : 2) * kWBins; b += 32) hist0[b] = 0u;
        for (int b = lane; b < nwords * 4; b += 32) mbytes[b] = 0u;   // the bytes past the row's last vector stay zero: mask padding
        for (int b = lane; b < (G == 1 ? 4 : 64); b += 32) ctl[b] = 0u;
    }
    __syncthreads();

    const int64_t rows_per_cta = (total_rows + gridDim.x - 1) / gridDim.x;
    const int64_t cta_begin = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t cta_end = cta_begin + rows_per_cta < total_rows ? cta_begin + rows_per_cta : total_rows;
    int j = 0;
    uint32_t parity = 0u;   // which histogram / bin list / count slots the group's current row uses (G > 1)
    for (int64_t seg = cta_begin; seg < cta_end;) {
        while (seg >= jobs.job[j].row0 + jobs.job[j].rows) ++j;
        const PruneJob& J = jobs.job[j];
        const int64_t job_end = J.row0 + J.rows;
        const int64_t seg_end = cta_end < job_end ? cta_end : job_end;
        const uint32_t uk = (uint32_t)J.k;
        const int64_t ldw = J.ldw;

        // ---------------- job set-up: norms, window, thresholds
        __syncthreads();   // every warp is done with the previous job's tables
        bool fin = true;
        for (int c = tid; c < cols; c += nthreads) {
            const float n = __ldg(J.norms + c);
            nrm[c] = n;
            fin = fin && n >= 0.0f && n <= 3.402823466e38f;   // false for NaN, inf and negative norms
        }
        if (tid < 64) misc[tid] = 0u;
        bool valid = __syncthreads_and(fin ? 1 : 0) != 0;
        uint32_t lo = 0u, width = 0u;
        int shift = 0;
        if (valid) {
            // One estimate per warp: the k-th score of row (rows-1)*wid/(nwarps-1), taken as the matching
            // quantile of the exact keys of a quarter of the row (four evenly spaced vectors per lane),
            // which the lane keeps in registers through a 4 x 8-bit radix select.
            const int64_t srow = (J.rows - 1) * wid / (nwarps > 1 ? nwarps - 1 : 1);
            const uint16_t* src = J.W_in + srow * ldw;
            uint32_t key[32];
            uint32_t n_valid = 0u;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int vec = (i * (V * G / 4)) * 32 + lane;
                if (FULL || vec < nvec) {
                    // (in place, another CTA may be writing this row: any value will do for an estimate)
                    const uint4 r = ld_stream16(src + (int64_t)vec * kVec);
                    const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                    const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e) key[i * 8 + e] = exact_key(r, n8, e);
                    n_valid += 8u;
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) key[i * 8 + e] = 0xFFFFFFFFu;   // in no histogram
                }
            }
            n_valid = __reduce_add_sync(0xFFFFFFFFu, n_valid);
            {
                uint32_t rank = (uint32_t)(((uint64_t)uk * n_valid + (uint32_t)cols / 2u) / (uint32_t)cols);
                rank = rank < 1u ? 1u : (rank > n_valid ? n_valid : rank);
                uint32_t prefix = 0u, pmask = 0u;
                for (int turn = 0; turn < G; ++turn) {   // the warps of a group share a histogram: one after the other
                    if (turn == sub) {
#pragma unroll 1
                        for (int sh = 24; sh >= 0; sh -= 8) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if ((key[i] & pmask) == prefix && key[i] != 0xFFFFFFFFu) atomicAdd(&hist0[(key[i] >> sh) & 0xFFu], 1u);
                            __syncwarp();
                            uint32_t bin = 0u, rr = 0u, cc = 0u;
                            warp_find_bin<true>(hist0, 0u, rank, lane, &bin, &rr, &cc);
                            prefix |= bin << sh;
                            pmask |= 0xFFu << sh;
                            rank = rr;
                            __syncwarp();
                        }
                    }
                    if (G > 1) group_barrier<G>(gid);
                }
                if (lane == 0) {
                    misc[wid] = prefix;
                    atomicAdd(&misc[17], n_valid);
                }
            }
            __syncthreads();
            // median of the estimates (every thread ranks them the same way: by value, then by warp)
            uint32_t center = 0u;
            for (int a = 0; a < nwarps; ++a) {
                const uint32_t va = misc[a];
                int less = 0;
                for (int b = 0; b < nwarps; ++b) {
                    const uint32_t vb = misc[b];
                    less += (vb < va || (vb == va && b < a)) ? 1 : 0;
                }
                if (less == nwarps / 2) center = va;
            }
            // How wide must the window be?  A row's threshold scatters over about +-3.25 sigma ranks around the
            // typical one, sigma^2 = k (1 - k/cols), and the centre itself is only an estimate (allow cols/64
            // ranks).  The samples tell how many keys lie how far from the centre: misc[32 + b] counts those
            // whose distance has bit length b, i.e. lies in [2^(b-1), 2^b).
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (key[i] != 0xFFFFFFFFu) {
                    const uint32_t dist = key[i] > center ? key[i] - center : center - key[i];
                    atomicAdd(&misc[32 + (32 - __clz(dist))], 1u);   // dist < 2^31: bit length 0..31
                }
            __syncthreads();
            {
                const double p = (double)uk / (double)cols;
                const double want_row = 6.5 * sqrt((double)cols * p * (1.0 - p)) + (double)cols / 64.0 + 16.0;
                const uint32_t n_samples = misc[17];
                const double want = want_row * (double)n_samples / (double)cols;   // ... among the samples
                // smallest half-width h with  #{distance < h} >= want, interpolated inside the bit-length class
                double below = 0.0, half_w = 0.0;
                bool found = false;
                for (int b = 0; b < 32 && !found; ++b) {
                    const double c = (double)misc[32 + b];
                    if (below + c >= want) {
                        const double base = b == 0 ? 0.0 : ldexp(1.0, b - 1), span = b == 0 ? 1.0 : ldexp(1.0, b - 1);
                        half_w = base + span * (c > 0.0 ? (want - below) / c : 1.0);
                        found = true;
                    }
                    below += c;
                }
                if (!found) half_w = 2147483648.0;
                double w_d = 2.0 * half_w;
                if (w_d < 4096.0) w_d = 4096.0;
                valid = w_d <= 8388608.0;   // a window of more than an octave of keys is no window
                if (valid) {
                    uint32_t w_u = (uint32_t)w_d;
                    shift = 32 - __clz(w_u) - 8;                                  // at most 256 bins of 2^shift keys
                    shift = shift < 0 ? 0 : shift;
                    const uint32_t nb = (w_u + (1u << shift) - 1u) >> shift;     // 128 < nb <= 256
                    width = nb << shift;
                    const uint32_t half = width >> 1;
                    // the window must start above key 0 (a zero weight has to be below it) and end at or below +inf
                    valid = center > half && center - half <= 0x7F800000u - width;
                    lo = center - half;
                }
            }
            if (valid) {
                // A_lo + D = A_hi <= 0x7F80 for every column, which the borrow-free subtraction needs
                for (int vec = tid; vec < nvec; vec += nthreads) {
                    const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                    const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
                    thresholds_of_vector(n8, lo, lo + width, &alo[vec], &dep[vec]);
                }
            }
        }
        __syncthreads();

        // ---------------- rows of the segment, one per group at a time
        auto fetch = [&](int64_t rr) {   // this warp's vectors of global row rr into the group's buffer (one cp.async group)
            const uint16_t* src = J.W_in + (rr - J.row0) * ldw;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int vec = v * TG + gl;
                if (FULL || vec < nvec) cp_async16(&row[vec], src + (int64_t)vec * kVec);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        if (seg + gid < seg_end) fetch(seg + gid);
        for (int64_t r = seg + gid; r < seg_end; r += ngroups, parity ^= (G == 1 ? 0u : 1u)) {
            const int64_t lrow = r - J.row0;
            uint16_t* out_row = J.W_out != nullptr ? J.W_out + lrow * ldw : nullptr;
            uint32_t* mask_row = J.mask != nullptr ? reinterpret_cast<uint32_t*>(J.mask + lrow * J.mask_row_bytes) : nullptr;
            uint32_t* hist = hist0 + parity * kWBins;
            uint32_t* bkey = bkey0 + parity * kWBinList;
            uint32_t* bcol = bcol0 + parity * kWBinList;
            uint32_t* below_of = ctl + parity * 16u;   // [sub]   (G > 1)
            uint32_t* fill = ctl + 32u + parity;       //         (G > 1)
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();   // a warp reads only the vectors it copied itself

            bool done = false;
            if (valid) {
                // ---- classification
                uint32_t candw[NW];
#pragma unroll
                for (int w = 0; w < NW; ++w) candw[w] = 0u;
                uint32_t below = 0u;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int vec = v * TG + gl;
                    if (FULL || vec < nvec) {
                        const uint4 rr = row[vec], a = alo[vec], d = dep[vec];
                        const uint32_t t0 = (rr.x | 0x80008000u) - a.x, t1 = (rr.y | 0x80008000u) - a.y,
                                       t2 = (rr.z | 0x80008000u) - a.z, t3 = (rr.w | 0x80008000u) - a.w;
                        const uint32_t keepf = flags8(t0, t1, t2, t3);
                        const uint32_t above = flags8(t0 - d.x, t1 - d.y, t2 - d.z, t3 - d.w);
                        candw[v >> 2] |= (keepf & ~above) >> (2 * (v & 3));
                        below += 8u - (uint32_t)__popc(keepf);
                        mbytes[vec] = (uint8_t)byte_of_flags(keepf);   // candidates count as kept until the threshold says otherwise
                    }
                }
                // ---- queue the warp's candidates (their columns)
                uint32_t cnt = 0u;
#pragma unroll
                for (int w = 0; w < NW; ++w) cnt += (uint32_t)__popc(candw[w]);
                const uint32_t incl = warp_incl_scan(cnt, lane);
                const uint32_t qn = __shfl_sync(0xFFFFFFFFu, incl, 31);
                const bool fits = qn <= (uint32_t)L.qcap;
                if (fits) {
                    uint32_t off = incl - cnt;
#pragma unroll
                    for (int w = 0; w < NW; ++w) {
                        const uint32_t col0 = (uint32_t)(w * 32 * TG + gl * 8);
                        for (uint32_t c = candw[w]; c != 0u;) {   // two per turn: both table reads in flight together
                            const int p0 = __ffs(c) - 1;
                            c &= c - 1u;
                            const bool two = c != 0u;
                            const int p1 = two ? __ffs(c) - 1 : p0;
                            c &= c - 1u;
                            const uint32_t f0 = flagtab[p0], f1 = flagtab[p1];
                            qcol[off] = (uint16_t)(col0 + f0);
                            if (two) qcol[off + 1u] = (uint16_t)(col0 + f1);
                            off += two ? 2u : 1u;
                        }
                    }
                    __syncwarp();
                    // ---- exact keys of the candidates, four rounds of 32 at a time
                    for (uint32_t base = lane; base < qn; base += 128u) {
                        uint32_t col[4], a[4];
                        float n[4];
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t i = base + 32u * g;
                            col[g] = i < qn ? (uint32_t)qcol[i] : (uint32_t)(gl * 8);   // a spare slot reads a column of its own
                        }
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            a[g] = ((uint32_t)row16[col[g]] & 0x7FFFu) << 16;
                            n[g] = nrm[col[g]];
                        }
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t i = base + 32u * g;
                            if (i < qn) {
                                const uint32_t key = __float_as_uint(__fmul_rn(n[g], __uint_as_float(a[g])));
                                const uint32_t d = key - lo;   // key < lo wraps to >= 2^31 (key, lo < 2^31)
                                if (d < width) atomicAdd(&hist[d >> shift], 1u);
                                else below += d >> 31;
                                const uint32_t b = d >> shift;   // bin of the window; 255 also stands for everything above it
                                qbin[i] = (uint8_t)((d >> 31) ? 0u : (b < 255u ? b : 255u));
                            }
                        }
                    }
                }
                below = __reduce_add_sync(0xFFFFFFFFu, below);
                bool ok = fits;
                if (G > 1) {   // the group's count of sure-below weights, and whether every warp's queue held
                    if (lane == 0) below_of[sub] = fits ? below : kWOverflow;
                    group_barrier<G>(gid);
                    below = 0u;
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const uint32_t b = below_of[g];
                        ok = ok && b != kWOverflow;
                        below += b;
                    }
                } else {
                    __syncwarp();
                }
                // ---- the bin that holds rank k, then the rank inside it under (key, column)
                uint32_t bin = 0u, r_bin = 0u, n_bin = 0u;
                if (ok) ok = warp_find_bin<G == 1>(hist, below, uk, lane, &bin, &r_bin, &n_bin) && n_bin <= (uint32_t)kWBinList;
                if (ok) {
                    // The queue again, by bin code: a candidate of a lower bin is pruned (its keep bit
                    // cleared); one whose code matches the bin goes on the bin list after its exact
                    // key confirms it (code 255 also covers keys above the window).
                    auto prune_col = [&](uint32_t col) { atomicAnd(&mwords[col >> 5], ~(1u << (col & 31u))); };
                    uint32_t nl = 0u;
                    for (uint32_t base = 0u; base < qn; base += 128u) {   // four rounds of 32 per turn
                        uint32_t code[4], col[4];
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t i = base + 32u * g + lane;
                            code[g] = i < qn ? (uint32_t)qbin[i] : 0xFFFFu;
                            col[g] = i < qn ? (uint32_t)qcol[i] : 0u;
                        }
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            if (code[g] < bin) prune_col(col[g]);
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            bool in = false;
                            uint32_t key = 0u;
                            if (code[g] == bin) {
                                key = __float_as_uint(__fmul_rn(nrm[col[g]], __uint_as_float(((uint32_t)row16[col[g]] & 0x7FFFu) << 16)));
                                const uint32_t d = key - lo;
                                if (d >> 31) prune_col(col[g]);   // below the window (cannot happen with exact thresholds)
                                else in = d < width && (d >> shift) == bin;
                            }
                            const unsigned m = __ballot_sync(0xFFFFFFFFu, in);
                            if (m == 0u) continue;
                            if (G > 1) {   // the group's list is filled by all its warps: take a range of it
                                uint32_t first = 0u;
                                if (lane == 0) first = atomicAdd(fill, (uint32_t)__popc(m));
                                nl = __shfl_sync(0xFFFFFFFFu, first, 0);
                            }
                            if (in) {
                                const uint32_t pos = nl + (uint32_t)__popc(m & ((1u << lane) - 1u));
                                bkey[pos] = key;
                                bcol[pos] = col[g];
                            }
                            if (G == 1) nl += (uint32_t)__popc(m);
                        }
                    }
                    group_barrier<G>(gid);
                    const bool have = (uint32_t)lane < n_bin;
                    const uint32_t mk = have ? bkey[lane] : 0xFFFFFFFFu, mc = have ? bcol[lane] : 0xFFFFFFFFu;
                    uint32_t less = 0u;
                    for (uint32_t jj = 0u; jj < n_bin; ++jj) {
                        const uint32_t ok2 = __shfl_sync(0xFFFFFFFFu, mk, (int)jj), oc = __shfl_sync(0xFFFFFFFFu, mc, (int)jj);
                        less += (ok2 < mk || (ok2 == mk && oc < mc)) ? 1u : 0u;
                    }
                    if (G > 1 && sub == 0) {   // every warp has read this row's histogram: clean for the row after next
                        warp_clear_hist(hist, lane);
                        if (lane == 0) *fill = 0u;
                    }
                    // ---- the entries of the bin at or below rank r_bin are pruned (a warp clears the bits of its own columns only:
                    //      the other warps of the group may already be at their next row)
                    if (have && less < r_bin && (G == 1 || (int)((mc >> 3) % (uint32_t)TG) / 32 == sub)) prune_col(mc);
                    __syncwarp();
                    // ---- store: each weight under its keep bit
                    if (out_row != nullptr) {
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            const int vec = v * TG + gl;
                            if (FULL || vec < nvec) {
                                const uint4 rr = row[vec];
                                const uint32_t kb = (uint32_t)mbytes[vec];
                                // kb * (2^(15-2i) + 2^(30-2i)) has bit 2i of kb on bit 15 and bit 2i+1 on bit 31
                                st_stream16(out_row + (int64_t)vec * kVec,
                                            make_uint4(rr.x & lane_mask(kb * 0x40008000u), rr.y & lane_mask(kb * 0x10002000u),
                                                       rr.z & lane_mask(kb * 0x04000800u), rr.w & lane_mask(kb * 0x01000200u)));
                            }
                        }
                    }
                    done = true;
                }
            }
            if (!done) slow_row<V, G>(row, nrm, nvec, uk, hist, mbytes, out_row, gid, sub);
            __syncwarp();   // the warp's part of the row buffer is free, its keep bytes are complete
            if (r + ngroups < seg_end) fetch(r + ngroups);   // the next row travels while the keep words leave
            if (mask_row != nullptr) {
                // the warp's vectors v*TG + sub*32 .. +31 are 32 keep bytes = 8 keep words per v
                for (int idx = lane; idx < V * 8; idx += 32) {
                    const int w = ((idx >> 3) * TG + sub * 32) / 4 + (idx & 7);
                    if (w < nwords) mask_row[w] = reinterpret_cast<const uint32_t*>(mbytes)[w];
                }
            }
            __syncwarp();
        }
        seg = seg_end;
    }
}

// Group size, group count and vectors per thread for rows of `cols` columns: the most resident
// warps shared memory allows (at most kWMaxWarps), the smaller group on a tie.
struct WarpShape {
    int G, groups, V;
};
static WarpShape shape_for(int cols) {
    WarpShape best{0, 0, 0};
    const int nvec = cols / 8;
    for (int G = 1; G <= 8; G *= 2) {
        const int v = (nvec + 32 * G - 1) / (32 * G);
        const int V = v <= 8 ? 8 : (v <= 10 ? 10 : (v <= 12 ? 12 : (v <= 14 ? 14 : (v <= 16 ? 16 : (v <= 20 ? 20 : 0)))));
        if (V == 0) continue;
        const WarpLayout L = warp_layout(cols, G);
        if (L.off_group0 + L.per_group > kWSmemBudget) continue;
        int groups = (int)((kWSmemBudget - L.off_group0) / L.per_group);
        if (groups > kWMaxWarps / G) groups = kWMaxWarps / G;
        if (groups * G < 3) continue;
        if (groups * G > best.groups * best.G) best = WarpShape{G, groups, V};
    }
    return best;
}

template <int V, int G, int NJ, bool FULL>
static int launch_warp_v(const PruneJobList<NJ>& jobs, int64_t total_rows, int cols, int groups, cudaStream_t st) {
    const WarpLayout L = warp_layout(cols, G);
    const size_t dyn = (size_t)L.off_group0 + (size_t)groups * L.per_group;
    static DeviceCache opted;   // the shared-memory opt-in belongs to one device's copy of the kernel
    const int ok = opted.get([&]() -> int {
        if (cudaFuncSetAttribute(prune_rows_warp_kernel<V, G, NJ, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kWSmemBudget) != cudaSuccess) {
            (void)cudaGetLastError();
            return -1;
        }
        return 1;
    });
    if (ok < 0) return MOSAIC_ERR_CUDA;
    int64_t grid = sm_count();
    const int64_t need = (total_rows + groups - 1) / groups;
    if (grid > need) grid = need;
    if (grid < 1) grid = 1;
    prune_rows_warp_kernel<V, G, NJ, FULL><<<(unsigned)grid, groups * G * 32, dyn, st>>>(jobs, total_rows, cols);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

template <int NJ>
static int launch_warp_any(const PruneJobList<NJ>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    const WarpShape s = shape_for(cols);
    if (s.G == 0) return MOSAIC_ERR_INVALID_ARG;
    const bool full = cols == s.V * 256 * s.G;
#define MOSAIC_WARP_CASE(VV, GG)                                                                  \
    if (s.V == VV && s.G == GG)                                                                   \
        return full ? launch_warp_v<VV, GG, NJ, true>(jobs, total_rows, cols, s.groups, st)       \
                    : launch_warp_v<VV, GG, NJ, false>(jobs, total_rows, cols, s.groups, st)
    MOSAIC_WARP_CASE(8, 1);
    MOSAIC_WARP_CASE(10, 1);
    MOSAIC_WARP_CASE(12, 1);
    MOSAIC_WARP_CASE(14, 1);
    MOSAIC_WARP_CASE(16, 1);
    MOSAIC_WARP_CASE(20, 1);
    MOSAIC_WARP_CASE(8, 2);
    MOSAIC_WARP_CASE(10, 2);
    MOSAIC_WARP_CASE(12, 2);
    MOSAIC_WARP_CASE(14, 2);
    MOSAIC_WARP_CASE(16, 2);
    MOSAIC_WARP_CASE(20, 2);
    MOSAIC_WARP_CASE(8, 4);
    MOSAIC_WARP_CASE(10, 4);
    MOSAIC_WARP_CASE(12, 4);
    MOSAIC_WARP_CASE(14, 4);
    MOSAIC_WARP_CASE(16, 4);
    MOSAIC_WARP_CASE(8, 8);
#undef MOSAIC_WARP_CASE
    return MOSAIC_ERR_INVALID_ARG;
}

bool prune_warp_takes(int64_t cols) {
    return cols >= kWarpMinCols && cols <= kWarpMaxCols && cols % 8 == 0 && shape_for((int)cols).G != 0;
}

int launch_prune_warp(const PruneJobList<1>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    return launch_warp_any<1>(jobs, total_rows, cols, st);
}
int launch_prune_warp(const PruneJobList<kBatchJobs>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    return launch_warp_any<kBatchJobs>(jobs, total_rows, cols, st);
}

}  // namespace mosaic
