// Warp-per-row kernel of mosaic_prune_unstructured[_batch] for bf16 rows of 2048..8192 columns
// (Section 4.1.3, unstructured projection pruning; weight metric of Eq. 5): per output row, the k
// entries first under (score ascending, column ascending) become +0, fused with the keep bitmask.
//
// One persistent CTA per SM.  A CTA takes a contiguous range of the launch's rows, so it changes
// matrix (job) only a few times; per job it keeps three tables in shared memory - the norms and,
// for a window [lo, hi) of score keys that should contain every row's threshold, per column the
// bf16 magnitude patterns A_lo[j] <= / A_hi[j] >= below / from which a weight's score is surely
// under lo / at least hi (the score norm_j * |w| is monotone in |w|).  The window is centred on
// the median of one estimate per warp: the matching quantile of the exact scores of a quarter of
// one row of the job (rows spread evenly over the matrix), selected in registers.
//
// Each warp then works on whole rows by itself, with no block barrier on the row path:
//   1. the row arrives in the warp's shared-memory buffer by cp.async;
//   2. classification, two weights per integer subtract: (w | 0x8000) - A has bit 15 set iff the
//      magnitude is >= A.  Weights under A_lo are pruned for sure, weights from A_hi up are kept
//      for sure, the few per cent in between are the row's candidates;
//   3. the candidates are queued (their columns), get their exact fp32 score key from the row and
//      the norm table, and go into a 256-bin histogram of the window;
//   4. a warp scan finds the bin that holds rank k; the keys of that bin are ranked under
//      (key, column), which is the oracle's total order, so ties need no special case;
//   5. candidates at or below the threshold are zeroed in the row buffer.  A zeroed weight has
//      magnitude 0 < A_lo, so the store pass - which masks everything under A_lo - writes both the
//      sure and the selected zeros and the keep bits from one classification.
// A row whose threshold falls outside the window, whose candidates overflow the queue, or whose
// bin holds more than 32 keys, and every row of a job whose window is unusable (non-finite norms,
// thresholds near zero or overflow) takes slow_row(): a full 4 x 8-bit radix select by the warp on
// exact keys.  All paths give the oracle's bits.
#include "prune_jobs.cuh"

namespace mosaic {

constexpr int kWMaxWarps = 16;
constexpr int kWBins = 256;
constexpr int kWBinList = 32;

// Shared-memory carve-up for rows of `cols` columns (host and device agree on it).
struct WarpLayout {
    int nvec, qcap, nwords;
    uint32_t off_alo, off_ahi, off_nrm, off_misc, off_warp0, per_warp;   // bytes
    uint32_t o_qkey, o_qcol, o_hist, o_mbytes, o_bkey, o_bcol;           // bytes inside a warp's block
};
__host__ __device__ inline WarpLayout warp_layout(int cols) {
    WarpLayout L;
    L.nvec = cols >> 3;
    L.nwords = (cols + 31) >> 5;
    L.qcap = ((cols >> 3) + 31) & ~31;                 // candidates a row may have (1/8 of it) before it goes the slow way
    uint32_t o = 0;
    L.off_alo = o;   o += (uint32_t)L.nvec * 16u;
    L.off_ahi = o;   o += (uint32_t)L.nvec * 16u;
    L.off_nrm = o;   o += (uint32_t)cols * 4u;
    L.off_misc = o;  o += 64u;
    L.off_warp0 = o;
    uint32_t w = (uint32_t)L.nvec * 16u;               // the row
    L.o_qkey = w;    w += (uint32_t)L.qcap * 4u;
    L.o_qcol = w;    w += (uint32_t)L.qcap * 2u;
    w = (w + 15u) & ~15u;
    L.o_hist = w;    w += kWBins * 4u;
    L.o_mbytes = w;  w += ((uint32_t)L.nwords * 4u + 15u) & ~15u;
    L.o_bkey = w;    w += kWBinList * 4u;
    L.o_bcol = w;    w += kWBinList * 4u;
    L.per_warp = (w + 15u) & ~15u;
    return L;
}
constexpr uint32_t kWSmemBudget = 227u * 1024u - 1024u;   // dynamic shared memory a CTA may use (static arrays need a little)

// Warps per CTA for rows of `cols` columns: as many as shared memory holds, at most kWMaxWarps.
static int warps_for(int cols) {
    const WarpLayout L = warp_layout(cols);
    if (L.off_warp0 + 3u * L.per_warp > kWSmemBudget) return 0;
    int w = (int)((kWSmemBudget - L.off_warp0) / L.per_warp);
    return w > kWMaxWarps ? kWMaxWarps : w;
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem)), "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait() {
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
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
// flags8 word -> byte with bit e = flag of element e.  ((f >> 7) & 0x01010101) holds elements 0..3
// on bits 0, 8, 16, 24; times 0x01020408 brings them to bits 24..27 in order (no two partial
// products meet on a bit, so nothing carries).
__device__ __forceinline__ uint32_t byte_of_flags(uint32_t f) {
    const uint32_t lo = (((f >> 7) & 0x01010101u) * 0x01020408u) >> 24;
    const uint32_t hi = (((f >> 6) & 0x01010101u) * 0x01020408u) >> 24;
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
// Warp-wide; clears the histogram.  Returns false if no bin holds the rank.
__device__ __forceinline__ bool warp_find_bin(uint32_t* hist, uint32_t base0, uint32_t rank, int lane, uint32_t* bin,
                                              uint32_t* rank_in_bin, uint32_t* count) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
    const uint4 a = h4[lane * 2], b = h4[lane * 2 + 1];
    h4[lane * 2] = make_uint4(0u, 0u, 0u, 0u);
    h4[lane * 2 + 1] = make_uint4(0u, 0u, 0u, 0u);
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

// Exact score key of element e of vector `vec` of the row (sign bit cleared: norms are >= +0 by
// contract, and a negative one must not index past a histogram).
__device__ __forceinline__ uint32_t exact_key(const uint4& r, const float* nrm8, int e) {
    return __float_as_uint(__fmul_rn(nrm8[e], mag_f32(word_of(r, e >> 1), e & 1))) & 0x7FFFFFFFu;
}

// Exact k-th smallest key of the row in `row` (1 <= k <= cols) by the warp: 4 x 8-bit radix select
// from the top.  T = the key, n_eq = keys equal to it, q = how many of those are among the k
// smallest.  hist must be zero on entry and is zero on exit.
template <int V>
__device__ __noinline__ void warp_exact_select(const uint4* row, const float* nrm, int nvec, uint32_t k, uint32_t* hist,
                                               uint32_t* T, uint32_t* q, uint32_t* n_eq) {
    const int lane = threadIdx.x & 31;
    uint32_t prefix = 0u, pmask = 0u, rank = k, cnt = 0u;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
#pragma unroll 2
        for (int v = 0; v < V; ++v) {
            const int vec = v * 32 + lane;
            if (vec < nvec) {
                const uint4 r = row[vec];
                const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint32_t key = exact_key(r, n8, e);
                    if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 0xFFu], 1u);
                }
            }
        }
        __syncwarp();
        uint32_t bin = 0u, rr = 0u, cc = 0u;
        warp_find_bin(hist, 0u, rank, lane, &bin, &rr, &cc);   // always found: 1 <= rank <= keys that match the prefix
        prefix |= bin << shift;
        pmask |= 0xFFu << shift;
        rank = rr;
        cnt = cc;
        __syncwarp();
    }
    *T = prefix;
    *q = rank;
    *n_eq = cnt;
}

// The always-exact treatment of one row by its warp: full select, ties by column, store, keep bits.
// Leaves the keep bits of the row as bytes in mbytes (one per vector).
template <int V>
__device__ __noinline__ void slow_row(uint4* row, const float* nrm, int nvec, uint32_t k, uint32_t* hist, uint8_t* mbytes,
                                      uint16_t* out_row) {
    const int lane = threadIdx.x & 31;
    uint32_t T, q, n_eq;
    warp_exact_select<V>(row, nrm, nvec, k, hist, &T, &q, &n_eq);
    // column of the q-th key equal to T in column order (a lane's vectors v*32 + lane ascend with v, then lane)
    uint32_t colT = 0xFFFFFFFFu;
    if (q < n_eq) {
        uint32_t before = 0u;
        bool found = false;
#pragma unroll 1
        for (int v = 0; v < V && !found; ++v) {
            const int vec = v * 32 + lane;
            uint32_t eq = 0u;
            if (vec < nvec) {
                const uint4 r = row[vec];
                const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) eq |= (exact_key(r, n8, e) == T) ? (1u << e) : 0u;
            }
            const uint32_t mine = (uint32_t)__popc(eq);
            const uint32_t incl = warp_incl_scan(mine, lane);
            const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (before + tot >= q) {
                const uint32_t excl = before + incl - mine;
                const unsigned m = __ballot_sync(0xFFFFFFFFu, excl < q && q <= excl + mine);
                const int src = __ffs(m) - 1;
                uint32_t col = 0u;
                if (lane == src) {
                    uint32_t need = q - excl;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if ((eq >> e) & 1u) {
                            if (--need == 0u) col = (uint32_t)(vec * 8 + e);
                        }
                }
                colT = __shfl_sync(0xFFFFFFFFu, col, src);
                found = true;
            }
            before += tot;
        }
    }
#pragma unroll 2
    for (int v = 0; v < V; ++v) {
        const int vec = v * 32 + lane;
        if (vec < nvec) {
            uint4 r = row[vec];
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

// Thresholds of the window [lo, lo + 2^w) for one vector of 8 columns.  For column j with norm n:
//   magnitude pattern a <  A_lo  =>  score key < lo;      a >= A_hi  =>  score key >= hi.
// With x = fl(l / n) (correctly rounded) and g = its top 16 bits (the bf16 pattern at or just
// below x), patterns <= g-2 are more than a bf16 step (2^-8 relative) below l/n, so their product
// with n rounds below l; patterns >= g+2 are above it.  A_lo >= 1 always: a zero weight scores +0,
// under any usable lo.  Norm 0: every finite weight scores 0 (sure below), inf/NaN weights are
// candidates.  Norms outside [2^-100, 2^100]: every non-zero weight is a candidate.
__device__ __forceinline__ void thresholds_of_vector(const float* nrm8, float flo, float fhi, uint4* alo, uint4* ahi) {
    uint32_t al[8], ah[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float n = nrm8[e];
        if (n == 0.0f) {
            al[e] = 0x7F80u;
            ah[e] = 0x7F82u;
        } else if (!(n >= 0x1p-100f && n <= 0x1p100f)) {
            al[e] = 1u;
            ah[e] = 0x8000u;
        } else {
            const uint32_t gl = __float_as_uint(__fdiv_rn(flo, n)) >> 16;
            const uint32_t gh = __float_as_uint(__fdiv_rn(fhi, n)) >> 16;
            al[e] = gl > 3u ? gl - 2u : 1u;
            ah[e] = gh + 2u < 0x8000u ? gh + 2u : 0x8000u;
        }
    }
    *alo = make_uint4(al[0] | (al[1] << 16), al[2] | (al[3] << 16), al[4] | (al[5] << 16), al[6] | (al[7] << 16));
    *ahi = make_uint4(ah[0] | (ah[1] << 16), ah[2] | (ah[3] << 16), ah[4] | (ah[5] << 16), ah[6] | (ah[7] << 16));
}

// blockDim.x = 32 * warps (warps >= 3); dynamic shared memory = off_warp0 + warps * per_warp of warp_layout(cols).
// Every job: cols % 8 == 0, kWarpMinCols <= cols <= V * 256, 0 < k < cols.
// FULL: cols == V * 256, so every vector slot v * 32 + lane is inside the row and no bounds test is needed.
template <int V, int NJ, bool FULL>
__global__ void __launch_bounds__(kWMaxWarps * 32, 1) prune_rows_warp_kernel(const __grid_constant__ PruneJobList<NJ> jobs,
                                                                             int64_t total_rows, int cols) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint16_t flagtab[32];   // bit of a packed candidate word -> column offset (vector within the group of 4) * 256 + element
    const WarpLayout L = warp_layout(cols);
    const int nvec = L.nvec, nwords = L.nwords;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = blockDim.x >> 5, nthreads = blockDim.x;
    uint4* alo = reinterpret_cast<uint4*>(smem + L.off_alo);
    uint4* ahi = reinterpret_cast<uint4*>(smem + L.off_ahi);
    float* nrm = reinterpret_cast<float*>(smem + L.off_nrm);
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + L.off_misc);   // [0..15] the warps' threshold estimates
    unsigned char* mine = smem + L.off_warp0 + (size_t)wid * L.per_warp;
    uint4* row = reinterpret_cast<uint4*>(mine);
    uint16_t* row16 = reinterpret_cast<uint16_t*>(mine);
    uint32_t* qkey = reinterpret_cast<uint32_t*>(mine + L.o_qkey);
    uint16_t* qcol = reinterpret_cast<uint16_t*>(mine + L.o_qcol);
    uint32_t* hist = reinterpret_cast<uint32_t*>(mine + L.o_hist);
    uint8_t* mbytes = mine + L.o_mbytes;
    uint32_t* bkey = reinterpret_cast<uint32_t*>(mine + L.o_bkey);
    uint32_t* bcol = reinterpret_cast<uint32_t*>(mine + L.o_bcol);

    if (tid < 32) {
        const int p = tid & 7, s = (7 - p) >> 1;
        const int e = (tid >> 3) + ((p & 1) ? 0 : 4);
        flagtab[tid] = (uint16_t)(s * 256 + e);
    }
    for (int b = lane; b < kWBins; b += 32) hist[b] = 0u;
    for (int b = lane; b < nwords * 4; b += 32) mbytes[b] = 0u;   // the bytes past the row's last vector stay zero: mask padding
    __syncthreads();

    const int win_bits = cols >= 8192 ? 20 : 21;   // the k-th score of a row scatters like 1/sqrt(cols)
    const int shift = win_bits - 8;
    const uint32_t width = 1u << win_bits;

    const int64_t rows_per_cta = (total_rows + gridDim.x - 1) / gridDim.x;
    const int64_t cta_begin = (int64_t)blockIdx.x * rows_per_cta;
    const int64_t cta_end = cta_begin + rows_per_cta < total_rows ? cta_begin + rows_per_cta : total_rows;
    int j = 0;
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
            fin = fin && (n >= 0.0f) && (n <= 3.402823466e38f);
        }
        bool valid = __syncthreads_and(fin ? 1 : 0) != 0;
        uint32_t lo = 0u;
        if (valid) {
            // One estimate per warp: the k-th score of row (rows-1)*wid/(nwarps-1), taken as the matching
            // quantile of the exact keys of four of each lane's vectors (a quarter of the row), which
            // the lane keeps in registers through a 4 x 8-bit radix select.
            {
                const int64_t srow = (J.rows - 1) * wid / (nwarps > 1 ? nwarps - 1 : 1);
                const uint16_t* src = J.W_in + srow * ldw;
                uint32_t key[32];
                uint32_t n_valid = 0u;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int vec = (i * (V / 4)) * 32 + lane;
                    if (FULL || vec < nvec) {
                        const uint4 r = ld_stream16(src + (int64_t)vec * kVec);   // (in place, another CTA may be writing this row: any value will do for an estimate)
                        const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                        const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
#pragma unroll
                        for (int e = 0; e < 8; ++e) key[i * 8 + e] = exact_key(r, n8, e);
                        n_valid += 8u;
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) key[i * 8 + e] = 0xFFFFFFFFu;   // matches no prefix: in no histogram
                    }
                }
                n_valid = __reduce_add_sync(0xFFFFFFFFu, n_valid);
                uint32_t rank = (uint32_t)(((uint64_t)uk * n_valid + (uint32_t)cols / 2u) / (uint32_t)cols);
                rank = rank < 1u ? 1u : (rank > n_valid ? n_valid : rank);
                uint32_t prefix = 0u, pmask = 0u;
#pragma unroll 1
                for (int sh = 24; sh >= 0; sh -= 8) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((key[i] & pmask) == prefix && key[i] != 0xFFFFFFFFu) atomicAdd(&hist[(key[i] >> sh) & 0xFFu], 1u);
                    __syncwarp();
                    uint32_t bin = 0u, rr = 0u, cc = 0u;
                    warp_find_bin(hist, 0u, rank, lane, &bin, &rr, &cc);
                    prefix |= bin << sh;
                    pmask |= 0xFFu << sh;
                    rank = rr;
                    __syncwarp();
                }
                if (lane == 0) misc[wid] = prefix;
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
            const uint32_t half = width >> 1;
            // refused where scores could be subnormal (lo < 2^24) or the window could reach inf
            valid = center >= (1u << 24) + half && center - half <= 0x7F7FFFFFu - width;
            if (valid) {
                lo = center - half;
                const float flo = __uint_as_float(lo), fhi = __uint_as_float(lo + width);
                for (int vec = tid; vec < nvec; vec += nthreads) {
                    const float4 n0 = reinterpret_cast<const float4*>(nrm)[vec * 2], n1 = reinterpret_cast<const float4*>(nrm)[vec * 2 + 1];
                    const float n8[8] = {n0.x, n0.y, n0.z, n0.w, n1.x, n1.y, n1.z, n1.w};
                    thresholds_of_vector(n8, flo, fhi, &alo[vec], &ahi[vec]);
                }
            }
        }
        __syncthreads();

        // ---------------- rows of the segment, one per warp at a time
        auto fetch = [&](int64_t rr) {   // this warp's copy of global row rr into its buffer (one cp.async group)
            const uint16_t* src = J.W_in + (rr - J.row0) * ldw;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int vec = v * 32 + lane;
                if (FULL || vec < nvec) cp_async16(&row[vec], src + (int64_t)vec * kVec);
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        if (seg + wid < seg_end) fetch(seg + wid);
        for (int64_t r = seg + wid; r < seg_end; r += nwarps) {
            const int64_t lrow = r - J.row0;
            uint16_t* out_row = J.W_out != nullptr ? J.W_out + lrow * ldw : nullptr;
            uint32_t* mask_row = J.mask != nullptr ? reinterpret_cast<uint32_t*>(J.mask + lrow * J.mask_row_bytes) : nullptr;
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();

            bool done = false;
            if (valid) {
                // ---- classification
                uint32_t candw[(V + 3) / 4];
#pragma unroll
                for (int w = 0; w < (V + 3) / 4; ++w) candw[w] = 0u;
                uint32_t below = 0u;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int vec = v * 32 + lane;
                    if (FULL || vec < nvec) {
                        const uint4 rr = row[vec], a = alo[vec], h = ahi[vec];
                        const uint32_t x0 = rr.x | 0x80008000u, x1 = rr.y | 0x80008000u, x2 = rr.z | 0x80008000u,
                                       x3 = rr.w | 0x80008000u;
                        const uint32_t keepf = flags8(x0 - a.x, x1 - a.y, x2 - a.z, x3 - a.w);
                        const uint32_t above = flags8(x0 - h.x, x1 - h.y, x2 - h.z, x3 - h.w);
                        candw[v >> 2] |= (keepf & ~above) >> (2 * (v & 3));
                        below += 8u - (uint32_t)__popc(keepf);
                    }
                }
                // ---- queue the candidates' columns
                uint32_t cnt = 0u;
#pragma unroll
                for (int w = 0; w < (V + 3) / 4; ++w) cnt += (uint32_t)__popc(candw[w]);
                const uint32_t incl = warp_incl_scan(cnt, lane);
                const uint32_t qn = __shfl_sync(0xFFFFFFFFu, incl, 31);
                if (qn <= (uint32_t)L.qcap) {
                    uint32_t off = incl - cnt;
#pragma unroll
                    for (int w = 0; w < (V + 3) / 4; ++w)
                        for (uint32_t c = candw[w]; c != 0u; c &= c - 1u)
                            qcol[off++] = (uint16_t)(w * 1024 + lane * 8 + flagtab[__ffs(c) - 1]);
                    __syncwarp();
                    // ---- exact keys of the candidates, four rounds of 32 at a time
                    for (uint32_t base = lane; base < qn; base += 128u) {
                        uint32_t col[4], a[4];
                        float n[4];
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t i = base + 32u * g;
                            col[g] = i < qn ? (uint32_t)qcol[i] : 0u;
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
                                qkey[i] = key;
                                const uint32_t d = key - lo;   // key < lo wraps to >= 2^31 (key, lo < 2^31)
                                if (d < width) atomicAdd(&hist[d >> shift], 1u);
                                else below += d >> 31;
                            }
                        }
                    }
                    below = __reduce_add_sync(0xFFFFFFFFu, below);
                    __syncwarp();
                    // ---- the bin that holds rank k, then the rank inside it under (key, column)
                    uint32_t bin = 0u, r_bin = 0u, n_bin = 0u;
                    const bool hit = warp_find_bin(hist, below, uk, lane, &bin, &r_bin, &n_bin);
                    if (hit && n_bin <= (uint32_t)kWBinList) {
                        uint32_t nl = 0u;
                        for (uint32_t base = 0u; base < qn; base += 32u) {
                            const uint32_t i = base + lane;
                            const uint32_t key = i < qn ? qkey[i] : 0u;
                            const bool in = i < qn && ((key - lo) >> shift) == bin;
                            const unsigned m = __ballot_sync(0xFFFFFFFFu, in);
                            if (in) {
                                const uint32_t pos = nl + (uint32_t)__popc(m & ((1u << lane) - 1u));
                                bkey[pos] = key;
                                bcol[pos] = (uint32_t)qcol[i];
                            }
                            nl += (uint32_t)__popc(m);
                        }
                        __syncwarp();
                        const bool have = (uint32_t)lane < n_bin;
                        const uint32_t mk = have ? bkey[lane] : 0xFFFFFFFFu, mc = have ? bcol[lane] : 0xFFFFFFFFu;
                        uint32_t less = 0u;
                        for (uint32_t jj = 0u; jj < n_bin; ++jj) {
                            const uint32_t ok = __shfl_sync(0xFFFFFFFFu, mk, (int)jj), oc = __shfl_sync(0xFFFFFFFFu, mc, (int)jj);
                            less += (ok < mk || (ok == mk && oc < mc)) ? 1u : 0u;
                        }
                        const unsigned sel = __ballot_sync(0xFFFFFFFFu, have && less + 1u == r_bin);
                        const int src_l = __ffs(sel) - 1;   // exactly one entry holds rank r_bin: the pairs are distinct
                        const uint32_t T = __shfl_sync(0xFFFFFFFFu, mk, src_l), colT = __shfl_sync(0xFFFFFFFFu, mc, src_l);
                        // ---- zero the selected candidates in the row buffer
                        for (uint32_t i = lane; i < qn; i += 32u) {
                            const uint32_t key = qkey[i], col = (uint32_t)qcol[i];
                            if (key < T || (key == T && col <= colT)) row16[col] = (uint16_t)0;
                        }
                        __syncwarp();
                        // ---- store: everything under A_lo (the sure ones and the zeroed candidates) becomes +0
#pragma unroll
                        for (int v = 0; v < V; ++v) {
                            const int vec = v * 32 + lane;
                            if (FULL || vec < nvec) {
                                const uint4 rr = row[vec], a = alo[vec];
                                const uint32_t t0 = (rr.x | 0x80008000u) - a.x, t1 = (rr.y | 0x80008000u) - a.y,
                                               t2 = (rr.z | 0x80008000u) - a.z, t3 = (rr.w | 0x80008000u) - a.w;
                                if (out_row != nullptr)
                                    st_stream16(out_row + (int64_t)vec * kVec,
                                                make_uint4(rr.x & lane_mask(t0), rr.y & lane_mask(t1), rr.z & lane_mask(t2),
                                                           rr.w & lane_mask(t3)));
                                mbytes[vec] = (uint8_t)byte_of_flags(flags8(t0, t1, t2, t3));
                            }
                        }
                        done = true;
                    }
                }
            }
            if (!done) slow_row<V>(row, nrm, nvec, uk, hist, mbytes, out_row);
            __syncwarp();   // the row buffer is free, the keep bytes are complete
            if (r + nwarps < seg_end) fetch(r + nwarps);   // the next row travels while the keep words leave
            if (mask_row != nullptr)
                for (int w = lane; w < nwords; w += 32) mask_row[w] = reinterpret_cast<const uint32_t*>(mbytes)[w];
            __syncwarp();
        }
        seg = seg_end;
    }
}

template <int V, int NJ, bool FULL>
static int launch_warp_v(const PruneJobList<NJ>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    const int warps = warps_for(cols);
    if (warps < 3) return MOSAIC_ERR_INVALID_ARG;
    const WarpLayout L = warp_layout(cols);
    const size_t dyn = (size_t)L.off_warp0 + (size_t)warps * L.per_warp;
    static DeviceCache opted;   // the shared-memory opt-in belongs to one device's copy of the kernel
    const int ok = opted.get([&]() -> int {
        if (cudaFuncSetAttribute(prune_rows_warp_kernel<V, NJ, FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kWSmemBudget) != cudaSuccess) {
            (void)cudaGetLastError();
            return -1;
        }
        return 1;
    });
    if (ok < 0) return MOSAIC_ERR_CUDA;
    int64_t grid = sm_count();
    const int64_t need = (total_rows + warps - 1) / warps;
    if (grid > need) grid = need;
    if (grid < 1) grid = 1;
    prune_rows_warp_kernel<V, NJ, FULL><<<(unsigned)grid, warps * 32, dyn, st>>>(jobs, total_rows, cols);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

template <int NJ>
static int launch_warp_any(const PruneJobList<NJ>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    const int v = (cols / 8 + 31) / 32;   // vectors per lane
    const bool full = cols % 256 == 0;
#define MOSAIC_WARP_CASE(V)                                                                       \
    if (v <= V)                                                                                   \
        return (full && cols == V * 256) ? launch_warp_v<V, NJ, true>(jobs, total_rows, cols, st) \
                                         : launch_warp_v<V, NJ, false>(jobs, total_rows, cols, st)
    MOSAIC_WARP_CASE(8);
    MOSAIC_WARP_CASE(12);
    MOSAIC_WARP_CASE(16);
    MOSAIC_WARP_CASE(20);
    MOSAIC_WARP_CASE(24);
    MOSAIC_WARP_CASE(32);
#undef MOSAIC_WARP_CASE
    return MOSAIC_ERR_INVALID_ARG;
}

int launch_prune_warp(const PruneJobList<1>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    return launch_warp_any<1>(jobs, total_rows, cols, st);
}
int launch_prune_warp(const PruneJobList<kBatchJobs>& jobs, int64_t total_rows, int cols, cudaStream_t st) {
    return launch_warp_any<kBatchJobs>(jobs, total_rows, cols, st);
}

}  // namespace mosaic
