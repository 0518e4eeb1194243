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
#include <memory>
#include <new>
#include <vector>

#include "prune_jobs.cuh"
#include "select.cuh"

namespace mosaic {

// Rows of a CTA resident in shared memory: the one being selected and the next one on its way from HBM.
// A third (two in flight) was 2-4 % slower on every row length once the selection itself got faster.
constexpr int kRing = 2;
constexpr int kFastMaxCtas = 8;   // resident CTAs per SM the bf16 kernel is launched with, at most

constexpr int kListCap = kBins1;  // candidate list shares the histogram's storage
constexpr int kTrackBits = 21;    // width (log2, in key units) of a window carried from row to row
// The k-th score of a row scatters from row to row like 1/sqrt(cols): long rows get by with half the window
// (half the candidates).
__host__ __device__ constexpr int track_bits_for(int cols) { return cols >= 8192 ? kTrackBits - 1 : kTrackBits; }
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

// ---------------------------------------------------------------------------------------------
// bf16 rows, classified in the bf16 domain
// ---------------------------------------------------------------------------------------------
constexpr int kFastV = 4;          // vectors (of 8 columns) per thread
constexpr int kWinBins = 1024;     // histogram over the top 10 bits of a window
constexpr int kRoundGroup = 4;            // candidate rounds of a warp whose loads are issued together
constexpr int kQueueCap = 448;     // candidates a warp can queue (of its 1024 weights)
constexpr int kBinListCap = 512;   // keys of one histogram bin that warp 0 will rank; also the sample size limit

__device__ __forceinline__ float rcp_approx(float x) {   // relative error <= 2^-23 for normal x
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem)), "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_all_but() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// A norm of a candidate's column, read from L2 past L1.  The candidates of a row hit columns at
// random, so almost every 32-lane request has a lane that misses L1 whatever it holds, and a miss
// there costs more than the L2 access it leads to; with several norm vectors in turn (a batch)
// the L1 path was 15 % slower end to end.
__device__ __forceinline__ float ld_norm(const float* p) {
    float v;
    asm("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void sts_u16_zero(void* smem) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"((unsigned)__cvta_generic_to_shared(smem)), "h"((unsigned short)0) : "memory");
}

// A word holds two bf16 weights.  With x = word | 0x80008000 (sign bits forced on, so each 16-bit
// lane is 0x8000 + magnitude) and A two 16-bit thresholds <= 0x8000, the lanes of x - A never
// borrow from each other and bit 15 / bit 31 of the difference is set iff magnitude >= threshold.
// comb_flags gathers those two bits of the four words of a vector into one word: word i's low
// weight (element 2i) lands on bit 15-i, its high weight (element 2i+1) on bit 31-i.
__device__ __forceinline__ uint32_t comb_flags(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3) {
    return (t0 & 0x80008000u) | ((t1 >> 1) & 0x40004000u) | ((t2 >> 2) & 0x20002000u) | ((t3 >> 3) & 0x10001000u);
}
// Bit 15 / bit 31 of t spread over their 16-bit lane: 0xFFFF where the flag is set.  (prmt's
// generic mode replicates the top bit of the selected byte when bit 3 of the selector nibble is set.)
__device__ __forceinline__ uint32_t lane_mask_from_flags(uint32_t t) {
    uint32_t m;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(m) : "r"(t), "r"(0u), "r"(0xBB99u));
    return m;
}
__device__ __forceinline__ int flag_elem(int b) {   // flag bit of comb_flags -> element 0..7 of the vector
    const int half = b >> 4;
    const int i = (15 | (half << 4)) - b;
    return (i << 1) | half;
}

// Layout of a plan (32-bit words): [0] valid, [1] window lo, [2] window width log2, [3] unused, then
// for every vector slot vec = v*nt + tid eight words: Alo[0..3], Ahi[0..3].
constexpr int kPlanHeader = 4;
inline size_t plan_words(int nt) { return (size_t)kPlanHeader + (size_t)kFastV * nt * 8; }

// Thresholds of the window of width 2^w centred on `center`, for the columns of this thread
// (vectors v*nt + tid).  For column j with norm n:
//   magnitude bits a <  Alo  =>  score key < lo      (surely pruned once T >= lo)
//   magnitude bits a >= Ahi  =>  score key >= hi     (surely kept once T < hi)
// With x = l/n, the estimate x' = l * rcp(n) is within 2^-22 of x and g = top 16 bits of x' is
// the bf16 pattern just below or at x'.  Patterns <= g-2 are more than one bf16 step (2^-8)
// below x, so their product with n rounds below l; patterns >= g+2 are above x.  Alo = g-2 and
// Ahi = g+2 keep an extra step in hand.  The window is refused (false) where products could be
// subnormal (lo < 2^24) or overflow, and columns whose norm is outside [2^-100, 2^100] get
// thresholds that make every weight a candidate (norm 0: every finite weight scores 0).
template <int V>
__device__ __forceinline__ bool window_thresholds(uint32_t center, int w, const float* __restrict__ norms, int cols, int nt,
                                                  uint32_t (&Alo)[V][4], uint32_t (&Ahi)[V][4], uint32_t* lo_out) {
    const int tid = threadIdx.x;
    const uint32_t half = 1u << (w - 1);
    if (center < (1u << 24) + half) return false;
    const uint32_t lo = center - half;
    if (lo > 0x7F7FFFFFu - (1u << w)) return false;
    const float flo = __uint_as_float(lo), fhi = __uint_as_float(lo + (1u << w));
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t al[2], ah[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = (v * nt + tid) * kVec + 2 * i + h;
                al[h] = 0u;   // past the end of the row: never below, never a candidate
                ah[h] = 0u;
                if (c < cols) {
                    const float n = __ldg(norms + c);
                    if (n == 0.0f) {
                        al[h] = 0x7F80u;
                        ah[h] = 0x7F82u;
                    } else if (!(n >= 0x1p-100f && n <= 0x1p100f)) {
                        al[h] = 0u;
                        ah[h] = 0x8000u;
                    } else {
                        const float r = rcp_approx(n);
                        const uint32_t gl = __float_as_uint(__fmul_rn(flo, r)) >> 16;
                        const uint32_t gh = __float_as_uint(__fmul_rn(fhi, r)) >> 16;
                        al[h] = gl > 2u ? gl - 2u : 0u;
                        ah[h] = gh + 2u;
                    }
                }
            }
            Alo[v][i] = al[0] | (al[1] << 16);
            Ahi[v][i] = ah[0] | (ah[1] << 16);
        }
    *lo_out = lo;
    return true;
}

// True iff every norm of this thread's columns is finite and >= 0: the bf16-domain classification
// needs scores that are monotone in |w| for every column.
template <int V>
__device__ __forceinline__ bool norms_usable(const float* __restrict__ norms, int cols, int nt) {
    bool fin = true;
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const int c = (v * nt + (int)threadIdx.x) * kVec + e;
            if (c < cols) {
                const float n = __ldg(norms + c);
                fin = fin && (n >= 0.0f) && (n <= 3.402823466e38f);
            }
        }
    return fin;
}

// The candidate flags of the thread's four vectors share one word: vector v's flags move down by
// 4v bits (its eight flags sit on bits 12..15 and 28..31), so one loop over the set bits visits
// all candidates of the thread and lanes with few candidates in one vector do not wait for lanes
// with many in another.
__device__ __forceinline__ uint32_t pack_flags4(const uint32_t (&f)[4]) {
    return f[0] | (f[1] >> 4) | (f[2] >> 8) | (f[3] >> 12);
}
__device__ __forceinline__ int packed_vec(int b) { return 3 - ((b & 15) >> 2); }   // bit of the packed word -> vector

// The slow, always-exact treatment of one row held in shared memory: full radix select, ordered
// ties, store.  Returns the row's threshold key.  hist[0..kBins1) must be zero; it is zero after.
template <int V>
__device__ __noinline__ uint32_t generic_row_bf16(const uint4* my_vecs, int nt, const float* __restrict__ norms, int cols,
                                                  int nvec, uint32_t k, uint32_t* hist, uint32_t* warp_tot,
                                                  SelectResult* sel3, void* W_out, int64_t row_off, uint8_t* mask_bytes,
                                                  int64_t mask_off, int mask_row_bytes) {
    const int tid = threadIdx.x;
    Raw8<MOSAIC_BF16> raw[V];
    float nrm[V][kVec];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vec = v * nt + tid;
        if (vec < nvec) {
            const uint4 u = my_vecs[v * nt];
            raw[v].w[0] = u.x; raw[v].w[1] = u.y; raw[v].w[2] = u.z; raw[v].w[3] = u.w;
        } else {
            raw[v].clear();
        }
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            const int c = vec * kVec + e;
            nrm[v][e] = (c < cols) ? __ldg(norms + c) : __int_as_float(0x7F800000);
        }
    }
    auto key_of = [&](int v, int e) -> uint32_t { return __float_as_uint(__fmul_rn(nrm[v][e], raw[v].abs_f32(e))) & 0x7FFFFFFFu; };
    uint32_t T, q, n_eq, pruned[V];
    radix_select_row<V>(key_of, k, hist, warp_tot, sel3, nt, &T, &q, &n_eq);
    prune_flags<V>(key_of, T, q, n_eq, warp_tot, nt, pruned);
    store_row<MOSAIC_BF16, V>(raw, pruned, W_out, row_off, cols, nvec, nt, mask_bytes, mask_off, mask_row_bytes);
    return T;
}

// Every job: cols % 8 == 0, 0 < k < cols.  blockDim.x = nt, a multiple of 32 with kFastV*nt*8 >= cols and
// nt <= cols/8; dynamic shared memory: fast_dyn_smem(nt, RING).  total_rows = sum of the jobs' rows.  RING rows of the
// CTA are resident in shared memory: the one being selected and RING-1 in flight from HBM.
template <int MAXNT, int MINB, int NJ, int RING>
__global__ void __launch_bounds__(MAXNT, MINB) prune_rows_bf16_kernel(const __grid_constant__ PruneJobList<NJ> jobs,
                                                                       int64_t total_rows, int cols) {
    constexpr int V = kFastV;
    extern __shared__ __align__(16) uint4 rowbuf[];      // [RING][V][nt] row ring; then the queues
    __shared__ __align__(16) uint32_t buf[kBins1];       // window histogram + one key per bin, or the full select's histogram
    __shared__ __align__(16) uint32_t whist[256];        // warp 0's digit histogram
    __shared__ uint32_t coarse[32];                      // window histogram summed over groups of 32 bins
    __shared__ uint32_t list[kBinListCap];
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t red[32];
    __shared__ uint32_t n_list;
    __shared__ SelectResult sel3;
    __shared__ RowSelect sel;
    __shared__ uint8_t spread[16];                       // bits abcd -> 0a0b0c0d
    __shared__ uint16_t col_of_flag[32];                 // packed flag bit -> column of that weight relative to the lane's first column

    const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = nt >> 5;
    const int nvec = cols >> 3;
    const int track_bits = track_bits_for(cols);
    uint32_t* hist = buf;
    uint32_t* slot = buf + kWinBins;
    // Per warp: a queue of its candidates (who holds the weight, and its exact key), so that the
    // candidates of the warp are worked on 32 at a time whatever their spread over the lanes;
    // and per thread a word that collects which of its candidates end up pruned.
    uint32_t* qkey = reinterpret_cast<uint32_t*>(rowbuf + RING * V * nt) + wid * kQueueCap;
    uint32_t* gone_w = reinterpret_cast<uint32_t*>(rowbuf + RING * V * nt) + nwarps * kQueueCap;
    uint16_t* qid = reinterpret_cast<uint16_t*>(gone_w + nt) + wid * kQueueCap;
    // Keep-bitmask bytes of a finished row wait here (two rows' worth, alternating) and leave as
    // 4-byte stores after the next block barrier: single-byte global stores cost a third of the row time.
    uint8_t* mask_stage = reinterpret_cast<uint8_t*>(reinterpret_cast<uint16_t*>(gone_w + nt) + nwarps * kQueueCap);
    uint32_t* pending_mask = nullptr;   // where the staged bytes go (block-uniform), or nullptr
    int pending_slot = 0, stage_slot = 0;
    __shared__ uint32_t q_overflow;

    gone_w[tid] = 0u;
    if (tid == 0) q_overflow = 0u;
    for (int b = tid; b < kBins1; b += nt) buf[b] = 0u;
    if (tid < 32) coarse[tid] = 0u;
    if (tid < 16) spread[tid] = (uint8_t)((tid & 1) | ((tid & 2) << 1) | ((tid & 4) << 2) | ((tid & 8) << 3));
    if (tid < 32) col_of_flag[tid] = (uint16_t)(packed_vec(tid) * nt * kVec + flag_elem(tid + 4 * packed_vec(tid)));
    if (tid == 0) n_list = 0u;
    __syncthreads();

    // ---- the job the CTA is in (set when a row crosses into it)
    uint16_t* W_out = nullptr;
    const float* norms = nullptr;
    uint8_t* mask_bytes = nullptr;
    int64_t ldw = 0, row0 = 0, job_end = 0;
    int mask_row_bytes = 0;
    uint32_t uk = 0u;
    bool all_finite = false;

    auto prefetch = [&](int slot_idx, const uint16_t* src) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vec = v * nt + tid;
            if (vec < nvec) cp_async16(&rowbuf[(slot_idx * V + v) * nt + tid], src + (int64_t)vec * kVec);
        }
        cp_async_commit();
    };
    // Address of global row r; jj is a cursor into the job list that only moves forward.
    auto row_src = [&](int64_t r, int& jj) -> const uint16_t* {
        while (r >= jobs.job[jj].row0 + jobs.job[jj].rows) ++jj;
        return jobs.job[jj].W_in + (r - jobs.job[jj].row0) * jobs.job[jj].ldw;
    };

    // ---- window state: [win_lo, win_lo + 2^win_w) and the thread's per-column thresholds
    uint32_t Alo[V][4], Ahi[V][4];
    uint32_t win_lo = 0u;
    int win_w = 0;
    bool win_valid = false;

    auto set_window = [&](uint32_t center, int w) {
        win_valid = window_thresholds<V>(center, w, norms, cols, nt, Alo, Ahi, &win_lo);
        win_w = w;
    };

    // Exact score key of element e of the thread's vector v of the row in buffer `cur`.
    auto cand_key = [&](int cur, int v, int e) -> uint32_t {
        const uint16_t* p = reinterpret_cast<const uint16_t*>(&rowbuf[(cur * V + v) * nt + tid]);
        const uint32_t a = ((uint32_t)p[e] & 0x7FFFu) << 16;
        return __float_as_uint(__fmul_rn(__ldg(norms + (v * nt + tid) * kVec + e), __uint_as_float(a)));
    };

    // Stores the staged mask row.  Call only after a block barrier that follows the staging.
    auto flush_mask = [&]() {
        if (pending_mask != nullptr) {
            if (tid * 4 < mask_row_bytes)
                pending_mask[tid] = reinterpret_cast<const uint32_t*>(mask_stage + pending_slot * V * nt)[tid];
            pending_mask = nullptr;
        }
    };

    // Key of the matching quantile of one key per thread (element 0 of vector 0), or 0.
    auto sample_center = [&](int cur) -> uint32_t {
        __syncthreads();   // a slower warp may still be ranking the previous row's bin out of `list`
        list[tid] = cand_key(cur, 0, 0);
        __syncthreads();
        flush_mask();
        if (wid == 0) {
            uint32_t r_s = (uint32_t)(((uint64_t)uk * (uint32_t)nt + (uint32_t)cols / 2u) / (uint32_t)cols);
            r_s = r_s < 1u ? 1u : (r_s > (uint32_t)nt ? (uint32_t)nt : r_s);
            uint32_t t = 0u, qq = 0u, ne = 0u;
            const bool ok = warp_select(list, (uint32_t)nt, 0u, 31, r_s, whist, &t, &qq, &ne);
            if (lane == 0) {
                sel.ok = ok ? 1u : 0u;
                sel.lo = t;
            }
        }
        __syncthreads();
        return sel.ok != 0u ? sel.lo : 0u;
    };

    // One attempt on the current window.  0: row finished and stored (T_out set); 1: the k-th key
    // is outside the window; 2: the row needs the slow path (ties to split by column, bin overflow).
    auto fast_attempt = [&](int cur, int64_t row, uint32_t& T_out) -> int {
        const uint32_t lo = win_lo, width = 1u << win_w;
        const int shift = win_w - 10;
        uint32_t cand[V], keepf[V];   // flag words (comb_flags layout): candidates; weights not surely below lo
        uint32_t below = 0u;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const uint4 r = rowbuf[(cur * V + v) * nt + tid];
            const uint32_t x0 = r.x | 0x80008000u, x1 = r.y | 0x80008000u, x2 = r.z | 0x80008000u, x3 = r.w | 0x80008000u;
            keepf[v] = comb_flags(x0 - Alo[v][0], x1 - Alo[v][1], x2 - Alo[v][2], x3 - Alo[v][3]);
            const uint32_t above = comb_flags(x0 - Ahi[v][0], x1 - Ahi[v][1], x2 - Ahi[v][2], x3 - Ahi[v][3]);
            cand[v] = keepf[v] & ~above;
            below += 8u - (uint32_t)__popc(keepf[v]);
        }
        // queue the warp's candidates: entry = (lane that holds the weight) << 5 | packed flag bit
        const uint32_t cand_all = pack_flags4(cand);
        uint32_t q_n;
        {
            const uint32_t mine = (uint32_t)__popc(cand_all);
            uint32_t incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += n;
            }
            q_n = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (q_n > (uint32_t)kQueueCap) {
                if (lane == 0) q_overflow = 1u;   // the whole CTA gives the row to the slow path (after the barrier)
                q_n = 0u;
            } else {
                uint32_t off = incl - mine;
                for (uint32_t c = cand_all; c != 0u; c &= c - 1u) qid[off++] = (uint16_t)((lane << 5) | (__ffs(c) - 1));
            }
            __syncwarp();
        }
        // exact scores of the candidates, 32 at a time: below lo, or into the window histogram
        const uint16_t* row_elems = reinterpret_cast<const uint16_t*>(rowbuf + cur * V * nt);   // column c of the row is element c
        const int warp_col0 = (wid << 5) * kVec;
        // kRoundGroup rounds at a time, their dependent loads (entry, column, weight, norm) issued side by side
        for (uint32_t base = lane; base < q_n; base += 32u * kRoundGroup) {
            uint32_t id[kRoundGroup], a[kRoundGroup];
            int col[kRoundGroup];
            float nm[kRoundGroup];
#pragma unroll
            for (int g = 0; g < kRoundGroup; ++g) {
                const uint32_t i = base + 32u * g;
                id[g] = i < q_n ? (uint32_t)qid[i] : 0u;   // entry 0 of a spare slot: an in-range column, result unused
            }
#pragma unroll
            for (int g = 0; g < kRoundGroup; ++g) col[g] = warp_col0 + (int)(id[g] >> 5) * kVec + col_of_flag[id[g] & 31];
#pragma unroll
            for (int g = 0; g < kRoundGroup; ++g) {
                a[g] = ((uint32_t)row_elems[col[g]] & 0x7FFFu) << 16;
                nm[g] = ld_norm(norms + col[g]);
            }
#pragma unroll
            for (int g = 0; g < kRoundGroup; ++g) {
                const uint32_t i = base + 32u * g;
                if (i < q_n) {
                    const uint32_t key = __float_as_uint(__fmul_rn(nm[g], __uint_as_float(a[g])));
                    qkey[i] = key;
                    const uint32_t d = key - lo;   // key < lo wraps to >= 2^31
                    if (d < width) {
                        const uint32_t bin = d >> shift;
                        atomicAdd(&hist[bin], 1u);
                        atomicAdd(&coarse[bin >> 5], 1u);
                        slot[bin] = key;
                    } else {
                        below += d >> 31;
                    }
                }
            }
        }
        below = __reduce_add_sync(0xFFFFFFFFu, below);
        if (lane == 0) red[wid] = below;
        __syncthreads();
        flush_mask();
        if (wid == 0) {
            const uint32_t n_below = __reduce_add_sync(0xFFFFFFFFu, (lane < nwarps) ? red[lane] : 0u);
            const uint32_t cc = coarse[lane];
            uint32_t incl = cc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += n;
            }
            const uint32_t base = n_below + incl - cc;
            const unsigned m = __ballot_sync(0xFFFFFFFFu, base < uk && uk <= base + cc);
            bool ok = m != 0u;
            uint32_t bin = 0u, r_bin = 0u, n_bin = 0u;
            if (ok) {
                const int seg = __ffs(m) - 1;
                const uint32_t seg_base = __shfl_sync(0xFFFFFFFFu, base, seg);
                const uint32_t f = hist[seg * 32 + lane];
                uint32_t fi = f;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, fi, o);
                    if (lane >= o) fi += n;
                }
                const uint32_t fb = seg_base + fi - f;
                const unsigned m2 = __ballot_sync(0xFFFFFFFFu, fb < uk && uk <= fb + f);
                ok = m2 != 0u;
                if (ok) {
                    const int l2 = __ffs(m2) - 1;
                    bin = (uint32_t)(seg * 32 + l2);
                    r_bin = uk - __shfl_sync(0xFFFFFFFFu, fb, l2);
                    n_bin = __shfl_sync(0xFFFFFFFFu, f, l2);
                }
            }
            __syncwarp();
            uint4* h4 = reinterpret_cast<uint4*>(hist);   // left clean for the next attempt
#pragma unroll
            for (int j = 0; j < kWinBins / 128; ++j) h4[j * 32 + lane] = make_uint4(0u, 0u, 0u, 0u);
            coarse[lane] = 0u;
            if (lane == 0) {
                sel.ok = ok ? 1u : 0u;
                sel.bin = bin;
                sel.q = r_bin;       // rank inside the bin
                sel.n_eq = n_bin;    // keys in the bin
                sel.T = slot[bin];   // the key itself if it is alone in its bin
                sel.lo = q_overflow;  // some warp had more candidates than its queue holds
                q_overflow = 0u;
                n_list = 0u;
            }
        }
        __syncthreads();
        if (sel.lo != 0u) return 2;
        if (sel.ok == 0u) return 1;
        const uint32_t bin = sel.bin, r_bin = sel.q, n_bin = sel.n_eq;
        uint32_t T = sel.T;
        if (n_bin > 1u) {
            if (n_bin > (uint32_t)kBinListCap) return 2;
            // collect the keys of that bin; warp 0 ranks them
            for (uint32_t base = lane; base < q_n; base += 32u * kRoundGroup) {
                uint32_t key[kRoundGroup];
#pragma unroll
                for (int g = 0; g < kRoundGroup; ++g) {
                    const uint32_t i = base + 32u * g;
                    key[g] = i < q_n ? qkey[i] : lo - 1u;   // a key below the window is in no bin
                }
#pragma unroll
                for (int g = 0; g < kRoundGroup; ++g)
                    if (((key[g] - lo) >> shift) == bin) {
                        const uint32_t pos = atomicAdd(&n_list, 1u);
                        if (pos < (uint32_t)kBinListCap) list[pos] = key[g];
                    }
            }
            __syncthreads();
            if (n_bin <= 32u) {
                // a handful of keys: every warp ranks them for itself (same list, same answer), which
                // spares the hand-over through warp 0 and its barrier
                const uint32_t mine = lane < (int)n_bin ? list[lane] : 0xFFFFFFFFu;
                uint32_t less = 0u, eq = 0u;
                for (uint32_t j = 0; j < n_bin; ++j) {
                    const uint32_t o = __shfl_sync(0xFFFFFFFFu, mine, (int)j);
                    less += (o < mine) ? 1u : 0u;
                    eq += (o == mine) ? 1u : 0u;
                }
                const unsigned hit = __ballot_sync(0xFFFFFFFFu, lane < (int)n_bin && less < r_bin && r_bin <= less + eq);
                const int src = __ffs(hit) - 1;   // some key holds rank r_bin (1 <= r_bin <= n_bin)
                T = __shfl_sync(0xFFFFFFFFu, mine, src);
                // a tie group that is only partly pruned goes the slow way
                if (hit == 0u || r_bin - __shfl_sync(0xFFFFFFFFu, less, src) != __shfl_sync(0xFFFFFFFFu, eq, src)) return 2;
            } else {
                if (wid == 0) {
                    uint32_t t = 0u, qq = 0u, ne = 0u;
                    const bool ok = warp_select(list, n_bin, lo + (bin << shift), shift, r_bin, whist, &t, &qq, &ne);
                    if (lane == 0) {
                        sel.ok = (ok && qq == ne) ? 1u : 0u;   // a tie group that is only partly pruned goes the slow way
                        sel.T = t;
                    }
                }
                __syncthreads();
                if (sel.ok == 0u) return 2;
                T = sel.T;
            }
        }

        // prune: surely below lo, or a candidate whose exact key is <= T
        const uint32_t thr = T + 1u;
        uint16_t* out_row = W_out + row * ldw;
        for (uint32_t base = lane; base < q_n; base += 32u * kRoundGroup) {
            uint32_t key[kRoundGroup], id[kRoundGroup];
#pragma unroll
            for (int g = 0; g < kRoundGroup; ++g) {
                const uint32_t i = base + 32u * g;
                key[g] = i < q_n ? qkey[i] : 0xFFFFFFFFu;   // never below thr <= 2^31
                id[g] = i < q_n ? (uint32_t)qid[i] : 0u;
            }
#pragma unroll
            for (int g = 0; g < kRoundGroup; ++g)
                if (key[g] < thr) {
                    const int col = warp_col0 + (int)(id[g] >> 5) * kVec + col_of_flag[id[g] & 31];
                    sts_u16_zero(reinterpret_cast<uint16_t*>(rowbuf + cur * V * nt) + col);
                    atomicOr(&gone_w[(wid << 5) | (int)(id[g] >> 5)], 1u << (id[g] & 31));
                }
        }
        __syncwarp();
        const uint32_t gone_all = gone_w[tid];
        gone_w[tid] = 0u;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int vec = v * nt + tid;
            const uint32_t gone = (gone_all << (4 * v)) & 0xF000F000u;
            if (vec < nvec) {
                const uint4 r = rowbuf[(cur * V + v) * nt + tid];
                uint4 o;
                // byte 1 / byte 3 of a difference carry the "not below" flag in their top bit: spread it over the lane
                o.x = r.x & lane_mask_from_flags((r.x | 0x80008000u) - Alo[v][0]);
                o.y = r.y & lane_mask_from_flags((r.y | 0x80008000u) - Alo[v][1]);
                o.z = r.z & lane_mask_from_flags((r.z | 0x80008000u) - Alo[v][2]);
                o.w = r.w & lane_mask_from_flags((r.w | 0x80008000u) - Alo[v][3]);
                if (W_out != nullptr) st_stream16(out_row + (int64_t)vec * kVec, o);
            }
            if (mask_bytes != nullptr) {
                uint32_t keep = 0u;
                if (vec < nvec) {
                    const uint32_t rr = __brev(keepf[v] & ~gone);   // odd elements on bits 0..3, even ones on bits 16..19
                    keep = (uint32_t)spread[(rr >> 16) & 0xFu] | ((uint32_t)spread[rr & 0xFu] << 1);
                }
                mask_stage[stage_slot * V * nt + vec] = (uint8_t)keep;   // slots past the row's end hold the padding zeros
            }
        }
        if (mask_bytes != nullptr) {
            pending_mask = reinterpret_cast<uint32_t*>(mask_bytes + row * mask_row_bytes);
            pending_slot = stage_slot;
            stage_slot ^= 1;
        }
        T_out = T;
        return 0;
    };

    int cur = 0, nxt = RING - 1, j_next = 0, j_cur = 0;
    int64_t r = blockIdx.x;
#pragma unroll
    for (int d = 0; d < RING - 1; ++d) {   // fill the ring: rows r, r+grid, ... (one copy group each, possibly empty)
        if (r + d * (int64_t)gridDim.x < total_rows) prefetch(d, row_src(r + d * (int64_t)gridDim.x, j_next));
        else cp_async_commit();
    }
    for (; r < total_rows; r += gridDim.x, cur = (cur + 1 == RING ? 0 : cur + 1), nxt = (nxt + 1 == RING ? 0 : nxt + 1)) {
        const int64_t r_far = r + (RING - 1) * (int64_t)gridDim.x;
        if (r_far < total_rows) prefetch(nxt, row_src(r_far, j_next));
        else cp_async_commit();
        cp_async_wait_all_but<RING - 1>();   // this row has landed (the RING-1 younger groups may still be in flight)
        __syncwarp();                        // ... for every lane of the warp: lanes read each other's vectors

        if (r >= job_end) {   // the row belongs to the next job: pick up its parameters and its plan
            while (r >= jobs.job[j_cur].row0 + jobs.job[j_cur].rows) ++j_cur;
            const PruneJob& J = jobs.job[j_cur];
            W_out = J.W_out;
            norms = J.norms;
            mask_bytes = J.mask;
            ldw = J.ldw;
            row0 = J.row0;
            job_end = J.row0 + J.rows;
            mask_row_bytes = J.mask_row_bytes;
            uk = (uint32_t)J.k;
            win_valid = false;
            const uint32_t* plan = J.plan;
            const bool planned = plan != nullptr && plan[0] != 0u;   // a valid plan vouches for the norms
            all_finite = planned || __syncthreads_and(norms_usable<V>(norms, cols, nt) ? 1 : 0) != 0;
            if (planned) {
                win_lo = plan[1];
                win_w = (int)plan[2];
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const uint4* p = reinterpret_cast<const uint4*>(plan + kPlanHeader + (size_t)(v * nt + tid) * 8);
                    const uint4 a = p[0], b = p[1];
                    Alo[v][0] = a.x; Alo[v][1] = a.y; Alo[v][2] = a.z; Alo[v][3] = a.w;
                    Ahi[v][0] = b.x; Ahi[v][1] = b.y; Ahi[v][2] = b.z; Ahi[v][3] = b.w;
                }
                win_valid = true;
            }
        }
        const int64_t row = r - row0;   // row inside the job

        int status = 1;
        uint32_t T_row = 0u;
        if (all_finite) {
            for (int tries = 0; tries < 2 && status == 1; ++tries) {
                if (!win_valid || tries == 1) {
                    set_window(sample_center(cur), kSampleBits);
                }
                if (!win_valid) break;
                status = fast_attempt(cur, row, T_row);
            }
        }
        if (status != 0) {
            for (int b = tid; b < kWinBins; b += nt) slot[b] = 0u;
            __syncthreads();
            flush_mask();
            T_row = generic_row_bf16<V>(&rowbuf[(cur * V) * nt + tid], nt, norms, cols, nvec, uk, buf, warp_tot, &sel3, W_out,
                                        row * ldw, mask_bytes, row * mask_row_bytes, mask_row_bytes);
        }
        if (all_finite && (status != 0 || win_w != track_bits)) set_window(T_row, track_bits);
    }
    __syncthreads();
    flush_mask();
}

// One CTA per job: the exact thresholds of three rows (first, middle, last) by the full radix
// select, a window of width 2^track_bits_for(cols) centred on their median, and the per-column thresholds
// of that window in the layout the pruning kernel loads (same nt).
template <int MAXNT, int NJ>
__global__ void __launch_bounds__(MAXNT, 1) prune_plan_kernel(const __grid_constant__ PruneJobList<NJ> jobs, int cols) {
    constexpr int V = kFastV;
    __shared__ __align__(16) uint32_t hist[kBins1];
    __shared__ uint32_t warp_tot[32];
    __shared__ SelectResult sel3;
    const int nt = blockDim.x, tid = threadIdx.x;
    const int nvec = cols >> 3;
    const PruneJob& J = jobs.job[blockIdx.x];
    uint32_t* plan = J.plan;
    if (plan == nullptr) return;
    for (int b = tid; b < kBins1; b += nt) hist[b] = 0u;
    const bool usable = __syncthreads_and(norms_usable<V>(J.norms, cols, nt) ? 1 : 0) != 0;
    bool valid = usable;
    uint32_t Alo[V][4], Ahi[V][4], lo = 0u;
    if (usable) {
        float nrm[V][kVec];
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int e = 0; e < kVec; ++e) {
                const int c = (v * nt + tid) * kVec + e;
                nrm[v][e] = (c < cols) ? __ldg(J.norms + c) : __int_as_float(0x7F800000);
            }
        uint32_t Ts[3];
#pragma unroll 1
        for (int s = 0; s < 3; ++s) {
            const int64_t row = (s == 0) ? 0 : (s == 1 ? J.rows / 2 : J.rows - 1);
            Raw8<MOSAIC_BF16> raw[V];
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int vec = v * nt + tid;
                if (vec < nvec) raw[v].template load<true>(J.W_in + row * J.ldw + (int64_t)vec * kVec);
                else raw[v].clear();
            }
            auto key_of = [&](int v, int e) -> uint32_t { return __float_as_uint(__fmul_rn(nrm[v][e], raw[v].abs_f32(e))) & 0x7FFFFFFFu; };
            uint32_t q, n_eq;
            radix_select_row<V>(key_of, (uint32_t)J.k, hist, warp_tot, &sel3, nt, &Ts[s], &q, &n_eq);
        }
        const uint32_t mx = max(max(Ts[0], Ts[1]), Ts[2]), mn = min(min(Ts[0], Ts[1]), Ts[2]);
        const uint32_t median = (uint32_t)((uint64_t)Ts[0] + Ts[1] + Ts[2] - mx - mn);
        valid = window_thresholds<V>(median, track_bits_for(cols), J.norms, cols, nt, Alo, Ahi, &lo);
    }
    if (valid) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            uint4* p = reinterpret_cast<uint4*>(plan + kPlanHeader + (size_t)(v * nt + tid) * 8);
            p[0] = make_uint4(Alo[v][0], Alo[v][1], Alo[v][2], Alo[v][3]);
            p[1] = make_uint4(Ahi[v][0], Ahi[v][1], Ahi[v][2], Ahi[v][3]);
        }
    }
    if (tid == 0) {
        plan[0] = valid ? 1u : 0u;
        plan[1] = lo;
        plan[2] = (uint32_t)track_bits_for(cols);
        plan[3] = 0u;
    }
}

// Row ring (`ring` rows of kFastV*nt vectors), per-warp queues (key + id per entry), one word per thread,
// two staged mask rows.
static size_t fast_dyn_smem(int nt, int ring) {
    return (size_t)ring * kFastV * nt * sizeof(uint4) + (size_t)(nt / 32) * kQueueCap * 6 + (size_t)nt * 4 +
           (size_t)2 * kFastV * nt;
}

// Launches the pruning kernel (and, with_plan, the planning kernel before it) over a list of jobs.
template <int MAXNT, int MINB, int NJ, int RING>
static int launch_prune_bf16(const PruneJobList<NJ>& jobs, int64_t total_rows, int cols, int nt, bool with_plan,
                             cudaStream_t st) {
    // The shared-memory opt-in and the occupancy belong to one device's copy of the kernel: both are
    // looked up once per device and per CTA size (value -1: the opt-in was refused).
    static DeviceCache blocks_per_sm[MAXNT / 32 + 1];
    const size_t dyn = fast_dyn_smem(nt, RING);
    const int bps = blocks_per_sm[nt / 32].get([&]() -> int {
        if (cudaFuncSetAttribute(prune_rows_bf16_kernel<MAXNT, MINB, NJ, RING>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)fast_dyn_smem(MAXNT, RING)) != cudaSuccess) {
            (void)cudaGetLastError();
            return -1;
        }
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, prune_rows_bf16_kernel<MAXNT, MINB, NJ, RING>, nt, dyn) != cudaSuccess ||
            n < 1) {
            (void)cudaGetLastError();
            n = 1;
        }
        return n > kFastMaxCtas ? kFastMaxCtas : n;
    });
    if (bps < 0) return MOSAIC_ERR_CUDA;
    if (with_plan) {
        prune_plan_kernel<MAXNT, NJ><<<(unsigned)jobs.n, nt, 0, st>>>(jobs, cols);
        MOSAIC_LAUNCH_CHECK();
    }
    int64_t grid = (int64_t)sm_count() * bps;
    if (grid > total_rows) grid = total_rows;
    prune_rows_bf16_kernel<MAXNT, MINB, NJ, RING><<<(unsigned)grid, nt, dyn, st>>>(jobs, total_rows, cols);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

template <int NJ>
static int dispatch_prune_bf16(const PruneJobList<NJ>& jobs, int64_t total_rows, int cols, int nt, bool with_plan,
                               cudaStream_t st) {
    // CTAs per SM are chosen so that a thread keeps about 128 registers where shared memory allows it: with the
    // thresholds in registers, a smaller budget spills them (rows of 5120 / 8192 columns ran 25 % slower at 80).
    if (nt <= 128) return launch_prune_bf16<128, 4, NJ, kRing>(jobs, total_rows, cols, nt, with_plan, st);
    if (nt <= 160) return launch_prune_bf16<160, 3, NJ, kRing>(jobs, total_rows, cols, nt, with_plan, st);
    if (nt <= 256) return launch_prune_bf16<256, 2, NJ, kRing>(jobs, total_rows, cols, nt, with_plan, st);
    if (nt <= 352) return launch_prune_bf16<352, 2, NJ, kRing>(jobs, total_rows, cols, nt, with_plan, st);
    if (nt <= 384) return launch_prune_bf16<384, 2, NJ, kRing>(jobs, total_rows, cols, nt, with_plan, st);
    return launch_prune_bf16<512, 1, NJ, kRing>(jobs, total_rows, cols, nt, with_plan, st);
}

// True iff the warp-per-row kernel (prune_warp.cu) takes rows of this shape.
static bool warp_kernel_takes(int dtype, int64_t cols, int64_t k) {
    return dtype == MOSAIC_BF16 && cols % kVec == 0 && k > 0 && k < cols && cols >= kWarpMinCols && cols <= kWarpMaxCols;
}

// Threads per CTA of the CTA-per-row bf16 kernel for rows of `cols` columns, or 0 if the shape is not for it.
static int fast_threads(int dtype, int64_t cols, int64_t k) {
    if (dtype != MOSAIC_BF16 || cols % kVec != 0 || k <= 0 || k >= cols) return 0;
    const int64_t nvec = cols / kVec;
    const int64_t nt = ((nvec + kFastV - 1) / kFastV + 31) / 32 * 32;
    return (nvec >= 256 && nt <= 512) ? (int)nt : 0;
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
                              reinterpret_cast<uint8_t*>(mask_out), nullptr, rows, ldw, 0, (int)k,
                              (int)((cols + 31) / 32) * 4};
        return launch_prune_warp(one, rows, (int)cols, st);
    }
    if (const int nt = fast_threads(dtype, cols, k)) {
        PruneJobList<1> one;
        one.n = 1;
        one.job[0] = PruneJob{static_cast<const uint16_t*>(W_in), static_cast<uint16_t*>(W_out), norms,
                              reinterpret_cast<uint8_t*>(mask_out), nullptr, rows, ldw, 0, (int)k,
                              (int)((cols + 31) / 32) * 4};
        return dispatch_prune_bf16<1>(one, rows, (int)cols, nt, false, st);
    }
    if (dtype == MOSAIC_BF16)
        return dispatch_prune<MOSAIC_BF16>(W_in, W_out, rows, (int)cols, ldw, norms, (int)k, mask_out, st);
    return dispatch_prune<MOSAIC_F32>(W_in, W_out, rows, (int)cols, ldw, norms, (int)k, mask_out, st);
}

// Workspace of the batched call: one plan (window + per-column thresholds) per job that the bf16
// kernel takes, 256-byte aligned, in job order.
static size_t batch_plan_bytes(const mosaic_prune_job& j, int dtype) {
    if (warp_kernel_takes(dtype, j.cols, j.k)) return 0;   // that kernel finds its windows itself
    const int nt = (j.rows > 0) ? fast_threads(dtype, j.cols, j.k) : 0;
    return nt ? align_up(plan_words(nt) * sizeof(uint32_t), 256) : 0;
}

extern "C" size_t mosaic_prune_unstructured_batch_workspace_bytes(const mosaic_prune_job* jobs, int64_t n_jobs, int dtype) {
    size_t total = 256;
    if (jobs == nullptr) return total;
    for (int64_t i = 0; i < n_jobs; ++i) total += batch_plan_bytes(jobs[i], dtype);
    return total;
}

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
    const size_t need = mosaic_prune_unstructured_batch_workspace_bytes(jobs, n_jobs, dtype);
    if (need > 256) {
        if (ws == nullptr) return MOSAIC_ERR_NULL_PTR;
        if (reinterpret_cast<uintptr_t>(ws) & 255u) return MOSAIC_ERR_MISALIGNED;
        if (ws_bytes < need) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // jobs for the bf16 kernel are launched together, one launch (plus its planning launch) per
    // distinct row length and per kBatchJobs jobs; everything else goes through the single call
    std::vector<char> done((size_t)n_jobs, 0);
    std::vector<size_t> plan_off((size_t)n_jobs, 0);
    size_t off = 0;
    for (int64_t i = 0; i < n_jobs; ++i) {
        plan_off[(size_t)i] = off;
        off += batch_plan_bytes(jobs[i], dtype);
    }
    // host staging of the kernel parameter (18 KB: on the heap, one per call, so concurrent callers do not meet)
    std::unique_ptr<PruneJobList<kBatchJobs>> list_mem(new (std::nothrow) PruneJobList<kBatchJobs>);
    if (!list_mem) return MOSAIC_ERR_INVALID_ARG;
    PruneJobList<kBatchJobs>& list = *list_mem;
    for (int64_t i = 0; i < n_jobs; ++i) {
        if (done[(size_t)i]) continue;
        const mosaic_prune_job& lead = jobs[i];
        const bool by_warp = lead.rows > 0 && warp_kernel_takes(dtype, lead.cols, lead.k);
        const int nt = (lead.rows > 0 && !by_warp) ? fast_threads(dtype, lead.cols, lead.k) : 0;
        if (by_warp) {   // all jobs of this row length that the warp-per-row kernel takes, kBatchJobs per launch
            list.n = 0;
            int64_t total_rows = 0;
            for (int64_t m = i; m < n_jobs; ++m) {
                const mosaic_prune_job& j = jobs[m];
                if (done[(size_t)m] || j.cols != lead.cols || j.rows <= 0 || !warp_kernel_takes(dtype, j.cols, j.k)) continue;
                done[(size_t)m] = 1;
                list.job[list.n] = PruneJob{static_cast<const uint16_t*>(j.W_in), static_cast<uint16_t*>(j.W_out), j.norms,
                                            reinterpret_cast<uint8_t*>(j.mask_out), nullptr, j.rows, j.ldw, total_rows,
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
        if (nt == 0) {   // short or very long rows, fp32, k = 0 or k = cols: the general kernel, one launch per job
            done[(size_t)i] = 1;
            const int rc = mosaic_prune_unstructured(lead.W_in, lead.W_out, lead.rows, lead.cols, lead.ldw, dtype, lead.norms,
                                                     lead.k, lead.mask_out, nullptr, 0, stream);
            if (rc != MOSAIC_OK) return rc;
            continue;
        }
        list.n = 0;
        int64_t total_rows = 0;
        for (int64_t m = i; m < n_jobs; ++m) {
            const mosaic_prune_job& j = jobs[m];
            if (done[(size_t)m] || j.cols != lead.cols || j.rows <= 0 || warp_kernel_takes(dtype, j.cols, j.k) ||
                fast_threads(dtype, j.cols, j.k) == 0)
                continue;
            done[(size_t)m] = 1;
            list.job[list.n] = PruneJob{static_cast<const uint16_t*>(j.W_in), static_cast<uint16_t*>(j.W_out), j.norms,
                                        reinterpret_cast<uint8_t*>(j.mask_out),
                                        reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + plan_off[(size_t)m]), j.rows,
                                        j.ldw, total_rows, (int)j.k, (int)((j.cols + 31) / 32) * 4};
            total_rows += j.rows;
            if (++list.n == kBatchJobs || m == n_jobs - 1) {
                const int rc = dispatch_prune_bf16<kBatchJobs>(list, total_rows, (int)lead.cols, nt, true, st);
                if (rc != MOSAIC_OK) return rc;
                list.n = 0;
                total_rows = 0;
            }
        }
        if (list.n > 0) {
            const int rc = dispatch_prune_bf16<kBatchJobs>(list, total_rows, (int)lead.cols, nt, true, st);
            if (rc != MOSAIC_OK) return rc;
        }
    }
    return MOSAIC_OK;
}
