// mosaic_score (Eq. 5 materialised) and mosaic_outlier_ratio (Eq. 6 /
// the outlier-count step of Algorithm 1): fp64 sum of the weight metric over a projection,
// threshold tau = alpha * mean, strict outlier count.
//
// Decomposition of both sweeps: a CTA of 128 threads owns a chunk of 1024
// columns (a thread owns 8 adjacent columns, whose norms stay in registers)
// and a contiguous range of rows; 8 row loads are in flight per thread.
// Sweep 1 writes one fp64 partial per CTA; the last CTA to finish adds the
// partials in index order (so the sum does not depend on scheduling) and
// publishes tau.  Sweep 2 walks the CTAs in reverse order, so that it starts on
// the part of W that sweep 1 touched last and finds it in L2, and compares in
// fp32 against tau rounded toward -inf: for an fp32 score s,
// (double)s > tau  <=>  s > fl32_down(tau), so no fp64 work is needed.
#include "common.cuh"

namespace mosaic {

constexpr int kOutThreads = 128;
constexpr int kOutChunk = kOutThreads * kVec;  // 1024 columns
constexpr int kOutUnroll = 8;

struct OutlierWs {           // layout of the workspace head
    unsigned int done;       // CTAs of sweep 1 that have published their partial
    unsigned int pad;
    float tau_down;          // alpha*mean rounded toward -inf to fp32
    float pad2;
    double sum;              // S
    double tau;              // alpha*mean in fp64
    double partial[1];       // [grid]
};

struct OutlierPlan {
    int chunks, splits, rows_per_split;
};

static OutlierPlan outlier_plan(int64_t rows, int64_t cols) {
    OutlierPlan p;
    p.chunks = (int)((cols + kOutChunk - 1) / kOutChunk);
    int64_t target = (int64_t)sm_count() * 16;
    int64_t splits = target / p.chunks;
    if (splits < 1) splits = 1;
    int64_t max_splits = (rows + kOutUnroll - 1) / kOutUnroll;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    int64_t rps = (rows + splits - 1) / splits;
    rps = (rps + kOutUnroll - 1) / kOutUnroll * kOutUnroll;
    p.rows_per_split = (int)rps;
    p.splits = (int)((rows + rps - 1) / rps);
    if (p.splits < 1) p.splits = 1;
    return p;
}

template <int DT>
__global__ void __launch_bounds__(kOutThreads) score_sum_kernel(const void* __restrict__ W, int64_t rows, int64_t cols,
                                                                 int64_t ldw, const float* __restrict__ norms, int chunks,
                                                                 int rows_per_split, float alpha, OutlierWs* ws,
                                                                 double* score_sum_out) {
    __shared__ double red[32];
    __shared__ bool is_last;
    const int chunk = blockIdx.x % chunks, split = blockIdx.x / chunks;
    const int64_t c0 = (int64_t)chunk * kOutChunk + threadIdx.x * kVec;
    const int64_t r0 = (int64_t)split * rows_per_split;
    const int64_t r1 = (r0 + rows_per_split < rows) ? r0 + rows_per_split : rows;

    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    if (c0 < cols) {
        float nrm[kVec];
#pragma unroll
        for (int e = 0; e < kVec; ++e) nrm[e] = (c0 + e < cols) ? norms[c0 + e] : 0.0f;
        int64_t r = r0;
        for (; r + kOutUnroll <= r1; r += kOutUnroll) {
            Raw8<DT> v[kOutUnroll];
#pragma unroll
            for (int u = 0; u < kOutUnroll; ++u) load_vec<DT, true>(v[u], W, (r + u) * ldw, c0, cols);
#pragma unroll
            for (int u = 0; u < kOutUnroll; ++u)
#pragma unroll
                for (int e = 0; e < kVec; ++e) acc[u & 3] += (double)__fmul_rn(nrm[e], v[u].abs_f32(e));
        }
        for (; r < r1; ++r) {
            Raw8<DT> v;
            load_vec<DT, true>(v, W, r * ldw, c0, cols);
#pragma unroll
            for (int e = 0; e < kVec; ++e) acc[0] += (double)__fmul_rn(nrm[e], v.abs_f32(e));
        }
    }
    const double mine = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    const double blk = block_sum(mine, red);
    if (threadIdx.x == 0) {
        ws->partial[blockIdx.x] = blk;
        __threadfence();
        const unsigned prev = atomicAdd(&ws->done, 1u);
        is_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // last CTA: add all partials in index order (thread-strided, then a fixed tree)
    double s = 0.0;
    for (unsigned i = threadIdx.x; i < gridDim.x; i += kOutThreads) s += __ldcg(&ws->partial[i]);
    const double total = block_sum(s, red);
    if (threadIdx.x == 0) {
        const double mean = total / (double)(rows * cols);
        const double tau = (double)alpha * mean;
        ws->sum = total;
        ws->tau = tau;
        ws->tau_down = __double2float_rd(tau);
        ws->done = 0u;
        if (score_sum_out) *score_sum_out = total;
    }
}

template <int DT>
__global__ void __launch_bounds__(kOutThreads) outlier_count_kernel(const void* __restrict__ W, int64_t rows, int64_t cols,
                                                                     int64_t ldw, const float* __restrict__ norms,
                                                                     int chunks, int rows_per_split, const OutlierWs* ws,
                                                                     unsigned long long* count_out) {
    __shared__ unsigned int red[32];
    const unsigned b = gridDim.x - 1 - blockIdx.x;  // reverse order of sweep 1
    const int chunk = b % chunks, split = b / chunks;
    const int64_t c0 = (int64_t)chunk * kOutChunk + threadIdx.x * kVec;
    const int64_t r0 = (int64_t)split * rows_per_split;
    const int64_t r1 = (r0 + rows_per_split < rows) ? r0 + rows_per_split : rows;
    const float tau = ws->tau_down;

    unsigned int cnt = 0;
    if (c0 < cols) {
        float nrm[kVec];
        bool valid[kVec];
#pragma unroll
        for (int e = 0; e < kVec; ++e) {
            valid[e] = (c0 + e < cols);
            nrm[e] = valid[e] ? norms[c0 + e] : 0.0f;
        }
        int64_t r = r1;
        for (; r - kOutUnroll >= r0; r -= kOutUnroll) {
            Raw8<DT> v[kOutUnroll];
#pragma unroll
            for (int u = 0; u < kOutUnroll; ++u) load_vec<DT, true>(v[u], W, (r - 1 - u) * ldw, c0, cols);
#pragma unroll
            for (int u = 0; u < kOutUnroll; ++u)
#pragma unroll
                for (int e = 0; e < kVec; ++e) cnt += (valid[e] && __fmul_rn(nrm[e], v[u].abs_f32(e)) > tau) ? 1u : 0u;
        }
        for (; r > r0; --r) {
            Raw8<DT> v;
            load_vec<DT, true>(v, W, (r - 1) * ldw, c0, cols);
#pragma unroll
            for (int e = 0; e < kVec; ++e) cnt += (valid[e] && __fmul_rn(nrm[e], v.abs_f32(e)) > tau) ? 1u : 0u;
        }
    }
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) red[wid] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int i = 0; i < kOutThreads / 32; ++i) t += red[i];
        if (t) atomicAdd(count_out, t);   // integer: exact in any order
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

extern "C" size_t mosaic_outlier_ratio_workspace_bytes(int64_t rows, int64_t cols) {
    if (rows <= 0 || cols <= 0) return 256;
    const OutlierPlan p = outlier_plan(rows, cols);
    return align_up(sizeof(OutlierWs) + sizeof(double) * (size_t)p.chunks * (size_t)p.splits, 256);
}

extern "C" int mosaic_outlier_ratio(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                    const float* norms, float alpha, int64_t* outlier_count_out, double* score_sum_out,
                                    void* ws, size_t ws_bytes, void* stream) {
    int rc = check_matrix(W, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (rows == 0) return MOSAIC_ERR_INVALID_ARG;
    if (!norms || !outlier_count_out || !ws) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) || (reinterpret_cast<uintptr_t>(outlier_count_out) & 7u) ||
        (reinterpret_cast<uintptr_t>(score_sum_out) & 7u) || (reinterpret_cast<uintptr_t>(norms) & 3u))
        return MOSAIC_ERR_MISALIGNED;
    if (ws_bytes < mosaic_outlier_ratio_workspace_bytes(rows, cols)) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const OutlierPlan p = outlier_plan(rows, cols);
    const unsigned grid = (unsigned)(p.chunks * p.splits);
    OutlierWs* w = static_cast<OutlierWs*>(ws);
    MOSAIC_CUDA_TRY(cudaMemsetAsync(w, 0, 16, st));
    MOSAIC_CUDA_TRY(cudaMemsetAsync(outlier_count_out, 0, sizeof(int64_t), st));
    if (dtype == MOSAIC_BF16) {
        score_sum_kernel<MOSAIC_BF16><<<grid, kOutThreads, 0, st>>>(W, rows, cols, ldw, norms, p.chunks, p.rows_per_split,
                                                                  alpha, w, score_sum_out);
        MOSAIC_LAUNCH_CHECK();
        outlier_count_kernel<MOSAIC_BF16><<<grid, kOutThreads, 0, st>>>(
            W, rows, cols, ldw, norms, p.chunks, p.rows_per_split, w, reinterpret_cast<unsigned long long*>(outlier_count_out));
    } else {
        score_sum_kernel<MOSAIC_F32><<<grid, kOutThreads, 0, st>>>(W, rows, cols, ldw, norms, p.chunks, p.rows_per_split,
                                                                 alpha, w, score_sum_out);
        MOSAIC_LAUNCH_CHECK();
        outlier_count_kernel<MOSAIC_F32><<<grid, kOutThreads, 0, st>>>(
            W, rows, cols, ldw, norms, p.chunks, p.rows_per_split, w, reinterpret_cast<unsigned long long*>(outlier_count_out));
    }
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

// ------------------------------------------------------------------------------------------
// mosaic_outlier_ratio_static: the same computation with the scratch memory built into the
// library, for callers that have no device allocator to take a workspace from.
// ------------------------------------------------------------------------------------------
namespace mosaic {

// Scratch of mosaic_outlier_ratio_static.  Every device that loads the library carries these
// 64 KiB until the process exits.  It holds the sweep counter, the threshold and one fp64
// partial sum per CTA of the first sweep (a few thousand at most on current parts).
constexpr size_t kStaticScratchBytes = MOSAIC_OUTLIER_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_outlier_scratch[kStaticScratchBytes];

// Device address of g_outlier_scratch on the current device.  In host code the array's name is
// only a handle for the runtime, not something a kernel can dereference, so the address is asked
// for once per device (with that device current) and remembered.
static int static_scratch_address(void** out) {
    static void* cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOSAIC_ERR_CUDA;
    if (dev >= 0 && dev < 64 && cached[dev] != nullptr) {
        *out = cached[dev];
        return MOSAIC_OK;
    }
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_outlier_scratch) != cudaSuccess || p == nullptr) {
        (void)cudaGetLastError();
        return MOSAIC_ERR_CUDA;
    }
    if (dev >= 0 && dev < 64) cached[dev] = p;
    *out = p;
    return MOSAIC_OK;
}

}  // namespace mosaic

extern "C" size_t mosaic_outlier_ratio_static_max_workspace_bytes(void) { return mosaic::kStaticScratchBytes; }

extern "C" int mosaic_outlier_ratio_static(const void* W, int64_t rows, int64_t cols, int64_t ldw, int dtype,
                                           const float* norms, float alpha, int64_t* outlier_count_out,
                                           double* score_sum_out, void* stream) {
    // argument errors first, so that a bad call costs no CUDA work
    int rc = check_matrix(W, rows, cols, ldw, dtype);
    if (rc != MOSAIC_OK) return rc;
    if (rows == 0) return MOSAIC_ERR_INVALID_ARG;
    if (mosaic_outlier_ratio_workspace_bytes(rows, cols) > kStaticScratchBytes) return MOSAIC_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != MOSAIC_OK) return rc;
    // The regular entry point clears the part of the scratch that must start at zero (the sweep
    // counter) on the stream before the first kernel, so what an earlier call left behind is harmless.
    return mosaic_outlier_ratio(W, rows, cols, ldw, dtype, norms, alpha, outlier_count_out, score_sum_out, scratch,
                                kStaticScratchBytes, stream);
}
