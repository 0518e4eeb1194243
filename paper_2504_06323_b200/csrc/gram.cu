// mosaic_gram_accumulate: G += X^T X for one chunk of calibration tokens (bf16 activations, fp32
// accumulation) - the second-moment matrix from which the inverse-Hessian back-end of Section
// 4.1.2 forms its layer Hessian H = (2/T) G with the calibration samples of Section 4.1.3.  Its
// diagonal is the squared norm of Eq. 5.
//
// A dense contraction over the token dimension, so it runs on the tensor cores:
//   * G is cut into 256 x 256 blocks; only blocks on or above the diagonal are computed, the
//     mirror image of an off-diagonal block is written by the same epilogue;
//   * one persistent CTA per SM walks its blocks.  Per block the 512 columns of tensor memory
//     hold the 256 x 256 fp32 accumulator as two 128-row halves;
//   * both operands are column blocks of X, read straight from the row-major [tokens, cols]
//     tensor by TMA in boxes of 64 columns x 64 tokens with the 128-byte swizzle.  In shared
//     memory the columns of a token lie contiguous, i.e. both operands are "MN-major", which
//     tcgen05.mma takes through its instruction descriptor - X is never transposed;
//   * warp 0 issues the TMA loads of a 3-stage ring, one thread of warp 1 issues the MMAs (eight
//     128 x 256 x 16 per stage) and commits each stage back to the loader, warps 2..9 drain the
//     accumulator with tcgen05.ld once the block's last MMA has completed.  On a diagonal block the
//     two operands are the same columns: they are loaded once.
// A block is accumulated by one CTA in token order, so results do not depend on the grid.
// Every wait on an mbarrier is bounded; a wait that runs out sets the kernel's error word, all
// roles leave their loops, loads in flight are awaited (bounded), tensor memory is freed.
#include <cuda.h>   // CUtensorMap and its enums; the encoder itself is looked up at run time

#include "common.cuh"

namespace mosaic {
namespace {

constexpr int kGBlk = 256;                                               // block edge
constexpr int kGTok = 64;                                                // tokens per stage
constexpr int kGStages = 3;
constexpr int kGBoxCols = 64;                                            // 64 bf16 = one 128-byte swizzle row
constexpr uint32_t kGBoxBytes = kGBoxCols * kGTok * 2;                   // 8 KB
constexpr uint32_t kGOperandBytes = (kGBlk / kGBoxCols) * kGBoxBytes;    // 256 columns x 64 tokens = 32 KB
constexpr uint32_t kGStageBytes = 2 * kGOperandBytes;                    // A block, then B block
constexpr int kGEpiWarps = 8;                                            // two per quarter of the tensor-memory lanes
constexpr int kGThreads = 64 + 32 * kGEpiWarps;
constexpr uint32_t kGTmemCols = 512;
constexpr size_t kGSmemBytes = (size_t)kGStages * kGStageBytes + 1024 /* alignment */ + 256 /* barriers */;
constexpr long long kGWaitCycles = 4000000000ll;                         // about two seconds

// Instruction descriptor of tcgen05.mma kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16
// (bits 7-9 and 10-12 = 1), A and B MN-major (bits 15, 16), N / 8 at bit 17, M / 16 at bit 24.
constexpr uint32_t kGInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0u;
}
// Waits for the phase of the given parity to complete.  False if it gave up: after kGWaitCycles
// (then it raises *err) or because another role raised *err.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* err, long long budget = kGWaitCycles) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*err != 0) return false;
        if (clock64() - t0 > budget) {
            *err = 1;
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_box(void* dst, const CUtensorMap* map, uint64_t* bar, int col, int token) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                     smem_u32(dst)),
                 "l"(map), "r"(smem_u32(bar)), "r"(col), "r"(token)
                 : "memory");
}

// Shared-memory operand descriptor, MN-major with the 128-byte swizzle: 64 columns of a token are
// contiguous (one swizzle row), the rows of 8 consecutive tokens lie 128 bytes apart, groups of 8
// tokens 1024 bytes apart (stride offset), the next 64 columns one TMA box further (leading offset).
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr) {
    uint64_t d = (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((kGBoxBytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((1024u >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version of this architecture
    d |= (uint64_t)2 << 61;   // 128-byte swizzle
    return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t"
        "}"
        :
        : "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(kGInstrDesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}
// The barrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 consecutive accumulator columns of this thread's lane of tensor memory.
__device__ __forceinline__ void tmem_load16(uint32_t addr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(addr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Block (bi, bj), bi <= bj, number `tile` in the row-by-row list of the blocks on or above the diagonal.
__device__ __forceinline__ void block_of_tile(int tile, int n_blk, int* bi, int* bj) {
    int i = 0, rem = tile;
    while (rem >= n_blk - i) {
        rem -= n_blk - i;
        ++i;
    }
    *bi = i;
    *bj = i + rem;
}

__global__ void __launch_bounds__(kGThreads, 1) gram_kernel(const __grid_constant__ CUtensorMap x_map, float* __restrict__ G, int64_t ldg,
                                                            int cols, int tokens, int n_blk, int n_tiles, int reset, int* status) {
    extern __shared__ unsigned char gram_smem_raw[];
    unsigned char* stages = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(gram_smem_raw) + 1023u) & ~(uintptr_t)1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(stages + (size_t)kGStages * kGStageBytes);
    uint64_t* full = bars;                    // [kGStages] loads of a stage have landed
    uint64_t* empty = bars + kGStages;        // [kGStages] the MMAs reading a stage have completed
    uint64_t* acc_full = bars + 2 * kGStages;       // the block's accumulator is complete
    uint64_t* acc_empty = bars + 2 * kGStages + 1;  // the epilogue has read it
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kGStages + 2);
    volatile int* err = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGStages; ++s) {
            mbar_init(&full[s], 1u);
            mbar_init(&empty[s], 1u);
        }
        mbar_init(acc_full, 1u);
        mbar_init(acc_empty, (uint32_t)kGEpiWarps);   // one arrival per epilogue warp
        *err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kGTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int nk = (tokens + kGTok - 1) / kGTok;
    uint32_t issued = 0;   // stages the loader thread has issued loads for

    if (warp == 0) {
        // ------------------------------------------------------------ loader
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                int bi, bj;
                block_of_tile(tile, n_blk, &bi, &bj);
                for (int k = 0; k < nk; ++k, ++it) {
                    const uint32_t s = it % kGStages, ph = (it / kGStages) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u, err)) {
                        ok = false;
                        break;
                    }
                    unsigned char* st = stages + (size_t)s * kGStageBytes;
                    mbar_expect_tx(&full[s], bi == bj ? kGOperandBytes : kGStageBytes);
#pragma unroll
                    for (int b = 0; b < kGBlk / kGBoxCols; ++b)
                        tma_load_box(st + kGOperandBytes + (size_t)b * kGBoxBytes, &x_map, &full[s], bj * kGBlk + b * kGBoxCols, k * kGTok);
                    if (bi != bj) {
#pragma unroll
                        for (int b = 0; b < kGBlk / kGBoxCols; ++b)
                            tma_load_box(st + (size_t)b * kGBoxBytes, &x_map, &full[s], bi * kGBlk + b * kGBoxCols, k * kGTok);
                    }
                }
            }
            issued = it;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issue
        if (lane == 0) {
            uint32_t it = 0, n = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++n) {
                int bi, bj;
                block_of_tile(tile, n_blk, &bi, &bj);
                if (!mbar_wait(acc_empty, (n & 1u) ^ 1u, err)) break;   // the epilogue has drained the previous block
                tc_fence_after();
                for (int k = 0; k < nk; ++k, ++it) {
                    const uint32_t s = it % kGStages, ph = (it / kGStages) & 1u;
                    if (!mbar_wait(&full[s], ph, err)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t st = smem_u32(stages + (size_t)s * kGStageBytes);
                    const uint32_t b_base = st + kGOperandBytes;
                    const uint32_t a_base = bi == bj ? b_base : st;
#pragma unroll
                    for (int kk = 0; kk < kGTok / 16; ++kk) {
                        // 16 tokens further = 16 swizzle rows = 2048 bytes
                        const uint64_t db = operand_desc(b_base + (uint32_t)kk * 2048u);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint64_t da = operand_desc(a_base + (uint32_t)h * 2u * kGBoxBytes + (uint32_t)kk * 2048u);
                            umma_bf16(tmem_base + (uint32_t)h * 256u, da, db, (k > 0 || kk > 0) ? 1u : 0u);
                        }
                    }
                    umma_commit(&empty[s]);
                }
                if (ok) umma_commit(acc_full);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9)
        // A warp reads the quarter (warp % 4) of the tensor-memory lanes; the two warps of a quarter
        // split the accumulator's columns.  Passes of 16 columns: all old values of a pass (direct
        // block and mirror block) are read before its first store, one round trip per pass.
        const int q = warp & 3;
        const int c_begin = ((warp - 2) >> 2) * (kGBlk / 2);
        uint32_t n = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++n) {
            int bi, bj;
            block_of_tile(tile, n_blk, &bi, &bj);
            if (!mbar_wait(acc_full, n & 1u, err)) break;
            tc_fence_after();
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                const int64_t row = (int64_t)bi * kGBlk + h * 128 + q * 32 + lane;   // accumulator row = lane of tensor memory
#pragma unroll 1
                for (int c0 = c_begin; c0 < c_begin + kGBlk / 2; c0 += 16) {
                    float v[16];
                    tmem_load16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * 256 + c0), v);
                    const int64_t col0 = (int64_t)bj * kGBlk + c0;
                    if (row < cols) {
                        float* g = G + row * ldg + col0;      // direct block: 64 bytes of the lane's own row
                        float* m = G + col0 * ldg + row;      // mirror block: a warp covers 32 adjacent rows of a column
                        const bool mirror = bi != bj;
                        float4 o[4];
                        float om[16];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {   // cols % 8 == 0: a group of four is inside or outside as a whole
                            o[e] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                            if (!reset && col0 + 4 * e < cols) o[e] = *reinterpret_cast<const float4*>(g + 4 * e);
                        }
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            om[e] = 0.0f;
                            if (!reset && mirror && col0 + e < cols) om[e] = m[(int64_t)e * ldg];
                        }
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (col0 + 4 * e < cols) {
                                float4 w = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
                                if (!reset) {
                                    w.x = __fadd_rn(o[e].x, w.x);
                                    w.y = __fadd_rn(o[e].y, w.y);
                                    w.z = __fadd_rn(o[e].z, w.z);
                                    w.w = __fadd_rn(o[e].w, w.w);
                                }
                                *reinterpret_cast<float4*>(g + 4 * e) = w;
                            }
                        }
                        if (mirror) {
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                if (col0 + e < cols) m[(int64_t)e * ldg] = reset ? v[e] : __fadd_rn(om[e], v[e]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kGTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && *err != 0) {
        // Some role gave up.  Every role has left its loop by now; let the loads of the last stages
        // land before the CTA leaves its shared memory (a completed phase answers at once; bounded).
        for (uint32_t back = 1; back <= (uint32_t)kGStages && back <= issued; ++back) {
            const uint32_t j = issued - back, s = j % kGStages, ph = (j / kGStages) & 1u;
            const long long t0 = clock64();
            while (!mbar_try_wait(&full[s], ph) && clock64() - t0 < kGWaitCycles) {
            }
        }
        if (status != nullptr) atomicExch(status, 1);
    }
}

// The bounded wait on its own: one thread waits, for at most `budget` cycles, on a barrier that
// nothing will ever complete, and reports how the wait ended.
__global__ void bounded_wait_selftest_kernel(long long budget, int* status) {
    __shared__ uint64_t bar;
    __shared__ int err;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1u);
        err = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool completed = mbar_wait(&bar, 0u, &err, budget);
        *status = completed ? 2 : (err != 0 ? 1 : 3);   // 1: gave up after the budget and raised the error word
    }
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder (a host-side function of the process, not of a device).
EncodeTiledFn encode_tiled() {
    static std::atomic<void*> cached{nullptr};
    void* fn = cached.load(std::memory_order_acquire);
    if (fn == nullptr) {
        cudaDriverEntryPointQueryResult found;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &found) != cudaSuccess ||
            found != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        cached.store(fn, std::memory_order_release);
    }
    return reinterpret_cast<EncodeTiledFn>(fn);
}

}  // namespace
}  // namespace mosaic

using namespace mosaic;

extern "C" int mosaic_gram_accumulate(const void* X, int64_t tokens, int64_t cols, int64_t ldx, int dtype, float* G, int64_t ldg,
                                      int flags, int* status_dev, void* stream) {
    if (dtype == MOSAIC_F32) return MOSAIC_ERR_BAD_DTYPE;   // the products must be exact in fp32: bf16 only
    if (dtype != MOSAIC_BF16) return MOSAIC_ERR_BAD_DTYPE;
    if (tokens < 0 || cols <= 0 || ldx < cols) return MOSAIC_ERR_INVALID_ARG;
    if (tokens > 0) {   // without tokens X is never read and may be NULL
        const int rc = check_matrix(X, tokens, cols, ldx, dtype);
        if (rc != MOSAIC_OK) return rc;
    }
    if ((cols % 8) != 0 || tokens > 0x7FFFFFFF - kGTok || cols > 0x7FFFFFFF - kGBlk || ldg < cols) return MOSAIC_ERR_INVALID_ARG;
    if (G == nullptr) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(G) & 15u) != 0 || (ldg % 4) != 0 || (reinterpret_cast<uintptr_t>(status_dev) & 3u) != 0)
        return MOSAIC_ERR_MISALIGNED;
    {   // G must not overlap X
        const char *a = static_cast<const char*>(X), *b = reinterpret_cast<const char*>(G);
        const size_t xs = tokens > 0 ? ((size_t)(tokens - 1) * (size_t)ldx + (size_t)cols) * 2u : 0u;   // 0: no overlap possible
        const size_t gs = ((size_t)(cols - 1) * (size_t)ldg + (size_t)cols) * 4u;
        if (a < b + gs && b < a + xs) return MOSAIC_ERR_ALIASING;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool reset = (flags & MOSAIC_RESET_ACCUM) != 0;
    if (status_dev != nullptr) MOSAIC_CUDA_TRY(cudaMemsetAsync(status_dev, 0, sizeof(int), st));
    if (tokens == 0) {
        if (reset) MOSAIC_CUDA_TRY(cudaMemset2DAsync(G, (size_t)ldg * 4u, 0, (size_t)cols * 4u, (size_t)cols, st));
        return MOSAIC_OK;
    }
    EncodeTiledFn encode = encode_tiled();
    if (encode == nullptr) return MOSAIC_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)tokens};
    const cuuint64_t gstride[1] = {(cuuint64_t)ldx * 2u};
    const cuuint32_t box[2] = {(cuuint32_t)kGBoxCols, (cuuint32_t)kGTok};
    const cuuint32_t estride[2] = {1u, 1u};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2u, const_cast<void*>(X), gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return MOSAIC_ERR_CUDA;
    static DeviceCache opted;   // the shared-memory opt-in belongs to one device's copy of the kernel
    const int ok = opted.get([&]() -> int {
        if (cudaFuncSetAttribute(gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGSmemBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return -1;
        }
        return 1;
    });
    if (ok < 0) return MOSAIC_ERR_CUDA;
    const int n_blk = (int)((cols + kGBlk - 1) / kGBlk);
    const int64_t n_tiles = (int64_t)n_blk * (n_blk + 1) / 2;
    if (n_tiles > 0x7FFFFFFF) return MOSAIC_ERR_INVALID_ARG;
    const int grid = (int)(n_tiles < sm_count() ? n_tiles : sm_count());
    gram_kernel<<<grid, kGThreads, kGSmemBytes, st>>>(map, G, ldg, (int)cols, (int)tokens, n_blk, (int)n_tiles, reset ? 1 : 0, status_dev);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}

extern "C" int mosaic_bounded_wait_selftest(int64_t budget_cycles, int* status_dev, void* stream) {
    if (status_dev == nullptr) return MOSAIC_ERR_NULL_PTR;
    if ((reinterpret_cast<uintptr_t>(status_dev) & 3u) != 0) return MOSAIC_ERR_MISALIGNED;
    if (budget_cycles < 1 || budget_cycles > 2000000000ll) return MOSAIC_ERR_INVALID_ARG;   // at most about a second
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MOSAIC_CUDA_TRY(cudaMemsetAsync(status_dev, 0, sizeof(int), st));
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>((long long)budget_cycles, status_dev);
    MOSAIC_LAUNCH_CHECK();
    return MOSAIC_OK;
}
