// Shared device/host helpers of the Mosaic pruning kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/mosaic.h"

namespace mosaic {

constexpr int kVec = 8;  // elements handled per thread per access: 16 B of bf16, 2 x 16 B of fp32

// ---------------------------------------------------------------- host side
int sm_count();                        // SMs of the current device (148 if it cannot be queried)
int current_device();                  // index of the current device, or -1 if it cannot be queried

// One small non-zero integer remembered per device (occupancy of a kernel, "attribute set"):
// function attributes and occupancy belong to one device's copy of a kernel, so a process that
// drives several GPUs needs them once per device, not once per process.  get() runs `compute`
// with the device current the first time that device asks; two host threads that race both
// compute the same value.  A device index beyond the table is computed every time.
constexpr int kMaxDevices = 64;
class DeviceCache {
    std::atomic<int> v_[kMaxDevices];   // static storage: starts at zero = "not computed yet"
public:
    template <class F>
    int get(F compute) {
        const int dev = current_device();
        if (dev < 0 || dev >= kMaxDevices) return compute();
        int x = v_[dev].load(std::memory_order_acquire);
        if (x == 0) {
            x = compute();
            v_[dev].store(x, std::memory_order_release);
        }
        return x;
    }
};
int check_matrix(const void* p, int64_t rows, int64_t cols, int64_t ld, int dtype);
inline size_t elem_size(int dtype) { return dtype == MOSAIC_F32 ? 4 : 2; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? MOSAIC_OK : MOSAIC_ERR_CUDA; }

#define MOSAIC_CUDA_TRY(expr)                                   \
    do {                                                        \
        cudaError_t e__ = (expr);                               \
        if (e__ != cudaSuccess) return MOSAIC_ERR_CUDA;         \
    } while (0)

#define MOSAIC_LAUNCH_CHECK()                                   \
    do {                                                        \
        cudaError_t e__ = cudaGetLastError();                   \
        if (e__ != cudaSuccess) return MOSAIC_ERR_CUDA;         \
    } while (0)

// ---------------------------------------------------------------- device side
#ifdef __CUDACC__

// Streaming 16-byte global load that does not pollute L1.
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// Read-only variant (data never written during the kernel).
__device__ __forceinline__ uint4 ld_stream16_ro(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream16(void* p, uint4 v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// Eight consecutive matrix elements as raw bits.
template <int DT> struct Raw8;
template <> struct Raw8<MOSAIC_BF16> {
    uint32_t w[4];  // element 2i = low half of w[i]
    static constexpr int kBytes = 16;
    template <bool RO> __device__ __forceinline__ void load(const void* p) {
        uint4 v = RO ? ld_stream16_ro(p) : ld_stream16(p);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    }
    __device__ __forceinline__ void store(void* p) const { st_stream16(p, make_uint4(w[0], w[1], w[2], w[3])); }
    __device__ __forceinline__ void clear() { w[0] = w[1] = w[2] = w[3] = 0u; }
    // |element e| as fp32 (exact widening, sign cleared)
    __device__ __forceinline__ float abs_f32(int e) const {
        uint32_t x = w[e >> 1];
        return __uint_as_float((e & 1) ? (x & 0x7FFF0000u) : ((x << 16) & 0x7FFFFFFFu));
    }
    __device__ __forceinline__ float f32(int e) const {
        uint32_t x = w[e >> 1];
        return __uint_as_float((e & 1) ? (x & 0xFFFF0000u) : (x << 16));
    }
    __device__ __forceinline__ void zero(int e) { w[e >> 1] &= (e & 1) ? 0x0000FFFFu : 0xFFFF0000u; }
    __device__ __forceinline__ void set_scalar(int e, const void* base, int64_t idx) {
        uint32_t b = reinterpret_cast<const uint16_t*>(base)[idx];
        w[e >> 1] = (e & 1) ? ((w[e >> 1] & 0x0000FFFFu) | (b << 16)) : ((w[e >> 1] & 0xFFFF0000u) | b);
    }
    __device__ __forceinline__ void put_scalar(int e, void* base, int64_t idx) const {
        reinterpret_cast<uint16_t*>(base)[idx] = (uint16_t)((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu));
    }
};
template <> struct Raw8<MOSAIC_F32> {
    uint32_t w[8];
    static constexpr int kBytes = 32;
    template <bool RO> __device__ __forceinline__ void load(const void* p) {
        uint4 a = RO ? ld_stream16_ro(p) : ld_stream16(p);
        uint4 b = RO ? ld_stream16_ro((const char*)p + 16) : ld_stream16((const char*)p + 16);
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
        w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
    }
    __device__ __forceinline__ void store(void* p) const {
        st_stream16(p, make_uint4(w[0], w[1], w[2], w[3]));
        st_stream16((char*)p + 16, make_uint4(w[4], w[5], w[6], w[7]));
    }
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = 0u;
    }
    __device__ __forceinline__ float abs_f32(int e) const { return __uint_as_float(w[e] & 0x7FFFFFFFu); }
    __device__ __forceinline__ float f32(int e) const { return __uint_as_float(w[e]); }
    __device__ __forceinline__ void zero(int e) { w[e] = 0u; }
    __device__ __forceinline__ void set_scalar(int e, const void* base, int64_t idx) {
        w[e] = reinterpret_cast<const uint32_t*>(base)[idx];
    }
    __device__ __forceinline__ void put_scalar(int e, void* base, int64_t idx) const {
        reinterpret_cast<uint32_t*>(base)[idx] = w[e];
    }
};

// Load the 8 elements starting at column c of a row (row_base = first element of
// the row); columns >= cols are left as zero bits.  Full vectors use 16-byte loads.
template <int DT, bool RO>
__device__ __forceinline__ void load_vec(Raw8<DT>& r, const void* mat, int64_t row_off, int64_t c, int64_t cols) {
    constexpr int esz = (DT == MOSAIC_F32) ? 4 : 2;
    if (c + kVec <= cols) {
        r.template load<RO>((const char*)mat + (row_off + c) * esz);
    } else {
        r.clear();
#pragma unroll
        for (int e = 0; e < kVec; ++e)
            if (c + e < cols) r.set_scalar(e, mat, row_off + c + e);
    }
}

// Deterministic fp64 warp sum (fixed butterfly).
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Deterministic fp64 block sum; result valid in thread 0.  `sm` holds >= 32 doubles.
__device__ __forceinline__ double block_sum(double v, double* sm) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    __syncthreads();
    if (lane == 0) sm[wid] = v;
    __syncthreads();
    double s = 0.0;
    if (threadIdx.x == 0)
        for (int i = 0; i < nw; ++i) s += sm[i];
    return s;
}

#endif  // __CUDACC__
}  // namespace mosaic
