// Host-only entry points and argument validation shared by the device calls.
#include <math.h>

#include <vector>

#include "common.cuh"

namespace mosaic {

int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    return dev;
}

int sm_count() {
    static DeviceCache cached;
    return cached.get([]() -> int {
        int n = 0;
        const int dev = current_device();
        if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = 148;
        }
        return n;
    });
}

int check_matrix(const void* p, int64_t rows, int64_t cols, int64_t ld, int dtype) {
    if (dtype != MOSAIC_F32 && dtype != MOSAIC_BF16) return MOSAIC_ERR_BAD_DTYPE;
    if (rows < 0 || cols <= 0 || ld < cols) return MOSAIC_ERR_INVALID_ARG;
    if (p == nullptr) return MOSAIC_ERR_NULL_PTR;
    const int64_t per16 = 16 / (int64_t)elem_size(dtype);
    if ((reinterpret_cast<uintptr_t>(p) & 15u) != 0 || (ld % per16) != 0) return MOSAIC_ERR_MISALIGNED;
    return MOSAIC_OK;
}

}  // namespace mosaic

extern "C" {

int mosaic_version(void) { return MOSAIC_VERSION; }

const char* mosaic_status_string(int status) {
    switch (status) {
        case MOSAIC_OK: return "ok";
        case MOSAIC_ERR_INVALID_ARG: return "invalid argument";
        case MOSAIC_ERR_NULL_PTR: return "null pointer";
        case MOSAIC_ERR_BAD_DTYPE: return "unsupported dtype";
        case MOSAIC_ERR_MISALIGNED: return "pointer or leading dimension not 16-byte aligned";
        case MOSAIC_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case MOSAIC_ERR_ALIASING: return "input and output overlap";
        case MOSAIC_ERR_CUDA: return "CUDA error";
        case MOSAIC_ERR_NONFINITE: return "non-finite input";
        case MOSAIC_ERR_INFEASIBLE: return "sparsity target clamped";
        case MOSAIC_ERR_TIMEOUT: return "device wait timed out";
        default: return "unknown status";
    }
}

double mosaic_ratio_from_count(int64_t outlier_count, int64_t numel) {
    // projection rank of Algorithm 1: R = O / C * 100
    return 100.0 * (double)outlier_count / (double)numel;
}

// normalize(R_LLM) + Projection Planner; see mosaic.h for the definition.
int mosaic_allocate_sparsity(const int64_t* outlier_counts, const int64_t* numels, const int64_t* cols,
                             int n_layers, int n_proj, double p, double lambda, int mode,
                             double* sparsity_out, int64_t* k_out) {
    if (!outlier_counts || !numels || !cols || !sparsity_out || !k_out) return MOSAIC_ERR_NULL_PTR;
    if (n_layers <= 0 || n_proj <= 0 || !(p >= 0.0 && p < 1.0) || !(lambda >= 0.0)) return MOSAIC_ERR_INVALID_ARG;
    if (mode & ~(MOSAIC_PER_CATEGORY_NORM | MOSAIC_WEIGHTED_MEAN | MOSAIC_REDISTRIBUTE)) return MOSAIC_ERR_INVALID_ARG;
    const bool per_category = (mode & MOSAIC_PER_CATEGORY_NORM) != 0, weighted = (mode & MOSAIC_WEIGHTED_MEAN) != 0;
    const bool redistribute = (mode & MOSAIC_REDISTRIBUTE) != 0;
    const int total = n_layers * n_proj;
    for (int q = 0; q < total; ++q)
        if (numels[q] <= 0 || cols[q] <= 0 || outlier_counts[q] < 0 || outlier_counts[q] > numels[q])
            return MOSAIC_ERR_INVALID_ARG;

    const int n_groups = per_category ? n_proj : 1;
    const int stride = per_category ? n_proj : 1;
    const int members = per_category ? n_layers : total;
    for (int g = 0; g < n_groups; ++g) {
        double lo = 0.0, hi = 0.0;
        for (int c = 0; c < members; ++c) {
            const int q = g + c * stride;
            const double R = mosaic_ratio_from_count(outlier_counts[q], numels[q]);
            if (c == 0 || R < lo) lo = R;
            if (c == 0 || R > hi) hi = R;
        }
        if (hi == lo) {
            for (int c = 0; c < members; ++c) sparsity_out[g + c * stride] = p;
            continue;
        }
        const double range = hi - lo;
        double dsum = 0.0, wsum = 0.0;
        for (int c = 0; c < members; ++c) {
            const int q = g + c * stride;
            const double r = (mosaic_ratio_from_count(outlier_counts[q], numels[q]) - lo) / range;
            const double d = 2.0 * lambda * r;
            const double w = weighted ? (double)numels[q] : 1.0;
            dsum = dsum + w * d;
            wsum = wsum + w;
        }
        const double dbar = dsum / wsum;
        for (int c = 0; c < members; ++c) {
            const int q = g + c * stride;
            const double r = (mosaic_ratio_from_count(outlier_counts[q], numels[q]) - lo) / range;
            const double d = 2.0 * lambda * r;
            sparsity_out[q] = (p + dbar) - d;
        }
    }
    int status = MOSAIC_OK;
    if (redistribute) {
        // Targets that leave [0, 1 - 1/cols] stay on the bound; the others of the group move by one
        // common amount t that brings the (plain or weighted) mean back to p, for as long as the move
        // pushes further targets over a bound.  sparsity_out holds the unclamped targets b_q on entry.
        std::vector<char> fixed((size_t)total, 0);
        std::vector<double> base(sparsity_out, sparsity_out + total);
        for (int g = 0; g < n_groups; ++g) {
            bool any = false;
            for (int c = 0; c < members; ++c) {
                const int q = g + c * stride;
                const double smax = 1.0 - 1.0 / (double)cols[q];
                if (sparsity_out[q] < 0.0 || sparsity_out[q] > smax) any = true;
            }
            if (!any) continue;   // nothing to clamp: the targets stand as they are
            for (int round = 0; round < members; ++round) {
                double wtot = 0.0, wfree = 0.0, sfixed = 0.0, sfree = 0.0;
                for (int c = 0; c < members; ++c) {
                    const int q = g + c * stride;
                    const double w = weighted ? (double)numels[q] : 1.0;
                    wtot = wtot + w;
                    if (fixed[(size_t)q]) sfixed = sfixed + w * sparsity_out[q];
                    else { wfree = wfree + w; sfree = sfree + w * base[(size_t)q]; }
                }
                if (wfree == 0.0) { status = MOSAIC_ERR_INFEASIBLE; break; }   // every target on a bound: p is out of reach
                const double t = (p * wtot - sfixed - sfree) / wfree;
                bool newly = false;
                for (int c = 0; c < members; ++c) {
                    const int q = g + c * stride;
                    if (fixed[(size_t)q]) continue;
                    const double smax = 1.0 - 1.0 / (double)cols[q];
                    const double v = base[(size_t)q] + t;
                    if (v < 0.0) { sparsity_out[q] = 0.0; fixed[(size_t)q] = 1; newly = true; }
                    else if (v > smax) { sparsity_out[q] = smax; fixed[(size_t)q] = 1; newly = true; }
                    else sparsity_out[q] = v;
                }
                if (!newly) break;
            }
        }
        for (int q = 0; q < total; ++q) k_out[q] = (int64_t)floor(sparsity_out[q] * (double)cols[q]);
        return status;
    }
    for (int q = 0; q < total; ++q) {
        const double smax = 1.0 - 1.0 / (double)cols[q];
        if (sparsity_out[q] < 0.0) { sparsity_out[q] = 0.0; status = MOSAIC_ERR_INFEASIBLE; }
        if (sparsity_out[q] > smax) { sparsity_out[q] = smax; status = MOSAIC_ERR_INFEASIBLE; }
        k_out[q] = (int64_t)floor(sparsity_out[q] * (double)cols[q]);
    }
    return status;
}

}  // extern "C"
