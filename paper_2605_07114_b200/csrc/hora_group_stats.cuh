// Group statistics shared by the advantage kernels (Sec. 3.1; RLOO paragraph of Sec. 4): mean and scale of one
// group, adv = (r - mean) * scale with scale = 1/(std + eps) for GRPO and n/(n - 1) for RLOO.
#pragma once
#include "hora_common.cuh"

namespace hora {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
    return v;
}

// scale of one group from its statistics (run by the lane that owns the group)
__device__ __forceinline__ double group_scale(int32_t mode, double ss, int64_t n, int32_t ddof, double eps) {
    if (mode == HORA_ADV_RLOO) return n > 1 ? (double)n / (double)(n - 1) : 0.0;
    const double var = (n - ddof > 0) ? ss / (double)(n - ddof) : 0.0;
    const double den = sqrt(var) + eps;
    return den > 0.0 ? 1.0 / den : 0.0;
}

// Mean and scale of the group rewards[s, e), e > s, read from global memory by the whole warp (two-pass form,
// fp64, fixed butterfly order).  Every lane returns the same values.
__device__ __forceinline__ void group_mean_scale(const float *__restrict__ rewards, int64_t s, int64_t e, int32_t mode,
                                                 double eps, int32_t ddof, int lane, double &mean, double &scale) {
    const int64_t n = e - s;
    double part = 0.0;
    for (int64_t j = s + lane; j < e; j += kWarp) part += (double)__ldg(rewards + j);
    const double sum = warp_sum(part);
    mean = sum / (double)n;
    double ss = 0.0;
    if (mode == HORA_ADV_GRPO) {
        double sq = 0.0;
        for (int64_t j = s + lane; j < e; j += kWarp) {
            const double d = (double)__ldg(rewards + j) - mean;
            sq += d * d;
        }
        ss = warp_sum(sq);
    }
    scale = group_scale(mode, ss, n, ddof, eps);
}

}  // namespace hora
