// hora_group_advantage: GRPO / RLOO advantages over ragged (CSR) groups (Sec. 3.1; RLOO paragraph of Sec. 4).
//
// One warp owns one group.  Groups of up to 32*kRegs rewards (every group the allocator can produce
// with ld <= 256 and G0 <= 32) are held in registers: one coalesced read, two butterfly reductions in
// fp64 (sum, then squared deviations about the mean — the two-pass form), one coalesced write.
// Longer groups stream from global memory three times (the repeats hit L1/L2).  The butterfly
// (xor-shuffle) order is fixed, so results are bitwise reproducible and identical on every lane.
#include "hora_common.cuh"

namespace hora {

constexpr int kAdvWarps = 8;
constexpr int kRegs = 9;   // 9 * 32 = 288 >= 32 + 256

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
    return v;
}

__global__ void __launch_bounds__(kAdvWarps *kWarp)
group_advantage_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ off, int64_t N, int32_t mode,
                       double eps, int32_t ddof, float *__restrict__ adv, int32_t *status_dev) {
    const int lane = lane_id();
    const int64_t warp0 = (int64_t)blockIdx.x * kAdvWarps + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * kAdvWarps;
    for (int64_t g = warp0; g < N; g += stride) {
        const int64_t s = __ldg(off + g), e = __ldg(off + g + 1);
        const int64_t n = e - s;
        if (n < 0 || s < 0) {
            if (lane == 0) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
            continue;
        }
        if (n == 0) continue;
        const double dn = (double)n;
        if (n <= kRegs * kWarp) {
            float v[kRegs];
            double part = 0.0;
#pragma unroll
            for (int q = 0; q < kRegs; ++q) {
                const int64_t j = s + q * kWarp + lane;
                v[q] = (j < e) ? __ldg(rewards + j) : 0.0f;
                part += (double)v[q];
            }
            const double sum = warp_sum(part);
            if (mode == HORA_ADV_GRPO) {
                const double mean = sum / dn;
                double sq = 0.0;
#pragma unroll
                for (int q = 0; q < kRegs; ++q) {
                    const double d = (double)v[q] - mean;
                    if (s + q * kWarp + lane < e) sq += d * d;
                }
                const double ss = warp_sum(sq);
                const double var = (n - ddof > 0) ? ss / (double)(n - ddof) : 0.0;
                const double den = sqrt(var) + eps;
                const double inv = den > 0.0 ? 1.0 / den : 0.0;
#pragma unroll
                for (int q = 0; q < kRegs; ++q) {
                    const int64_t j = s + q * kWarp + lane;
                    if (j < e) adv[j] = (float)(((double)v[q] - mean) * inv);
                }
            } else {
                const double inv = n > 1 ? 1.0 / (double)(n - 1) : 0.0;
#pragma unroll
                for (int q = 0; q < kRegs; ++q) {
                    const int64_t j = s + q * kWarp + lane;
                    // = r - (S - r)/(n-1); n*r - S is exactly 0 for a constant group
                    if (j < e) adv[j] = (float)((dn * (double)v[q] - sum) * inv);
                }
            }
        } else {
            double part = 0.0;
            for (int64_t j = s + lane; j < e; j += kWarp) part += (double)__ldg(rewards + j);
            const double sum = warp_sum(part);
            if (mode == HORA_ADV_GRPO) {
                const double mean = sum / dn;
                double sq = 0.0;
                for (int64_t j = s + lane; j < e; j += kWarp) {
                    const double d = (double)__ldg(rewards + j) - mean;
                    sq += d * d;
                }
                const double ss = warp_sum(sq);
                const double var = (n - ddof > 0) ? ss / (double)(n - ddof) : 0.0;
                const double den = sqrt(var) + eps;
                const double inv = den > 0.0 ? 1.0 / den : 0.0;
                for (int64_t j = s + lane; j < e; j += kWarp) adv[j] = (float)(((double)__ldg(rewards + j) - mean) * inv);
            } else {
                const double inv = 1.0 / (double)(n - 1);
                for (int64_t j = s + lane; j < e; j += kWarp) {
                    const double r = (double)__ldg(rewards + j);
                    adv[j] = (float)((dn * r - sum) * inv);
                }
            }
        }
    }
}

}  // namespace hora

extern "C" hora_status_t hora_group_advantage(const float *rewards, const int64_t *group_offsets, int64_t N,
                                              int32_t mode, float eps, int32_t ddof, float *adv, int32_t *status_dev,
                                              void *stream) {
    using namespace hora;
    if (N < 0 || (mode != HORA_ADV_GRPO && mode != HORA_ADV_RLOO) || (ddof != 0 && ddof != 1) || !(eps >= 0.0f))
        return HORA_ERR_INVALID_ARG;
    if (N == 0) return HORA_OK;
    if (group_offsets == nullptr || rewards == nullptr || adv == nullptr) return HORA_ERR_INVALID_ARG;
    const int grid = clamp_grid((N + kAdvWarps - 1) / kAdvWarps, 8);
    group_advantage_kernel<<<grid, kAdvWarps * kWarp, 0, static_cast<cudaStream_t>(stream)>>>(
        rewards, group_offsets, N, mode, (double)eps, ddof, adv, status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
