// hora_group_advantage: GRPO / RLOO advantages over ragged (CSR) groups (Sec. 3.1; RLOO paragraph of Sec. 4).
//
// A warp takes 32 consecutive groups at a time.  Lane i reads group i's two offsets (one coalesced
// load) and ends up owning that group's statistics, so the per-group scalar work (mean, variance,
// square root, reciprocal — all fp64) is done once per group by one lane instead of 32 times by a
// whole warp; fp64 throughput, not memory, was the limit otherwise.  The elements of each group are
// visited by the whole warp, coalesced:
//   pass A   count and sum.  Rewards that are all 0 or 1 (the verifiable-reward case) are counted
//            with ballots and never touch the fp64 pipe; any other group is summed in fp64 by a
//            fixed butterfly, and its squared deviations about the mean in a second sweep
//            (the two-pass form).  For a 0/1 group sum (r - m)^2 = k (n - k) / n exactly.
//   pass C   adv = (r - mean) * scale, rounded to fp32 once.  scale = 1 / (std + eps) for GRPO and
//            n / (n - 1) for RLOO (r - (S - r)/(n-1) = (r - S/n) n/(n-1)).
// r - mean is exactly zero for a constant group (partial sums k*r are exact in fp64), so such groups
// get exactly zero.  Every order of operations is fixed: results are bitwise reproducible.
#include "hora_common.cuh"

namespace hora {

constexpr int kAdvWarps = 8;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
    return v;
}

__device__ __forceinline__ int64_t shfl_i64(int64_t v, int src) { return __shfl_sync(kFull, v, src); }

__global__ void __launch_bounds__(kAdvWarps *kWarp)
group_advantage_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ off, int64_t N, int32_t mode,
                       double eps, int32_t ddof, float *__restrict__ adv, int32_t *status_dev) {
    const int lane = lane_id();
    const int64_t warp0 = (int64_t)blockIdx.x * kAdvWarps + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * kAdvWarps;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    for (int64_t blk = warp0; blk < n_blocks; blk += stride) {
        const int64_t g0 = blk * kWarp;
        const int ng = (int)((N - g0 < kWarp) ? N - g0 : kWarp);
        int64_t my_s = 0, my_e = 0;
        if (lane < ng) {
            my_s = __ldg(off + g0 + lane);
            my_e = __ldg(off + g0 + lane + 1);
        }
        if (my_e < my_s || my_s < 0) {
            raise_status(status_dev, HORA_ERR_INVALID_VALUE);
            my_e = my_s = 0;                            // skip the group; nothing is read or written for it
        }
        const int64_t my_n = my_e - my_s;
        // ---- pass A: per-group sum (lane i keeps group i's) ----
        double my_sum = 0.0;
        unsigned binary_mask = 0;                       // bit i: group i holds only 0.0 / 1.0
        for (int i = 0; i < ng; ++i) {
            const int64_t s = shfl_i64(my_s, i), e = shfl_i64(my_e, i);
            int k = 0;
            bool bin = true;
            for (int64_t j0 = s; j0 < e; j0 += kWarp) {
                const int64_t j = j0 + lane;
                const bool in = j < e;
                const float v = in ? __ldg(rewards + j) : 0.0f;
                const unsigned m1 = __ballot_sync(kFull, in && v == 1.0f);
                const unsigned mz = __ballot_sync(kFull, v == 0.0f);
                k += __popc(m1);
                bin = bin && ((m1 | mz) == kFull);
            }
            double sum = (double)k;
            if (!bin) {
                double part = 0.0;
                for (int64_t j = s + lane; j < e; j += kWarp) part += (double)__ldg(rewards + j);
                sum = warp_sum(part);
            }
            if (lane == i) my_sum = sum;
            if (bin) binary_mask |= 1u << i;
        }
        const double dn = (double)my_n;
        const double my_mean = my_n > 0 ? my_sum / dn : 0.0;
        double my_scale;
        if (mode == HORA_ADV_RLOO) {
            my_scale = my_n > 1 ? dn / (double)(my_n - 1) : 0.0;
        } else {
            // ---- squared deviations: closed form for 0/1 groups, a second sweep for the others ----
            double my_ss = my_sum * (dn - my_sum) / (my_n > 0 ? dn : 1.0);
            unsigned general = ~binary_mask & (ng == kWarp ? kFull : ((1u << ng) - 1u));
            while (general) {
                const int i = __ffs(general) - 1;
                general &= general - 1;
                const int64_t s = shfl_i64(my_s, i), e = shfl_i64(my_e, i);
                const double mean = __shfl_sync(kFull, my_mean, i);
                double sq = 0.0;
                for (int64_t j = s + lane; j < e; j += kWarp) {
                    const double d = (double)__ldg(rewards + j) - mean;
                    sq += d * d;
                }
                const double ss = warp_sum(sq);
                if (lane == i) my_ss = ss;
            }
            const double var = (my_n - ddof > 0) ? my_ss / (double)(my_n - ddof) : 0.0;
            const double den = sqrt(var) + eps;
            my_scale = den > 0.0 ? 1.0 / den : 0.0;
        }
        // ---- pass C: write ----
        for (int i = 0; i < ng; ++i) {
            const int64_t s = shfl_i64(my_s, i), e = shfl_i64(my_e, i);
            const double mean = __shfl_sync(kFull, my_mean, i);
            const double scale = __shfl_sync(kFull, my_scale, i);
            if ((binary_mask >> i) & 1u) {              // two possible outputs: pick, no per-element fp64
                const float a0 = (float)((0.0 - mean) * scale), a1 = (float)((1.0 - mean) * scale);
                for (int64_t j = s + lane; j < e; j += kWarp) adv[j] = (__ldg(rewards + j) != 0.0f) ? a1 : a0;
            } else {
                for (int64_t j = s + lane; j < e; j += kWarp)
                    adv[j] = (float)(((double)__ldg(rewards + j) - mean) * scale);
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
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    const int grid = clamp_grid((n_blocks + kAdvWarps - 1) / kAdvWarps, 8);
    group_advantage_kernel<<<grid, kAdvWarps * kWarp, 0, static_cast<cudaStream_t>(stream)>>>(
        rewards, group_offsets, N, mode, (double)eps, ddof, adv, status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
