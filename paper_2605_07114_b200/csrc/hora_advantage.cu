// hora_group_advantage: GRPO / RLOO advantages over ragged (CSR) groups (Sec. 3.1; RLOO paragraph of Sec. 4).
//
// A warp takes 32 consecutive groups at a time.  Lane i reads group i's two offsets (one coalesced
// load) and ends up owning that group's statistics, so the per-group scalar work (mean, variance,
// square root, reciprocal — all fp64) is done once per group by one lane instead of 32 times by a
// whole warp; fp64 throughput, not memory, was the limit otherwise.
//
// The rewards of those 32 groups are one contiguous run of memory.  As many whole groups as fit the
// warp's shared-memory slab (kSlab floats) are staged with independent coalesced loads — all in flight
// together, which is what hides DRAM latency here — processed in place, and streamed back out:
//   pass A   count and sum.  Rewards that are all 0 or 1 (the verifiable-reward case) are counted
//            with ballots and never touch the fp64 pipe; any other group is summed in fp64 by a
//            fixed butterfly, and its squared deviations about the mean in a second sweep
//            (the two-pass form).  For a 0/1 group sum (r - m)^2 = k (n - k) / n exactly.
//   pass C   adv = (r - mean) * scale, rounded to fp32 once.  scale = 1 / (std + eps) for GRPO and
//            n / (n - 1) for RLOO (r - (S - r)/(n-1) = (r - S/n) n/(n-1)).
// A group longer than the slab is streamed from global memory instead (same arithmetic).
// r - mean is exactly zero for a constant group (partial sums k*r are exact in fp64), so such groups
// get exactly zero.  Every order of operations is fixed: results are bitwise reproducible.
#include "hora_common.cuh"

namespace hora {

constexpr int kAdvWarps = 8;
constexpr int kSlab = 2048;                                   // floats per warp
constexpr size_t kAdvSmem = (size_t)kAdvWarps * kSlab * sizeof(float);

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
    return v;
}

__device__ __forceinline__ int64_t shfl_i64(int64_t v, int src) { return __shfl_sync(kFull, v, src); }

// scale of one group from its statistics (run by the lane that owns the group)
__device__ __forceinline__ double group_scale(int32_t mode, double ss, int64_t n, int32_t ddof, double eps) {
    if (mode == HORA_ADV_RLOO) return n > 1 ? (double)n / (double)(n - 1) : 0.0;
    const double var = (n - ddof > 0) ? ss / (double)(n - ddof) : 0.0;
    const double den = sqrt(var) + eps;
    return den > 0.0 ? 1.0 / den : 0.0;
}

// One group streamed from global memory by the whole warp (groups longer than the slab).
__device__ void advantage_streamed(const float *__restrict__ rewards, int64_t s, int64_t e, int32_t mode, double eps,
                                   int32_t ddof, float *__restrict__ adv, int lane) {
    const int64_t n = e - s;
    double part = 0.0;
    for (int64_t j = s + lane; j < e; j += kWarp) part += (double)__ldg(rewards + j);
    const double sum = warp_sum(part);
    const double mean = sum / (double)n;
    double ss = 0.0;
    if (mode == HORA_ADV_GRPO) {
        double sq = 0.0;
        for (int64_t j = s + lane; j < e; j += kWarp) {
            const double d = (double)__ldg(rewards + j) - mean;
            sq += d * d;
        }
        ss = warp_sum(sq);
    }
    const double scale = group_scale(mode, ss, n, ddof, eps);
    for (int64_t j = s + lane; j < e; j += kWarp) adv[j] = (float)(((double)__ldg(rewards + j) - mean) * scale);
}

__global__ void __launch_bounds__(kAdvWarps *kWarp)
group_advantage_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ off, int64_t N, int32_t mode,
                       double eps, int32_t ddof, float *__restrict__ adv, int32_t *status_dev) {
    extern __shared__ float s_slab[];
    const int lane = lane_id();
    float *buf = s_slab + (threadIdx.x >> 5) * kSlab;
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
            my_e = my_s;                                      // treat as empty: nothing is read or written for it
        }
        const int64_t my_n = my_e - my_s;
        int done = 0;
        while (done < ng) {
            // ---- how many whole groups, starting at `done`, fit the slab ----
            const int64_t base = shfl_i64(my_s, done);
            const int64_t rel_end = my_e - base;              // meaningful for lanes >= done
            const bool fits = lane >= done && lane < ng && my_s >= base && rel_end >= 0 && rel_end <= kSlab;
            const unsigned fit_mask = __ballot_sync(kFull, fits) >> done;
            const int nfit = (fit_mask == kFull) ? kWarp : __ffs(~fit_mask) - 1;
            if (nfit == 0) {                                  // group `done` alone is longer than the slab
                const int64_t s = shfl_i64(my_s, done), e = shfl_i64(my_e, done);
                if (e > s) advantage_streamed(rewards, s, e, mode, eps, ddof, adv, lane);
                ++done;
                continue;
            }
            const int last = done + nfit - 1;
            const int total = (int)shfl_i64(rel_end, last);
            const int32_t my_rs = (int32_t)(my_s - base), my_re = (int32_t)rel_end;   // slab-relative, lanes done..last
            // ---- stage ----
            for (int j = lane; j < total; j += kWarp) buf[j] = __ldg(rewards + base + j);
            __syncwarp();
            // ---- pass A: per-group sum (lane i keeps group i's) ----
            double my_sum = 0.0;
            unsigned binary_mask = 0;                         // bit i: group i holds only 0.0 / 1.0
            for (int i = done; i <= last; ++i) {
                const int s = __shfl_sync(kFull, my_rs, i), e = __shfl_sync(kFull, my_re, i);
                int k = 0;
                bool bin = true;
                for (int j0 = s; j0 < e; j0 += kWarp) {
                    const int j = j0 + lane;
                    const bool in = j < e;
                    const float v = in ? buf[j] : 0.0f;
                    const unsigned m1 = __ballot_sync(kFull, in && v == 1.0f);
                    const unsigned mz = __ballot_sync(kFull, v == 0.0f);
                    k += __popc(m1);
                    bin = bin && ((m1 | mz) == kFull);
                }
                double sum = (double)k;
                if (!bin) {
                    double part = 0.0;
                    for (int j = s + lane; j < e; j += kWarp) part += (double)buf[j];
                    sum = warp_sum(part);
                }
                if (lane == i) my_sum = sum;
                if (bin) binary_mask |= 1u << i;
            }
            const double dn = (double)my_n;
            const double my_mean = my_n > 0 ? my_sum / dn : 0.0;
            double my_ss = my_sum * (dn - my_sum) / (my_n > 0 ? dn : 1.0);   // exact form for 0/1 groups
            if (mode == HORA_ADV_GRPO) {
                const unsigned range = (nfit == kWarp ? kFull : ((1u << nfit) - 1u)) << done;
                unsigned general = ~binary_mask & range;
                while (general) {                             // second sweep for groups with other values
                    const int i = __ffs(general) - 1;
                    general &= general - 1;
                    const int s = __shfl_sync(kFull, my_rs, i), e = __shfl_sync(kFull, my_re, i);
                    const double mean = __shfl_sync(kFull, my_mean, i);
                    double sq = 0.0;
                    for (int j = s + lane; j < e; j += kWarp) {
                        const double d = (double)buf[j] - mean;
                        sq += d * d;
                    }
                    const double ss = warp_sum(sq);
                    if (lane == i) my_ss = ss;
                }
            }
            const double my_scale = group_scale(mode, my_ss, my_n, ddof, eps);
            // ---- pass C: advantages in place ----
            for (int i = done; i <= last; ++i) {
                const int s = __shfl_sync(kFull, my_rs, i), e = __shfl_sync(kFull, my_re, i);
                const double mean = __shfl_sync(kFull, my_mean, i);
                const double scale = __shfl_sync(kFull, my_scale, i);
                if ((binary_mask >> i) & 1u) {                // two possible outputs: pick, no per-element fp64
                    const float a0 = (float)((0.0 - mean) * scale), a1 = (float)((1.0 - mean) * scale);
                    for (int j = s + lane; j < e; j += kWarp) buf[j] = (buf[j] != 0.0f) ? a1 : a0;
                } else {
                    for (int j = s + lane; j < e; j += kWarp) buf[j] = (float)(((double)buf[j] - mean) * scale);
                }
            }
            __syncwarp();
            for (int j = lane; j < total; j += kWarp) adv[base + j] = buf[j];
            __syncwarp();
            done += nfit;
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
    if (cudaFuncSetAttribute(group_advantage_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAdvSmem) !=
        cudaSuccess)
        return HORA_ERR_CUDA;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    const int grid = clamp_grid((n_blocks + kAdvWarps - 1) / kAdvWarps, 3);
    group_advantage_kernel<<<grid, kAdvWarps * kWarp, kAdvSmem, static_cast<cudaStream_t>(stream)>>>(
        rewards, group_offsets, N, mode, (double)eps, ddof, adv, status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
