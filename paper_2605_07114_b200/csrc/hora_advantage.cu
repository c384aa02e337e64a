// hora_group_advantage: GRPO / RLOO advantages over ragged (CSR) groups (Sec. 3.1; RLOO paragraph of Sec. 4).
//
// A warp takes 32 consecutive groups at a time; lane i reads group i's two offsets (one coalesced load)
// and owns that group's statistics, so the per-group scalar work (mean, variance, square root,
// reciprocal — fp64) is done once per group by one lane.  The rewards of those groups are one contiguous
// run of memory.  As many whole groups as fit the warp's shared-memory slab are staged with independent
// coalesced loads (all in flight together: that is what hides DRAM latency here) and then handled FLAT,
// 32 elements per step regardless of where the group boundaries fall:
//   statistics  per 32-element chunk two ballots: which rewards are 1.0, which are neither 0.0 nor 1.0.
//               With their running counts, lane i gets its group's number of ones and of "other" values
//               from two lookups at its start and end offsets.  A group of 0/1 rewards (the verifiable-
//               reward case) is finished there: sum = k, sum (r - m)^2 = k (n - k) / n exactly.  A group with
//               other values is summed in fp64 by the whole warp (fixed butterfly) and its squared
//               deviations taken in a second sweep (the two-pass form).
//   output      a bitmap of group starts with running counts maps every element to its group;
//               adv = (r - mean) * scale, rounded to fp32 once, stored coalesced.
//               scale = 1 / (std + eps) for GRPO, n / (n - 1) for RLOO (r - (S - r)/(n-1) = (r - S/n) n/(n-1)).
// A group longer than the slab is streamed from global memory instead (same arithmetic).
// r - mean is exactly zero for a constant group (partial sums k*r are exact in fp64), so such groups
// get exactly zero.  Every order of operations is fixed: results are bitwise reproducible.
#include "hora_group_stats.cuh"

namespace hora {

constexpr int kAdvWarps = 8;
constexpr int kSlab = 1536;                                   // floats per warp
constexpr int kChunks = kSlab / kWarp;                        // 48

struct AdvWarpSmem {
    float buf[kSlab];
    unsigned int ones[kChunks], other[kChunks], starts[kChunks];        // one bit per element
    int cum_ones[kChunks], cum_other[kChunks], cum_starts[kChunks];     // exclusive running counts per chunk
    double mean[kWarp], scale[kWarp];                                   // per group
    int group_of_rank[kWarp];                                           // r-th non-empty group of the batch
};
constexpr size_t kAdvSmem = sizeof(AdvWarpSmem) * kAdvWarps;

// Asynchronous global -> shared copy of one 4-byte word (the data does not pass through registers).
__device__ __forceinline__ void cp_async_4(float *smem_dst, const float *gmem_src) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ int64_t shfl_i64(int64_t v, int src) { return __shfl_sync(kFull, v, src); }

// One group streamed from global memory by the whole warp (groups longer than the slab).
__device__ void advantage_streamed(const float *__restrict__ rewards, int64_t s, int64_t e, int32_t mode, double eps,
                                   int32_t ddof, float *__restrict__ adv, int lane) {
    double mean, scale;
    group_mean_scale(rewards, s, e, mode, eps, ddof, lane, mean, scale);
    for (int64_t j = s + lane; j < e; j += kWarp) adv[j] = (float)(((double)__ldg(rewards + j) - mean) * scale);
}

// exclusive running count over chunks of popc(word[c]); chunks beyond n_chunks count as empty
__device__ __forceinline__ void running_counts(const unsigned int *word, int *cum, int n_chunks, int lane) {
    int carry = 0;
    for (int c0 = 0; c0 < n_chunks; c0 += kWarp) {
        const int c = c0 + lane;
        const int v = c < n_chunks ? __popc(word[c]) : 0;
        int inc = v;
#pragma unroll
        for (int d = 1; d < kWarp; d <<= 1) {
            const int t = __shfl_up_sync(kFull, inc, d);
            if (lane >= d) inc += t;
        }
        if (c < n_chunks) cum[c] = carry + inc - v;
        carry += __shfl_sync(kFull, inc, kWarp - 1);
    }
}

// number of set bits among elements [0, pos) of a bitmap with running counts
__device__ __forceinline__ int count_before(const unsigned int *word, const int *cum, int pos) {
    if (pos <= 0) return 0;
    const int p = pos - 1;
    return cum[p >> 5] + __popc(word[p >> 5] & (0xFFFFFFFFu >> (31 - (p & 31))));
}

__global__ void __launch_bounds__(kAdvWarps *kWarp)
group_advantage_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ off, int64_t N, int32_t mode,
                       double eps, int32_t ddof, float *__restrict__ adv, int32_t *status_dev) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    AdvWarpSmem &sm = reinterpret_cast<AdvWarpSmem *>(s_raw)[threadIdx.x >> 5];
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
            const bool mine = lane >= done && lane <= last;   // this lane's group is part of the batch
            const int total = (int)shfl_i64(rel_end, last);
            const int my_rs = mine ? (int)(my_s - base) : 0, my_re = mine ? (int)rel_end : 0;
            const int n_chunks = (total + kWarp - 1) / kWarp;
            if (total == 0) { done += nfit; continue; }       // only empty groups
            // ---- stage: asynchronous 4-byte copies, every chunk of the batch in flight at once ----
            for (int c = 0; c < n_chunks; ++c) {
                const int j = c * kWarp + lane;
                if (j < total) cp_async_4(&sm.buf[j], rewards + base + j);
            }
            cp_async_wait_all();
            __syncwarp();
            // ---- per chunk: which rewards are 1.0, which are neither 0.0 nor 1.0 ----
            for (int c = 0; c < n_chunks; ++c) {
                const int j = c * kWarp + lane;
                const float v = j < total ? sm.buf[j] : 0.0f;
                const unsigned w1 = __ballot_sync(kFull, v == 1.0f);
                const unsigned wo = __ballot_sync(kFull, v != 0.0f && v != 1.0f);
                if (lane == 0) { sm.ones[c] = w1; sm.other[c] = wo; sm.starts[c] = 0u; }
            }
            __syncwarp();
            running_counts(sm.ones, sm.cum_ones, n_chunks, lane);
            running_counts(sm.other, sm.cum_other, n_chunks, lane);
            // group starts (non-empty groups only: they have distinct starts) and their order
            const bool nonempty = mine && my_re > my_rs;
            if (nonempty) atomicOr(&sm.starts[my_rs >> 5], 1u << (my_rs & 31));
            const unsigned ne_mask = __ballot_sync(kFull, nonempty);
            if (nonempty) sm.group_of_rank[__popc(ne_mask & ((1u << lane) - 1u))] = lane;
            __syncwarp();
            running_counts(sm.starts, sm.cum_starts, n_chunks, lane);
            __syncwarp();
            // ---- per-group statistics (lane i: group i) ----
            const int k_ones = count_before(sm.ones, sm.cum_ones, my_re) - count_before(sm.ones, sm.cum_ones, my_rs);
            const int k_other = count_before(sm.other, sm.cum_other, my_re) - count_before(sm.other, sm.cum_other, my_rs);
            const double dn = (double)my_n;
            double my_sum = (double)k_ones;
            unsigned general = __ballot_sync(kFull, mine && k_other > 0);   // groups with values other than 0/1
            for (unsigned gm = general; gm; gm &= gm - 1) {
                const int i = __ffs(gm) - 1;
                const int s = __shfl_sync(kFull, my_rs, i), e = __shfl_sync(kFull, my_re, i);
                double part = 0.0;
                for (int j = s + lane; j < e; j += kWarp) part += (double)sm.buf[j];
                const double sum = warp_sum(part);
                if (lane == i) my_sum = sum;
            }
            const double my_mean = my_n > 0 ? my_sum / dn : 0.0;
            double my_ss = my_sum * (dn - my_sum) / (my_n > 0 ? dn : 1.0);   // exact form for 0/1 groups
            if (mode == HORA_ADV_GRPO) {
                for (unsigned gm = general; gm; gm &= gm - 1) {
                    const int i = __ffs(gm) - 1;
                    const int s = __shfl_sync(kFull, my_rs, i), e = __shfl_sync(kFull, my_re, i);
                    const double mean = __shfl_sync(kFull, my_mean, i);
                    double sq = 0.0;
                    for (int j = s + lane; j < e; j += kWarp) {
                        const double d = (double)sm.buf[j] - mean;
                        sq += d * d;
                    }
                    const double ss = warp_sum(sq);
                    if (lane == i) my_ss = ss;
                }
            }
            sm.mean[lane] = my_mean;
            sm.scale[lane] = group_scale(mode, my_ss, my_n, ddof, eps);
            __syncwarp();
            // ---- flat output: element -> group through the start bitmap ----
            for (int c = 0; c < n_chunks; ++c) {
                const int j = c * kWarp + lane;
                if (j < total) {
                    const int rank = sm.cum_starts[c] + __popc(sm.starts[c] & (0xFFFFFFFFu >> (31 - lane))) - 1;
                    const int g = sm.group_of_rank[rank];
                    adv[base + j] = (float)(((double)sm.buf[j] - sm.mean[g]) * sm.scale[g]);
                }
            }
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
