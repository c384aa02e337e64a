// hora_group_advantage: GRPO / RLOO advantages over ragged (CSR) groups (Sec. 3.1; RLOO paragraph of Sec. 4).
//
// A warp takes 32 consecutive groups at a time; lane i reads group i's two offsets (one coalesced load)
// and owns that group's statistics, so the per-group scalar work (mean, variance, square root,
// reciprocal — fp64) is done once per group by one lane.  The rewards of those groups are one contiguous
// run of memory.  As many whole groups as fit 1536 elements form a batch; a lane loads the batch as up to
// twelve 16-byte pieces (all in flight together: that is what hides DRAM latency here) and KEEPS them in
// registers, 128 elements of the batch per "row" of the warp, regardless of where the group boundaries fall:
//   statistics  per row four ballots (which rewards are 1.0) give every lane the number of ones before its
//               four elements; that count and the lane's own four bits go to shared memory as one word,
//               so lane i gets its group's number of ones from two lookups, at its start and end offsets.
//               A group of 0/1 rewards (the verifiable-reward case) is finished there: sum = k,
//               sum (r - m)^2 = k (n - k) / n exactly, and its two possible advantages — of a 0 and of a 1 —
//               are computed once, in fp64, rounded to fp32 once.
//   output      a bitmap of group starts with running counts maps every element to its group; the element
//               picks one of its group's two values; 16-byte stores.
// If any reward of the batch is neither 0.0 nor 1.0 the batch takes the general route instead: the rows go
// to a shared-memory slab, each group is summed in fp64 by the whole warp (fixed butterfly), its squared
// deviations taken in a second sweep (the two-pass form), and every element evaluated as
// adv = (r - mean) * scale in fp64, scale = 1 / (std + eps) for GRPO, n / (n - 1) for RLOO
// (r - (S - r)/(n-1) = (r - S/n) n/(n-1)); for a 0/1 group both routes perform the same operations.
// A group longer than a batch is streamed from global memory (same arithmetic).
// r - mean is exactly zero for a constant group (partial sums k*r are exact in fp64), so such groups
// get exactly zero.  Every order of operations is fixed: results are bitwise reproducible.
#include "hora_group_stats.cuh"

namespace hora {

constexpr int kAdvWarps = 8;
constexpr int kRows = 12;                                     // 128-element rows a batch may span
constexpr int kSlab = kRows * 128;                            // 1536 elements
constexpr unsigned kOne = 0x3F800000u;                        // bit pattern of 1.0f

struct __align__(16) AdvWarpSmem {
    float buf[kSlab];                                         // general route only
    unsigned int pre[kSlab / 4 + 4];                          // per 4 elements: (ones before them << 4) | their own bits
    unsigned int starts[kSlab / 32];                          // one bit per element: a non-empty group starts here
    int cum_starts[kSlab / 32];                               // exclusive running counts per word
    float2 two[kWarp];                                        // per non-empty group, in order: advantage of a 0, of a 1
    double mean[kWarp], scale[kWarp];                         // per non-empty group, in order (general route)
};
constexpr size_t kAdvSmem = sizeof(AdvWarpSmem) * kAdvWarps;

__device__ __forceinline__ int64_t shfl_i64(int64_t v, int src) { return __shfl_sync(kFull, v, src); }

// One group streamed from global memory by the whole warp (groups longer than a batch).
__device__ void advantage_streamed(const float *__restrict__ rewards, int64_t s, int64_t e, int32_t mode, double eps,
                                   int32_t ddof, float *__restrict__ adv, int lane) {
    double mean, scale;
    group_mean_scale(rewards, s, e, mode, eps, ddof, lane, mean, scale);
    for (int64_t j = s + lane; j < e; j += kWarp) adv[j] = (float)(((double)__ldg(rewards + j) - mean) * scale);
}

// exclusive running count over words of popc(word[c]); words beyond n_words count as empty
__device__ __forceinline__ void running_counts(const unsigned int *word, int *cum, int n_words, int lane) {
    int carry = 0;
    for (int c0 = 0; c0 < n_words; c0 += kWarp) {
        const int c = c0 + lane;
        const int v = c < n_words ? __popc(word[c]) : 0;
        int inc = v;
#pragma unroll
        for (int d = 1; d < kWarp; d <<= 1) {
            const int t = __shfl_up_sync(kFull, inc, d);
            if (lane >= d) inc += t;
        }
        if (c < n_words) cum[c] = carry + inc - v;
        carry += __shfl_sync(kFull, inc, kWarp - 1);
    }
}

// ones among elements [0, pos) of the batch, from the packed prefix words
__device__ __forceinline__ int ones_before(const unsigned int *pre, int pos) {
    const unsigned w = pre[pos >> 2];
    return (int)(w >> 4) + __popc(w & ((1u << (pos & 3)) - 1u));
}

// VEC4: rewards and adv are 16-byte aligned, so a batch is read and written in 16-byte pieces starting at
// the 4-element boundary at or below its first element.
template <bool VEC4>
__global__ void __launch_bounds__(kAdvWarps *kWarp, 2)
group_advantage_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ off, int64_t N, int32_t mode,
                       double eps, int32_t ddof, float *__restrict__ adv, int32_t *status_dev) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    AdvWarpSmem &sm = reinterpret_cast<AdvWarpSmem *>(s_raw)[threadIdx.x >> 5];
    const int lane = lane_id();
    const unsigned lt = (1u << lane) - 1u;
    const int64_t warp0 = (int64_t)blockIdx.x * kAdvWarps + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * kAdvWarps;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    const int64_t n_all = __ldg(off + N);                     // nothing is read at or beyond this element
    for (int64_t blk = warp0; blk < n_blocks; blk += stride) {
        const int64_t g0 = blk * kWarp;
        const int ng = (int)((N - g0 < kWarp) ? N - g0 : kWarp);
        int64_t my_s = 0, my_e = 0;
        if (lane < ng) {
            my_s = __ldg(off + g0 + lane);
            my_e = __ldg(off + g0 + lane + 1);
        }
        if (my_e < my_s || my_s < 0 || my_e > n_all) {
            raise_status(status_dev, HORA_ERR_INVALID_VALUE);
            my_e = my_s = 0;                                  // treat as empty: nothing is read or written for it
        }
        const int64_t my_n = my_e - my_s;
        int done = 0;
        while (done < ng) {
            // ---- how many whole groups, starting at `done`, fit a batch ----
            const int64_t base = shfl_i64(my_s, done);
            const int64_t start = VEC4 ? (base & ~(int64_t)3) : base;
            const int64_t rel_end = my_e - start;             // meaningful for lanes >= done
            const bool fits = lane >= done && lane < ng && my_s >= base && rel_end >= 0 && rel_end <= kSlab;
            const unsigned fit_mask = __ballot_sync(kFull, fits) >> done;
            const int nfit = (fit_mask == kFull) ? kWarp : __ffs(~fit_mask) - 1;
            if (nfit == 0) {                                  // group `done` alone is longer than a batch
                const int64_t s = shfl_i64(my_s, done), e = shfl_i64(my_e, done);
                if (e > s) advantage_streamed(rewards, s, e, mode, eps, ddof, adv, lane);
                ++done;
                continue;
            }
            const int last = done + nfit - 1;
            const bool mine = lane >= done && lane <= last;   // this lane's group is part of the batch
            const int span = (int)shfl_i64(rel_end, last);    // the batch is elements [lead, span) counted from `start`
            const int lead = (int)(base - start);
            if (span == lead) { done += nfit; continue; }     // only empty groups
            const int my_rs = mine ? (int)(my_s - start) : 0, my_re = mine ? (int)rel_end : 0;
            const int n_rows = (span + 127) >> 7;
            // ---- load: every piece of the batch in flight at once, then held in registers ----
            float4 v[kRows];
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                v[j] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                const int e0 = 128 * j + 4 * lane;
                if (j < n_rows && e0 < span) {
                    const int64_t e = start + e0;
                    if (VEC4 && e + 4 <= n_all) {
                        v[j] = __ldg(reinterpret_cast<const float4 *>(rewards + e));
                    } else {
                        if (e < n_all) v[j].x = __ldg(rewards + e);
                        if (e + 1 < n_all) v[j].y = __ldg(rewards + e + 1);
                        if (e + 2 < n_all) v[j].z = __ldg(rewards + e + 2);
                        if (e + 3 < n_all) v[j].w = __ldg(rewards + e + 3);
                    }
                }
            }
            // ---- which rewards are 1.0 (packed prefix words); is anything neither 0.0 nor 1.0? ----
            unsigned other = 0;
            int carry = 0;
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                if (j < n_rows) {
                    const unsigned ux = __float_as_uint(v[j].x), uy = __float_as_uint(v[j].y);
                    const unsigned uz = __float_as_uint(v[j].z), uw = __float_as_uint(v[j].w);
                    other |= min(ux, ux ^ kOne) | min(uy, uy ^ kOne) | min(uz, uz ^ kOne) | min(uw, uw ^ kOne);
                    const unsigned bx = __ballot_sync(kFull, ux == kOne), by = __ballot_sync(kFull, uy == kOne);
                    const unsigned bz = __ballot_sync(kFull, uz == kOne), bw = __ballot_sync(kFull, uw == kOne);
                    const int before = carry + __popc(bx & lt) + __popc(by & lt) + __popc(bz & lt) + __popc(bw & lt);
                    const unsigned own = (ux == kOne ? 1u : 0u) | (uy == kOne ? 2u : 0u) | (uz == kOne ? 4u : 0u) |
                                         (uw == kOne ? 8u : 0u);
                    sm.pre[32 * j + lane] = ((unsigned)before << 4) | own;
                    carry += __popc(bx) + __popc(by) + __popc(bz) + __popc(bw);
                }
            }
            if (lane == 0) sm.pre[32 * n_rows] = (unsigned)carry << 4;
            const bool general = __any_sync(kFull, other != 0u);
            // ---- group starts (non-empty groups only: they have distinct starts) and their order ----
            for (int w = lane; w < kSlab / 32; w += kWarp) sm.starts[w] = 0u;
            __syncwarp();
            const bool nonempty = mine && my_re > my_rs;
            if (nonempty) atomicOr(&sm.starts[my_rs >> 5], 1u << (my_rs & 31));
            const int my_rank = __popc(__ballot_sync(kFull, nonempty) & lt);
            __syncwarp();
            running_counts(sm.starts, sm.cum_starts, n_rows * 4, lane);
            __syncwarp();
            const double dn = (double)my_n;
            if (!general) {
                // ---- per-group statistics (lane i: group i), exact for 0/1 rewards ----
                const double k = (double)(ones_before(sm.pre, my_re) - ones_before(sm.pre, my_rs));
                const double mean = my_n > 0 ? k / dn : 0.0;
                const double ss = k * (dn - k) / (my_n > 0 ? dn : 1.0);
                const double scale = group_scale(mode, ss, my_n, ddof, eps);
                if (nonempty) sm.two[my_rank] = make_float2((float)((0.0 - mean) * scale), (float)((1.0 - mean) * scale));
                __syncwarp();
                // ---- output: element -> group through the start bitmap ----
#pragma unroll
                for (int j = 0; j < kRows; ++j) {
                    const int e0 = 128 * j + 4 * lane;
                    if (j < n_rows && e0 < span) {
                        const int bit = e0 & 31;
                        const unsigned sw = sm.starts[e0 >> 5];
                        const int r0 = sm.cum_starts[e0 >> 5] + __popc(sw & (0xFFFFFFFFu >> (31 - bit))) - 1;
                        const int r1 = r0 + (int)((sw >> (bit + 1)) & 1u);
                        const int r2 = r1 + (int)((sw >> (bit + 2)) & 1u);
                        const int r3 = r2 + (int)((sw >> (bit + 3)) & 1u);
                        // rank -1: an element before the batch's first group, loaded but never stored
                        const float2 a0 = sm.two[max(r0, 0)], a1 = sm.two[max(r1, 0)], a2 = sm.two[max(r2, 0)],
                                     a3 = sm.two[r3];
                        float4 o;
                        o.x = __float_as_uint(v[j].x) == kOne ? a0.y : a0.x;
                        o.y = __float_as_uint(v[j].y) == kOne ? a1.y : a1.x;
                        o.z = __float_as_uint(v[j].z) == kOne ? a2.y : a2.x;
                        o.w = __float_as_uint(v[j].w) == kOne ? a3.y : a3.x;
                        float *dst = adv + start + e0;
                        if (VEC4 && e0 >= lead && e0 + 4 <= span) {
                            *reinterpret_cast<float4 *>(dst) = o;
                        } else {
                            if (e0 >= lead && e0 < span) dst[0] = o.x;
                            if (e0 + 1 >= lead && e0 + 1 < span) dst[1] = o.y;
                            if (e0 + 2 >= lead && e0 + 2 < span) dst[2] = o.z;
                            if (e0 + 3 >= lead && e0 + 3 < span) dst[3] = o.w;
                        }
                    }
                }
            } else {
                // ---- general route: rows to the slab, whole-warp two-pass sums per group ----
#pragma unroll
                for (int j = 0; j < kRows; ++j)
                    if (j < n_rows) *reinterpret_cast<float4 *>(&sm.buf[128 * j + 4 * lane]) = v[j];
                __syncwarp();
                double my_mean = 0.0, my_ss = 0.0;
                for (int i = done; i <= last; ++i) {
                    const int s = __shfl_sync(kFull, my_rs, i), e = __shfl_sync(kFull, my_re, i);
                    if (e <= s) continue;
                    double part = 0.0;
                    for (int j = s + lane; j < e; j += kWarp) part += (double)sm.buf[j];
                    const double mean = warp_sum(part) / (double)(e - s);
                    double ss = 0.0;
                    if (mode == HORA_ADV_GRPO) {
                        double sq = 0.0;
                        for (int j = s + lane; j < e; j += kWarp) {
                            const double d = (double)sm.buf[j] - mean;
                            sq += d * d;
                        }
                        ss = warp_sum(sq);
                    }
                    if (lane == i) { my_mean = mean; my_ss = ss; }
                }
                if (nonempty) {
                    sm.mean[my_rank] = my_mean;
                    sm.scale[my_rank] = group_scale(mode, my_ss, my_n, ddof, eps);
                }
                __syncwarp();
#pragma unroll
                for (int j = 0; j < kRows; ++j) {
                    const int e0 = 128 * j + 4 * lane;
                    if (j < n_rows && e0 < span) {
                        const float val[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int el = e0 + q;
                            if (el >= lead && el < span) {
                                const int r = sm.cum_starts[el >> 5] +
                                              __popc(sm.starts[el >> 5] & (0xFFFFFFFFu >> (31 - (el & 31)))) - 1;
                                adv[start + el] = (float)(((double)val[q] - sm.mean[r]) * sm.scale[r]);
                            }
                        }
                    }
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
    const bool vec4 = ((reinterpret_cast<uintptr_t>(rewards) | reinterpret_cast<uintptr_t>(adv)) & 15u) == 0;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    const int grid = clamp_grid((n_blocks + kAdvWarps - 1) / kAdvWarps, 2);
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAdvSmem);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kAdvWarps * kWarp, kAdvSmem, static_cast<cudaStream_t>(stream)>>>(rewards, group_offsets, N, mode,
                                                                                         (double)eps, ddof, adv, status_dev);
        return cudaSuccess;
    };
    if ((vec4 ? go(group_advantage_kernel<true>) : go(group_advantage_kernel<false>)) != cudaSuccess) return HORA_ERR_CUDA;
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
