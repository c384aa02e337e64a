// hora_group_advantage: GRPO / RLOO advantages over ragged (CSR) groups (Sec. 3.1; RLOO paragraph of Sec. 4).
//
// A warp takes 32 consecutive groups at a time; lane i reads group i's two offsets (one coalesced load)
// and owns that group's statistics, so the per-group scalar work (mean, variance, square root,
// reciprocal — fp64) is done once per group by one lane.  The rewards of those groups are one contiguous
// run of memory.  As many whole groups as fit 1536 elements form a batch, staged in a per-warp shared-memory
// slab by asynchronous 16-byte copies (up to twelve per lane, all in flight together: that is what hides DRAM
// latency here) and handled in "rows" of 128 elements, a lane four consecutive elements of each row,
// regardless of where the group boundaries fall:
//   statistics  a warp scan (shared by four rows, one byte each) gives every lane the number of ones before
//               its four elements; that count and the lane's own four bits go to shared memory as one word,
//               so lane i gets its group's number of ones from two lookups, at its start and end offsets.
//               A group of 0/1 rewards (the verifiable-reward case) is finished there: sum = k,
//               sum (r - m)^2 = k (n - k) / n exactly, and its two possible advantages — of a 0 and of a 1 —
//               are computed once, in fp64, rounded to fp32 once.
//   output      a bitmap of group starts with running counts maps every element to its group; the element
//               picks one of its group's two values; 16-byte stores.
// If any reward of the batch is neither 0.0 nor 1.0 the batch takes the general route instead: each group
// is summed in fp64 by a sub-warp of 4, 8 or 32 lanes (fixed butterfly), its squared
// deviations taken in a second sweep (the two-pass form), and every element evaluated as
// adv = (r - mean) * scale in fp64, scale = 1 / (std + eps) for GRPO, n / (n - 1) for RLOO
// (r - (S - r)/(n-1) = (r - S/n) n/(n-1)); for a 0/1 group both routes perform the same operations.
// A group longer than a batch is streamed from global memory (same arithmetic).
// r - mean is exactly zero for a constant group (partial sums k*r are exact in fp64), so such groups
// get exactly zero.  Every order of operations is fixed: results are bitwise reproducible.
#define HORA_FILE_ID 3
#include "hora_checked.cuh"
#include "hora_group_stats.cuh"

HORA_CHECKED_REGISTER()

namespace hora {

constexpr int kAdvWarps = 8;
constexpr int kRows = 12;                                     // 128-element rows a batch may span
constexpr int kSlab = kRows * 128;                            // 1536 elements

struct __align__(16) AdvWarpSmem {
    float buf[kSlab];                                         // the staged batch
    unsigned int pre[kSlab / 4 + 4];                          // per 4 elements: (ones before them << 4) | their own bits
    unsigned int starts[kSlab / 32];                          // one bit per element: a non-empty group starts here
    int cum_starts[kSlab / 32];                               // exclusive running counts per word
    float2 two[kWarp];                                        // per non-empty group, in order: advantage of a 0, of a 1
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
    const unsigned w = HORA_AT(pre, pos >> 2, kSlab / 4 + 4);
    return (int)(w >> 4) + __popc(w & ((1u << (pos & 3)) - 1u));
}

// Asynchronous 16-byte global -> shared copy (the data does not pass through registers or L1).
__device__ __forceinline__ void cp_async_16(float *smem_dst, const float *gmem_src) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// group (in the order of the batch's non-empty groups) of element el, through the start bitmap
__device__ __forceinline__ int rank_of(const AdvWarpSmem &sm, int el) {
    return sm.cum_starts[el >> 5] + __popc(sm.starts[el >> 5] & (0xFFFFFFFFu >> (31 - (el & 31)))) - 1;
}

// General rewards, one staged batch: groups done .. last of the warp's 32 (lane g owns group g; my_rs, my_re are
// its bounds inside the slab).  The warp is split into sub-warps of W lanes and a sub-warp walks one group, W
// elements a step: the sum (hence the mean), then for GRPO the squared deviations (the two-pass form), both in
// fp64 with a fixed butterfly over the W lanes; the lane that owns the group turns them into its scale; a last
// walk replaces every staged reward by (r - mean) * scale.  A whole warp per group, the first form of this route,
// left 27 of 32 lanes idle on groups of five.
template <int W>
__device__ __forceinline__ void general_batch(float *buf, int done, int last, int my_rs, int my_re, int64_t my_n,
                                              int32_t mode, double eps, int32_t ddof, int lane) {
    constexpr int kPer = kWarp / W;                           // groups per pass
    const int sub = lane / W, sl = lane % W;
    const int n_pass = (last - done + kPer) / kPer;
    const bool mine = lane >= done && lane <= last;
    const int my_pass = mine ? (lane - done) / kPer : -1, my_src = mine ? ((lane - done) % kPer) * W : 0;
    double mean_mine = 0.0, ss_mine = 0.0;
    for (int p = 0; p < n_pass; ++p) {
        const int g = done + p * kPer + sub;
        const int s = __shfl_sync(kFull, my_rs, g & 31), e = __shfl_sync(kFull, my_re, g & 31);
        double part = 0.0;
        if (g <= last)
            for (int j = s + sl; j < e; j += W) part += (double)HORA_AT(buf, j, kSlab);
#pragma unroll
        for (int d = 1; d < W; d <<= 1) part += __shfl_xor_sync(kFull, part, d);
        const double mean = e > s ? part / (double)(e - s) : 0.0;
        double sq = 0.0;
        if (mode == HORA_ADV_GRPO) {
            if (g <= last)
                for (int j = s + sl; j < e; j += W) {
                    const double dv = (double)HORA_AT(buf, j, kSlab) - mean;
                    sq += dv * dv;
                }
#pragma unroll
            for (int d = 1; d < W; d <<= 1) sq += __shfl_xor_sync(kFull, sq, d);
        }
        const double tm = __shfl_sync(kFull, mean, my_src), ts = __shfl_sync(kFull, sq, my_src);
        if (p == my_pass) { mean_mine = tm; ss_mine = ts; }
    }
    const double scale_mine = group_scale(mode, ss_mine, my_n, ddof, eps);
    for (int p = 0; p < n_pass; ++p) {
        const int g = done + p * kPer + sub;
        const int s = __shfl_sync(kFull, my_rs, g & 31), e = __shfl_sync(kFull, my_re, g & 31);
        const double M = __shfl_sync(kFull, mean_mine, g & 31), S = __shfl_sync(kFull, scale_mine, g & 31);
        if (g <= last)
            for (int j = s + sl; j < e; j += W) HORA_AT(buf, j, kSlab) = (float)(((double)HORA_AT(buf, j, kSlab) - M) * S);
    }
}

// VEC4: rewards and adv are 16-byte aligned, so a batch is staged and written in 16-byte pieces starting at
// the 4-element boundary at or below its first element.
template <bool VEC4>
__global__ void __launch_bounds__(kAdvWarps *kWarp, 3)
group_advantage_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ off, int64_t N, int32_t mode,
                       double eps, int32_t ddof, float *__restrict__ adv, int32_t *status_dev) {
    pdl_enter();
    extern __shared__ __align__(16) unsigned char s_raw[];
    AdvWarpSmem &sm = reinterpret_cast<AdvWarpSmem *>(s_raw)[threadIdx.x >> 5];
    const int lane = lane_id();
    const unsigned lt = (1u << lane) - 1u;
    const int64_t warp0 = (int64_t)blockIdx.x * kAdvWarps + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * kAdvWarps;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    const int64_t n_all = __ldg(off + N);                     // nothing is read at or beyond this element
    // a lane's two offsets of the warp's NEXT 32 groups are fetched while the current ones are worked on
    auto fetch_offsets = [&](int64_t blk, int64_t &s, int64_t &e) {
        s = e = 0;
        const int64_t g = blk * kWarp + lane;
        if (blk < n_blocks && g < N) {
            s = __ldg(off + g);
            e = __ldg(off + g + 1);
        }
    };
    int64_t nxt_s, nxt_e;
    fetch_offsets(warp0, nxt_s, nxt_e);
    for (int64_t blk = warp0; blk < n_blocks; blk += stride) {
        const int64_t g0 = blk * kWarp;
        const int ng = (int)((N - g0 < kWarp) ? N - g0 : kWarp);
        int64_t my_s = nxt_s, my_e = nxt_e;
        fetch_offsets(blk + stride, nxt_s, nxt_e);
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
            // ---- stage: every piece of the batch in flight at once; pieces past the batch read as zeros ----
            const bool tail = start + 128 * (int64_t)n_rows > n_all;   // the last pieces may cross the end of the array
            if (VEC4 && !tail) {
                const float *src = rewards + start + 4 * lane;
                for (int j = 0; j < n_rows; ++j) {
                    if (128 * j + 4 * lane < span) cp_async_16(&HORA_AT(sm.buf, 128 * j + 4 * lane, kSlab - 3), src + 128 * j);
                    else *reinterpret_cast<float4 *>(&sm.buf[128 * j + 4 * lane]) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                }
                cp_async_wait_all();
            } else {
                for (int j = lane; j < 128 * n_rows; j += kWarp)
                    HORA_AT(sm.buf, j, kSlab) = (j < span && start + j < n_all) ? __ldg(&HORA_AT(rewards, start + j, n_all)) : 0.0f;
            }
            __syncwarp();
            // ---- which rewards are 1.0 (packed prefix words); is anything neither 0.0 nor 1.0? ----
            // A lane takes four consecutive elements of each 128-element row.  Four rows share one warp scan:
            // their per-lane counts (at most 4 each, 128 per row) sit in the four bytes of a word.
            // r (r - 1) is +0.0 exactly for r = 0.0 and r = 1.0 and for nothing else.
            unsigned other = 0;
            int carry = 0;
            for (int j0 = 0; j0 < n_rows; j0 += 4) {
                unsigned own[4], packed = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    own[q] = 0;
                    if (j0 + q < n_rows) {
                        const float4 x = *reinterpret_cast<const float4 *>(&sm.buf[128 * (j0 + q) + 4 * lane]);
                        other |= __float_as_uint(fmaf(x.x, x.x, -x.x)) | __float_as_uint(fmaf(x.y, x.y, -x.y)) |
                                 __float_as_uint(fmaf(x.z, x.z, -x.z)) | __float_as_uint(fmaf(x.w, x.w, -x.w));
                        own[q] = (x.x == 1.0f ? 1u : 0u) | (x.y == 1.0f ? 2u : 0u) | (x.z == 1.0f ? 4u : 0u) |
                                 (x.w == 1.0f ? 8u : 0u);
                    }
                    packed |= (unsigned)__popc(own[q]) << (8 * q);
                }
                unsigned inc = packed;
#pragma unroll
                for (int d = 1; d < kWarp; d <<= 1) {
                    const unsigned t = __shfl_up_sync(kFull, inc, d);
                    if (lane >= d) inc += t;
                }
                const unsigned excl = inc - packed;            // byte-wise: no byte ever borrows
                const unsigned tot = __shfl_sync(kFull, inc, kWarp - 1);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (j0 + q < n_rows)
                        sm.pre[32 * (j0 + q) + lane] = ((unsigned)(carry + (int)((excl >> (8 * q)) & 0xFFu)) << 4) | own[q];
                    carry += (int)((tot >> (8 * q)) & 0xFFu);
                }
            }
            if (lane == 0) sm.pre[32 * n_rows] = (unsigned)carry << 4;
            const bool general = __any_sync(kFull, other != 0u);
            // ---- group starts (non-empty groups only: they have distinct starts) and their order ----
            for (int w = lane; w < 4 * n_rows; w += kWarp) sm.starts[w] = 0u;
            __syncwarp();
            const bool nonempty = mine && my_re > my_rs;
            if (nonempty) atomicOr(&HORA_AT(sm.starts, my_rs >> 5, kSlab / 32), 1u << (my_rs & 31));
            const int my_rank = __popc(__ballot_sync(kFull, nonempty) & lt);
            __syncwarp();
            running_counts(sm.starts, sm.cum_starts, 4 * n_rows, lane);
            __syncwarp();
            const double dn = (double)my_n;
            if (!general) {
                // ---- per-group statistics (lane i: group i), exact for 0/1 rewards ----
                const double k = (double)(ones_before(sm.pre, my_re) - ones_before(sm.pre, my_rs));
                const double mean = my_n > 0 ? k / dn : 0.0;
                const double ss = k * (dn - k) / (my_n > 0 ? dn : 1.0);
                const double scale = group_scale(mode, ss, my_n, ddof, eps);
                if (nonempty) HORA_AT(sm.two, my_rank, kWarp) = make_float2((float)((0.0 - mean) * scale), (float)((1.0 - mean) * scale));
                __syncwarp();
                // ---- output: element -> group through the start bitmap; whole 16-byte pieces here ----
                float *dst4 = adv + start + 4 * lane;
                for (int j = 0; j < n_rows; ++j) {
                    const int e0 = 128 * j + 4 * lane;
                    if (VEC4 && e0 >= lead && e0 + 4 <= span) {
                        const float4 x = *reinterpret_cast<const float4 *>(&sm.buf[e0]);
                        const int bit = e0 & 31;
                        const unsigned word = sm.starts[e0 >> 5], sw = word >> bit;
                        const int r0 = sm.cum_starts[e0 >> 5] + __popc(word & (0xFFFFFFFFu >> (31 - bit))) - 1;
                        const int r1 = r0 + (int)((sw >> 1) & 1u);
                        const int r2 = r1 + (int)((sw >> 2) & 1u);
                        const int r3 = r2 + (int)((sw >> 3) & 1u);
                        const float2 a0 = HORA_AT(sm.two, r0, kWarp), a1 = HORA_AT(sm.two, r1, kWarp), a2 = HORA_AT(sm.two, r2, kWarp),
                                     a3 = HORA_AT(sm.two, r3, kWarp);
                        float4 o;
                        o.x = x.x == 1.0f ? a0.y : a0.x;
                        o.y = x.y == 1.0f ? a1.y : a1.x;
                        o.z = x.z == 1.0f ? a2.y : a2.x;
                        o.w = x.w == 1.0f ? a3.y : a3.x;
                        *reinterpret_cast<float4 *>(&HORA_AT(dst4, 128 * j, n_all - start - 4 * lane - 3)) = o;
                    }
                }
                // ragged ends (at most 3 elements after `lead` and 3 before `span`; everything when the pointers
                // are not 16-byte aligned): one element per lane and step
                const int head_end = VEC4 ? min(span, (lead + 3) & ~3) : span;
                const int tail_beg = VEC4 ? max(head_end, span & ~3) : span;
                const int n_rag = (head_end - lead) + (span - tail_beg);
                for (int i = lane; i < n_rag; i += kWarp) {
                    const int el = i < head_end - lead ? lead + i : tail_beg + (i - (head_end - lead));
                    const float2 a = HORA_AT(sm.two, rank_of(sm, el), kWarp);
                    HORA_AT(adv, start + el, n_all) = HORA_AT(sm.buf, el, kSlab) == 1.0f ? a.y : a.x;
                }
            } else {
                // ---- general route: sub-warps of W lanes walk one group each over the slab (W by the batch's mean
                // group size); two walks for the statistics, a third overwrites every reward by its advantage ----
                const int mean_size = (span - lead) / nfit;
                if (mean_size > 48) general_batch<32>(sm.buf, done, last, my_rs, my_re, my_n, mode, eps, ddof, lane);
                else if (mean_size > 10) general_batch<8>(sm.buf, done, last, my_rs, my_re, my_n, mode, eps, ddof, lane);
                else general_batch<4>(sm.buf, done, last, my_rs, my_re, my_n, mode, eps, ddof, lane);
                __syncwarp();
                // the slab leaves in 16-byte pieces, the ragged ends one element per lane and step
                if (VEC4) {
                    float *dst4 = adv + start + 4 * lane;
                    for (int j = 0; j < n_rows; ++j) {
                        const int e0 = 128 * j + 4 * lane;
                        if (e0 >= lead && e0 + 4 <= span)
                            *reinterpret_cast<float4 *>(&HORA_AT(dst4, 128 * j, n_all - start - 4 * lane - 3)) =
                                *reinterpret_cast<const float4 *>(&HORA_AT(sm.buf, e0, kSlab - 3));
                    }
                }
                const int head_end = VEC4 ? min(span, (lead + 3) & ~3) : span;
                const int tail_beg = VEC4 ? max(head_end, span & ~3) : span;
                const int n_rag = (head_end - lead) + (span - tail_beg);
                for (int i = lane; i < n_rag; i += kWarp) {
                    const int el = i < head_end - lead ? lead + i : tail_beg + (i - (head_end - lead));
                    HORA_AT(adv, start + el, n_all) = HORA_AT(sm.buf, el, kSlab);
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
    const int grid = clamp_grid((n_blocks + kAdvWarps - 1) / kAdvWarps, 3);
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAdvSmem);
        if (e != cudaSuccess) return e;
        return launch_pdl(kernel, grid, kAdvWarps * kWarp, kAdvSmem, static_cast<cudaStream_t>(stream), rewards, group_offsets,
                          N, mode, (double)eps, ddof, adv, status_dev);
    };
    if ((vec4 ? go(group_advantage_kernel<true>) : go(group_advantage_kernel<false>)) != cudaSuccess) return HORA_ERR_CUDA;
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
