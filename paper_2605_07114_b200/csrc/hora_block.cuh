// Block-level building blocks shared by the selection kernels: the "last CTA" ticket, block-wide exclusive sums,
// rank location in a histogram (global or shared memory) and the scan of per-block sums.  Every kernel that
// uses them runs kSelThreads threads per CTA.
#pragma once

#include "hora_common.cuh"

namespace hora {

constexpr int kSelThreads = 256;
constexpr int kRowsPerBlock = 1024;          // prompts per CTA in the sum / output kernels (4 per thread)

// "Last CTA" ticket: returns true in exactly one CTA, after every other CTA's global writes are visible.
__device__ __forceinline__ bool last_block(unsigned int *ticket) {
    __shared__ bool s_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (s_last) __threadfence();
    return s_last;
}

// Block-wide exclusive sum over NT values (long long; NT threads per CTA, kSelThreads unless said otherwise), also
// returns the total.
template <int NT = kSelThreads>
__device__ __forceinline__ long long block_exclusive_sum(long long v, long long *total, long long *s_warp) {
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    long long inc = v;
#pragma unroll
    for (int d = 1; d < kWarp; d <<= 1) {
        const long long t = __shfl_up_sync(kFull, inc, d);
        if (lane >= d) inc += t;
    }
    __syncthreads();
    if (lane == kWarp - 1) s_warp[warp] = inc;
    __syncthreads();
    long long base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NT / kWarp; ++w) {
        const long long x = s_warp[w];
        if (w < warp) base += x;
        tot += x;
    }
    *total = tot;
    return base + inc - v;
}

// Two block-wide exclusive sums at once (one pair of barriers instead of two): v0, v1 in, their exclusive
// prefixes in e0, e1, the totals in t0, t1.  s_warp2 holds 2 * (NT / 32) values.
template <int NT = kSelThreads>
__device__ __forceinline__ void block_exclusive_sum2(long long v0, long long v1, long long &e0, long long &e1,
                                                     long long &t0, long long &t1, long long *s_warp2) {
    constexpr int kW = NT / kWarp;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    long long i0 = v0, i1 = v1;
#pragma unroll
    for (int d = 1; d < kWarp; d <<= 1) {
        const long long a = __shfl_up_sync(kFull, i0, d), b = __shfl_up_sync(kFull, i1, d);
        if (lane >= d) { i0 += a; i1 += b; }
    }
    __syncthreads();
    if (lane == kWarp - 1) { s_warp2[warp] = i0; s_warp2[kW + warp] = i1; }
    __syncthreads();
    long long b0 = 0, b1 = 0;
    t0 = t1 = 0;
#pragma unroll
    for (int w = 0; w < kW; ++w) {
        const long long x = s_warp2[w], y = s_warp2[kW + w];
        if (w < warp) { b0 += x; b1 += y; }
        t0 += x;
        t1 += y;
    }
    e0 = b0 + i0 - v0;
    e1 = b1 + i1 - v1;
}

// Run by ONE CTA.  Scanning from the top bin down, find the bin where the running count reaches `need`:
//   count(bins above d) < need <= count(bins above d) + count(d).
// Returns d (or -1 if need is out of range) to every thread, with the count above d in *above_out and the
// count of d in *count_out.  `bins` is a power of two and `hist` 16-byte aligned.  Two stages, neither of
// which walks memory serially (a dependent chain of 32 loads from L2 cost 16 us here): every thread sums a
// contiguous run of `per` bins, fetched by independent 16-byte loads that are all issued before the first
// is used, and a block scan picks the run that holds the crossing; then the first warp loads that run's
// bins one per lane (`per` <= 32) and a warp scan pins the bin.
__device__ inline int locate_rank(const unsigned long long *hist, int bins, long long need, long long *above_out,
                           long long *count_out, long long *s_warp) {
    __shared__ long long s_found[3];                        // top bin of the run, count above the run, found flag
    const int per = (bins + kSelThreads - 1) / kSelThreads; // 1, or an even number <= 32 for bins <= 8192
    const int top = bins - 1 - (int)threadIdx.x * per;      // this thread's run: bins top, top-1, ..., top-per+1
    long long local = 0;
    if (per == 1) {
        if (top >= 0) local = (long long)__ldcg(hist + top);
    } else {                                                // bins == kSelThreads * per: every run is complete
        const ulonglong2 *run = reinterpret_cast<const ulonglong2 *>(hist + (top - per + 1));
        const int nvec = per >> 1;
        ulonglong2 v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = u < nvec ? __ldcg(run + u) : make_ulonglong2(0ull, 0ull);
#pragma unroll
        for (int u = 0; u < 16; ++u) local += (long long)(v[u].x + v[u].y);
    }
    if (threadIdx.x == 0) s_found[2] = 0;
    long long total;
    const long long above = block_exclusive_sum(local, &total, s_warp);
    if (need >= 1 && above < need && need <= above + local) {
        s_found[0] = top;
        s_found[1] = above;
        s_found[2] = 1;
    }
    __syncthreads();
    int digit = -1;
    const bool found = s_found[2] != 0;
    const int run_top = (int)s_found[0];
    const long long run_above = s_found[1];
    __syncthreads();                                        // everyone has read the run before it is overwritten
    if (found) {
        if (threadIdx.x < kWarp) {
            const int lane = threadIdx.x;
            const int bin = run_top - lane;
            const long long cnt = (lane < per && bin >= 0) ? (long long)__ldcg(hist + bin) : 0;
            long long inc = cnt;
#pragma unroll
            for (int d = 1; d < kWarp; d <<= 1) {
                const long long t = __shfl_up_sync(kFull, inc, d);
                if (lane >= d) inc += t;
            }
            const bool here = run_above + inc - cnt < need && need <= run_above + inc;
            if (here) {
                s_found[0] = bin;
                s_found[1] = run_above + inc - cnt;
                s_found[2] = cnt;
            }
        }
        __syncthreads();
        digit = (int)s_found[0];
        *above_out = s_found[1];
        *count_out = s_found[2];
    }
    __syncthreads();
    return digit;
}

// Digit search over a histogram in SHARED memory, run by one CTA: the bin where the count from the top
// reaches `need`.  s_pick receives (digit, count above it, count of it); digit -1 if need is out of range.
__device__ __forceinline__ void locate_rank_shared(const unsigned int *s_hist, int bins, long long need, long long *s_warp,
                                                   long long *s_pick) {
    const int per = (bins + kSelThreads - 1) / kSelThreads;      // thread t owns bins top, top-1, ..., top-per+1
    const int top = bins - 1 - (int)threadIdx.x * per;
    long long local = 0;
    for (int j = 0; j < per; ++j)
        if (top - j >= 0) local += s_hist[top - j];
    if (threadIdx.x == 0) s_pick[0] = -1;
    long long total;
    const long long above = block_exclusive_sum(local, &total, s_warp);
    if (need >= 1 && above < need && need <= above + local) {    // at most one thread: the crossing is in its run
        long long run = above;
        for (int j = 0; j < per; ++j) {
            const long long cnt = s_hist[top - j];
            if (need <= run + cnt) {
                s_pick[0] = top - j;
                s_pick[1] = run;
                s_pick[2] = cnt;
                break;
            }
            run += cnt;
        }
    }
    __syncthreads();
}

// Exclusive scan of the block sums (plus, in list mode, the corrections held in shared memory for blocks
// [b0, b0 + n_here)), kSelThreads * 4 entries per step, in index order; run by one CTA.  s_warp holds
// 2 * (kSelThreads / 32) values.
__device__ inline void scan_block_sums(long long *bsum_hi, long long *bsum_t, int64_t b0, int64_t n_here,
                                const unsigned int *s_fix_hi, const unsigned int *s_fix_t, long long &run_hi,
                                long long &run_t, long long *s_warp) {
    constexpr int kRun = 4;                                      // consecutive block sums per thread
    for (int64_t c0 = 0; c0 < n_here; c0 += kRun * kSelThreads) {
        const int64_t c = c0 + (int64_t)threadIdx.x * kRun;
        long long vh[kRun], vt[kRun], sh = 0, st = 0;
#pragma unroll
        for (int u = 0; u < kRun; ++u) {
            const bool in = c + u < n_here;
            vh[u] = in ? __ldcg(bsum_hi + b0 + c + u) + (s_fix_hi ? (long long)s_fix_hi[c + u] : 0) : 0;
            vt[u] = in ? __ldcg(bsum_t + b0 + c + u) + (s_fix_t ? (long long)s_fix_t[c + u] : 0) : 0;
        }
#pragma unroll
        for (int u = 0; u < kRun; ++u) { sh += vh[u]; st += vt[u]; }
        long long th, tt, eh, et;
        block_exclusive_sum2(sh, st, eh, et, th, tt, s_warp);
        eh += run_hi;
        et += run_t;
#pragma unroll
        for (int u = 0; u < kRun; ++u) {
            if (c + u < n_here) { bsum_hi[b0 + c + u] = eh; bsum_t[b0 + c + u] = et; }
            eh += vh[u];
            et += vt[u];
        }
        run_hi += th;
        run_t += tt;
    }
}

// U_i(Delta) from the row's own entry: the product in U_i(Delta) = 1 - prod_{j<Delta} (b+j)/(a+b+j) is
// g_i(Delta) (b + Delta - 1) / a  (Eq. marginal), so one load replaces Delta multiplications.  Every operation
// is pinned to one rounding so that the value does not depend on which kernel evaluates it.
__device__ __forceinline__ double utility_from_gain(double g, double a, double b, int32_t Delta) {
    return __dsub_rn(1.0, __ddiv_rn(__dmul_rn(g, __dadd_rn(b, (double)(Delta - 1))), a));
}

}  // namespace hora
