// hora_allocate_batched: many small, independent allocation problems in one launch.
//
// The paper runs Phase-B allocation on mini-batches of the training batch (four shards of Gamma/4 = 15
// prompts, each with its own share of the budget; appendix "Training configurations"), and Proposition 1
// holds within each shard.  Here a shard ("segment") is a run of consecutive prompts with its own budget,
// and one CTA solves one segment entirely in shared memory:
//   1  gain rows of the segment's prompts, computed with the arithmetic of hora_gains (same bits), never
//      written to global memory;
//   2  the B_s-th largest key, built two bits a step from the top by one warp: a step is a binary search per sorted
//      row (inside a range that every step narrows) and three warp sums; with at most 32 rows a lane keeps its
//      row's range in registers and the last keys left in the interval are ranked directly;
//   3  per row the number of keys above and equal to the threshold (binary search in the sorted row);
//   4  ties: in prompt order (fp64 equality), or, in exact mode, by exact rational comparison of the at
//      most one candidate per row that lies within 2^-30 of the threshold (pairwise, cross-multiplied);
//   5  Delta, G, the segment's summary.
// Rows longer than 256 candidates are first cut to 256 (a narrow pass; exact unless a row takes them all), and
// only the segments that this does not settle are solved at full width.
// Group offsets over all prompts are an exclusive scan of G by two small kernels afterwards.
#include <algorithm>

#define HORA_FILE_ID 2
#include "hora_block.cuh"
#include "hora_checked.cuh"
#include "hora_common.cuh"
#include "hora_exact.cuh"
#include "hora_gains_chunk.cuh"
#include "hora_rank.cuh"

HORA_CHECKED_REGISTER()

namespace hora {

constexpr int kBThreads = kSelThreads;        // the shared block helpers are written for this many threads
constexpr int kBWarps = kBThreads / kWarp;
constexpr int kBMaxRows = 256;                 // prompts per segment (one thread per prompt in the row phases)
constexpr size_t kBMaxSmem = 200 * 1024;       // keys + bookkeeping must fit this
constexpr int kScanRows = 1024;                // rows per CTA in the offsets scan
constexpr int32_t kBNarrow = 256;              // candidates per row the narrow pass builds (one pass of 32 lanes x 8)

struct BatchedSmemFixed {
    unsigned long long lam_key;
    long long warp_tmp[2 * kBWarps];
    double obj_tmp[kBWarps];
    long long found[3];
    double lam_exact;
    int status;
    int redo;                      // narrow pass: this segment has to go through the full-width pass
};

// Per-prompt arrays of a segment, carved behind the fixed part for the longest segment of the call (so that
// calls with short segments — the paper's 15 prompts — leave shared memory for a fourth CTA per SM).
struct BatchedRows {
    double *a, *b;
    int32_t *cap, *band;           // band: Delta of the row's near-threshold candidate (exact mode), 0 if it has none
    int32_t *lo, *hi;              // selection: the row's count of keys >= the threshold lies in [lo, hi]
    int32_t *cnt2, *cnt3;          // selection: the row's counts for the second and third trial value of a step
    int32_t *capt;                 // the prompt's own cap (cap: what the pass works with, at most its row width)
};
constexpr size_t kBRowBytes = 2 * sizeof(double) + 7 * sizeof(int32_t);   // 44 bytes per prompt

__device__ __forceinline__ BatchedRows carve_rows(unsigned char *base, int rows_cap) {
    BatchedRows r;
    r.a = reinterpret_cast<double *>(base);
    r.b = r.a + rows_cap;
    r.cap = reinterpret_cast<int32_t *>(r.b + rows_cap);
    r.band = r.cap + rows_cap;
    r.lo = r.band + rows_cap;
    r.hi = r.lo + rows_cap;
    r.cnt2 = r.hi + rows_cap;
    r.cnt3 = r.cnt2 + rows_cap;
    r.capt = r.cnt3 + rows_cap;
    return r;
}

struct ScanHeader { unsigned int ticket; unsigned int n_redo; };   // n_redo: segments the narrow pass handed on

__host__ __device__ inline size_t batched_row_stride(int32_t ld) { return (size_t)ld | 1u; }

// Three binary searches in lockstep over keys[lo, hi) of one sorted (non-increasing) row: a_k = first position
// whose key is below t_k, i.e. the number of keys >= t_k given that lo keys are known to be and hi is the most.
__device__ __forceinline__ void search3(const unsigned long long *rk, int lo, int hi, int32_t ld, unsigned long long t1,
                                        unsigned long long t2, unsigned long long t3, int &a1, int &a2, int &a3) {
    int z1 = hi, z2 = hi, z3 = hi;
    a1 = a2 = a3 = lo;
    while (a1 < z1 || a2 < z2 || a3 < z3) {
        const int m1 = (a1 + z1) >> 1, m2 = (a2 + z2) >> 1, m3 = (a3 + z3) >> 1;
        const unsigned long long k1 = HORA_AT(rk, m1 < hi ? m1 : lo, ld), k2 = HORA_AT(rk, m2 < hi ? m2 : lo, ld),
                                 k3 = HORA_AT(rk, m3 < hi ? m3 : lo, ld);
        if (a1 < z1) { if (k1 >= t1) a1 = m1 + 1; else z1 = m1; }
        if (a2 < z2) { if (k2 >= t2) a2 = m2 + 1; else z2 = m2; }
        if (a3 < z3) { if (k3 >= t3) a3 = m3 + 1; else z3 = m3; }
    }
}

// NT threads per CTA: 256, or 128 when no segment of the call has more than 32 prompts.  The selection is a chain of
// dependent steps by one warp, so what an SM gets through is set by how many segments it holds at once: shared
// memory has room for five of the paper's 15-prompt segments, the registers of 256 threads for three CTAs only.
//
// Two passes when rows are longer than 256 candidates.  The NARROW pass (W = 256 < ld, todo == nullptr) builds and
// searches only the first W candidates of every row: half the row passes at ld = 360, and a segment's keys take a
// third less shared memory.  Its answer is the full problem's answer unless some row takes all W of its candidates
// while it has more (its next candidate might belong to the B largest), or the budget exceeds what the narrow rows
// hold; such a segment writes nothing and puts its index on the redo list.  The FULL pass (W = ld) then runs over
// that list (todo, *n_todo) — as a rule it is empty — or, where ld <= 256, over every segment (todo == nullptr).
template <int E, int NT, int PER_SM>
__global__ void __launch_bounds__(NT, PER_SM)
allocate_batched_kernel(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
                        const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                        int32_t ld, int32_t W, const int64_t *__restrict__ seg_off, const int64_t *__restrict__ budgets,
                        int64_t S, const int32_t *__restrict__ todo, const unsigned int *__restrict__ n_todo,
                        int32_t *__restrict__ redo, unsigned int *n_redo, uint32_t flags, int32_t rows_cap,
                        int32_t *__restrict__ delta, int32_t *__restrict__ G, hora_alloc_info *__restrict__ info) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    BatchedSmemFixed &sm = *reinterpret_cast<BatchedSmemFixed *>(s_raw);
    const BatchedRows rw = carve_rows(s_raw + sizeof(BatchedSmemFixed), rows_cap);
    unsigned long long *keys =
        reinterpret_cast<unsigned long long *>(s_raw + sizeof(BatchedSmemFixed) + (size_t)rows_cap * kBRowBytes);
    // Rows sit an odd number of keys apart: the selection has a lane per row probing the same column of many rows
    // at once, and with an even stride (ld = 360: rows 16 banks apart) those probes met in two banks.
    const size_t lds = batched_row_stride(W);
    constexpr int kWarps = NT / kWarp;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    const bool exact = (flags & HORA_FLAG_EXACT_INT) != 0;
    const bool narrow = W < ld;
    const int64_t n_seg = todo != nullptr ? (int64_t)*n_todo : S;
    for (int64_t idx = blockIdx.x; idx < n_seg; idx += gridDim.x) {
        const int64_t s = todo != nullptr ? (int64_t)todo[idx] : idx;
        const int64_t r0 = seg_off[s];
        const int n = (int)(seg_off[s + 1] - r0);
        const long long B = budgets[s];
        __syncthreads();
        if (threadIdx.x == 0) { sm.status = (B < 0) ? HORA_ERR_INVALID_VALUE : HORA_OK; sm.redo = 0; }
        __syncthreads();
        // ---- 1: gain rows into shared memory (a warp per row) ----
        Posterior nxt = warp < n ? load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, r0 + warp) : Posterior{};
        for (int r = warp; r < n; r += kWarps) {
            const Posterior p = nxt;                          // the next row's inputs are fetched while this row is built
            if (r + kWarps < n) nxt = load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, r0 + r + kWarps);
            if (!p.ok && lane == 0) sm.status = HORA_ERR_INVALID_VALUE;
            const double a = p.ok ? p.a : 1.0, b = p.ok ? p.b : 1.0;
            const int32_t ce = p.cap < W ? p.cap : W;          // what this pass builds of the row
            if (lane == 0) { rw.a[r] = a; rw.b[r] = b; rw.cap[r] = ce; rw.capt[r] = p.cap; rw.lo[r] = 0; rw.hi[r] = ce; }
            double carry = 1.0;
            double *out = reinterpret_cast<double *>(keys + (size_t)r * lds);
            for (int32_t k0 = 0; k0 < W; k0 += kWarp * E)
                gains_chunk<E, false, false>(a, b, a + b, ce, W, k0, lane, carry, out, nullptr, nullptr);
        }
        __syncthreads();
        long long sum_cap, sum_built;
        {
            long long e0, e1;
            block_exclusive_sum2<NT>(threadIdx.x < n ? rw.capt[threadIdx.x] : 0, threadIdx.x < n ? rw.cap[threadIdx.x] : 0, e0, e1,
                                     sum_cap, sum_built, sm.warp_tmp);
        }
        if (threadIdx.x == 0 && sm.status == HORA_OK) {
            if (B > sum_cap) sm.status = HORA_ERR_INFEASIBLE;
            else if (B > sum_built) sm.redo = 1;               // (narrow pass only: the budget reaches past its rows)
        }
        __syncthreads();
        const bool run = sm.status == HORA_OK && sm.redo == 0 && B > 0;   // the same in every thread
        // ---- 2: the B-th largest key, by warp 0 ----
        // The key is built from its top bits down, two bits a step: with p the bits so far, the three trial values
        // p | 1, p | 2, p | 3 (at the step's position) are counted at once — how many keys are >= each — and the
        // largest one that still has B keys at or above it gives the two bits.  A lane owns rows lane, lane + 32,
        // ...; a row is sorted, so a count is one binary search, and it can only move inside [lo, hi], which every
        // step narrows from both sides: after a few steps a search is a probe or two.  The bits that all keys share
        // (the sign, most of the exponent) are taken from the largest and the smallest key directly.
        // With at most 32 rows a lane owns ONE row and keeps its range in registers, and the steps stop as soon as no
        // row has more than one key left in the interval the bits describe (some ten steps of thirty): the keys
        // left, at most one a lane, are ranked directly.
        if (warp == 0 && run) {
            const bool small = n <= kWarp;
            unsigned long long kmax = 0ull, kmin = ~0ull;
            for (int r = lane; r < n; r += kWarp) {
                const int cp = rw.cap[r];
                if (cp > 0) {
                    const unsigned long long first = keys[(size_t)r * lds], last_k = keys[(size_t)r * lds + cp - 1];
                    kmax = first > kmax ? first : kmax;
                    kmin = last_k < kmin ? last_k : kmin;
                }
            }
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                const unsigned long long a = __shfl_xor_sync(kFull, kmax, d), z = __shfl_xor_sync(kFull, kmin, d);
                kmax = a > kmax ? a : kmax;
                kmin = z < kmin ? z : kmin;
            }
            // bits above `top` are the same in every key (B <= the number of keys, so the threshold is one of them)
            int top = 63 - __clzll((long long)((kmax ^ kmin) | 1ull));
            top |= 1;                                          // steps take bits (top, top - 1), ..., (1, 0)
            unsigned long long prefix = top >= 63 ? 0ull : (kmax >> (top + 1)) << (top + 1);
            const unsigned long long *my_rk = keys + (size_t)(lane < n ? lane : 0) * lds;
            int my_lo = 0, my_hi = (small && lane < n) ? rw.cap[lane] : 0;
            bool wide = true;                                  // some row still has more than one key in the interval
#pragma unroll 1
            for (int bit = top; bit >= 1 && wide; bit -= 2) {
                const unsigned long long t1 = prefix | (1ull << (bit - 1)), t2 = prefix | (2ull << (bit - 1)),
                                         t3 = prefix | (3ull << (bit - 1));
                int c1 = 0, c2 = 0, c3 = 0, m1 = 0, m2 = 0, m3 = 0;
                if (small) {
                    search3(my_rk, my_lo, my_hi, W, t1, t2, t3, m1, m2, m3);
                    c1 = m1; c2 = m2; c3 = m3;
                } else {
#pragma unroll 1
                    for (int r = lane; r < n; r += kWarp) {
                        int a1, a2, a3;
                        search3(keys + (size_t)r * lds, rw.lo[r], rw.hi[r], W, t1, t2, t3, a1, a2, a3);
                        c1 += a1; c2 += a2; c3 += a3;
                        rw.band[r] = a1;                       // (scratch until the tie step)
                        rw.cnt2[r] = a2;
                        rw.cnt3[r] = a3;
                    }
                }
                c1 = __reduce_add_sync(kFull, c1);            // at most 22528 keys in a segment
                c2 = __reduce_add_sync(kFull, c2);
                c3 = __reduce_add_sync(kFull, c3);
                // counts decrease with the trial value: take the largest trial that still has B keys at or above it
                const int pick = (long long)c3 >= B ? 3 : ((long long)c2 >= B ? 2 : ((long long)c1 >= B ? 1 : 0));
                prefix |= (unsigned long long)pick << (bit - 1);
                // #keys >= threshold lies between the count of the next larger trial and that of the picked one
                if (small) {
                    if (pick == 3) my_hi = m3;
                    else if (pick == 2) { my_lo = m3; my_hi = m2; }
                    else if (pick == 1) { my_lo = m2; my_hi = m1; }
                    else my_lo = m1;
                    wide = __any_sync(kFull, my_hi - my_lo > 1);
                } else {
#pragma unroll 1
                    for (int r = lane; r < n; r += kWarp) {
                        const int a1 = rw.band[r], a2 = rw.cnt2[r], a3 = rw.cnt3[r];
                        if (pick == 3) rw.hi[r] = a3;
                        else if (pick == 2) { rw.lo[r] = a3; rw.hi[r] = a2; }
                        else if (pick == 1) { rw.lo[r] = a2; rw.hi[r] = a1; }
                        else rw.lo[r] = a1;
                    }
                }
            }
            if (!wide) {
                // keys at or above the interval: sum of lo; the threshold is the need-th largest of the keys left
                const long long need = B - (long long)__reduce_add_sync(kFull, my_lo);
                const bool has = my_hi > my_lo;
                const unsigned long long mine = has ? my_rk[my_lo] : 0ull;
                int gt = 0, ge = 0;
                for (int j = 0; j < n; ++j) {
                    const unsigned long long other = __shfl_sync(kFull, mine, j);
                    const bool other_has = __shfl_sync(kFull, (int)has, j) != 0;
                    gt += other_has && other > mine;
                    ge += other_has && other >= mine;
                }
                const unsigned hit = __ballot_sync(kFull, has && gt < need && need <= ge);
                // (B keys exist and fewer than B lie above the interval, so some key qualifies; equal keys agree)
                prefix = __shfl_sync(kFull, mine, hit ? __ffs(hit) - 1 : 0);
                if (hit == 0u && lane == 0) sm.status = HORA_ERR_INTERNAL;
            }
            if (small && lane < n) { rw.lo[lane] = my_lo; rw.hi[lane] = my_hi; }   // where the count pass starts from
            if (lane == 0) sm.lam_key = prefix;
        }
        __syncthreads();
        const unsigned long long prefix = sm.lam_key;
        const unsigned long long lam_key = prefix;
        // ---- 3: per row, keys above and equal to the threshold ----
        int my_hi = 0, my_tied = 0, my_cap = 0;
        const unsigned long long *row = keys + (size_t)threadIdx.x * lds;
        if (threadIdx.x < n && run) {
            my_cap = rw.cap[threadIdx.x];
            // the selection left the row's range: keys before lo are above the threshold, keys from hi on below it
            int lo = rw.lo[threadIdx.x], hi = rw.hi[threadIdx.x];
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (HORA_AT(row, mid, W) > lam_key) lo = mid + 1; else hi = mid;
            }
            my_hi = lo;
            while (my_hi + my_tied < my_cap && HORA_AT(row, my_hi + my_tied, W) == lam_key) ++my_tied;
            // narrow pass: the row takes every candidate this pass built and has more: the full pass decides
            if (narrow && my_hi + my_tied >= W && rw.capt[threadIdx.x] > W) sm.redo = 1;
        }
        // ---- 4: ties ----
        int my_delta = 0;
        long long n_above = 0, n_tied = 0, n_taken = 0;
        double lambda = B > 0 ? __longlong_as_double((long long)lam_key) : 0.0;
        if (!exact) {
            long long tot_hi, tot_t;
            block_exclusive_sum<NT>(my_hi, &tot_hi, sm.warp_tmp);
            const long long pre_t = block_exclusive_sum<NT>(my_tied, &tot_t, sm.warp_tmp);
            const long long R = B - tot_hi;
            long long take = R - pre_t;
            take = take < 0 ? 0 : (take > my_tied ? my_tied : take);
            my_delta = my_hi + (int)take;
            n_above = tot_hi; n_tied = tot_t; n_taken = R;
        } else {
            // the one candidate of this row, if any, within 2^-30 (relative) of the fp64 threshold
            const double lam = __longlong_as_double((long long)lam_key);
            const unsigned long long k_hi = (unsigned long long)__double_as_longlong(lam * (1.0 + 9.313225746154785e-10));
            const unsigned long long k_lo = (unsigned long long)__double_as_longlong(lam * (1.0 - 9.313225746154785e-10));
            int q = my_hi, has = 0, err = 0;
            if (threadIdx.x < n && run) {
                const double al = alpha ? __ldg(alpha + r0 + threadIdx.x) : alpha0;
                const double be = beta ? __ldg(beta + r0 + threadIdx.x) : beta0;
                if (!(al >= 1.0 && be >= 1.0 && al == floor(al) && be == floor(be))) err = HORA_ERR_NOT_INTEGER;
                else if (al + be + (double)G0 + (double)ld >= 1048576.0) err = HORA_ERR_EXACT_RANGE;
                if (q > 0 && HORA_AT(row, q - 1, W) <= k_hi) {
                    --q;
                    if (q > 0 && HORA_AT(row, q - 1, W) <= k_hi) err = err ? err : HORA_ERR_EXACT_RANGE;
                }
                has = (q < my_cap) && (HORA_AT(row, q, W) >= k_lo);
                if (has && q + 1 < my_cap && HORA_AT(row, q + 1, W) >= k_lo) err = err ? err : HORA_ERR_EXACT_RANGE;
                if (err) atomicCAS(&sm.status, 0, err);
            }
            if ((int)threadIdx.x < rows_cap) rw.band[threadIdx.x] = (threadIdx.x < n && has && !err) ? q + 1 : 0;
            long long tot_q;
            block_exclusive_sum<NT>(q, &tot_q, sm.warp_tmp);           // has a barrier: band is visible after it
            const long long Rp = B - tot_q;                        // rollouts to hand out inside the band
            int better = 0, equal = 0;
            if (threadIdx.x < n && rw.band[threadIdx.x] && sm.status == HORA_OK) {
                // exact rank of this row's candidate among the band candidates: equal types need no arithmetic,
                // different ones are compared as exact fractions
                const unsigned long long a_t = (unsigned long long)rw.a[threadIdx.x], b_t = (unsigned long long)rw.b[threadIdx.x];
                const unsigned long long D_t = (unsigned long long)rw.band[threadIdx.x];
                bool ovf = false;
                int strictly = 0;
                for (int u = 0; u < n; ++u) {
                    if (!rw.band[u] || u == (int)threadIdx.x) continue;
                    const unsigned long long a_u = (unsigned long long)rw.a[u], b_u = (unsigned long long)rw.b[u];
                    const unsigned long long D_u = (unsigned long long)rw.band[u];
                    const int sgn = (a_u == a_t && b_u == b_t && D_u == D_t)
                                        ? 0 : exact_compare_types(a_u, b_u, D_u, a_t, b_t, D_t, &ovf);
                    strictly += sgn > 0;
                    better += (sgn > 0) || (sgn == 0 && u < (int)threadIdx.x);
                    equal += (sgn == 0);
                }
                if (ovf) atomicCAS(&sm.status, 0, (int)HORA_ERR_EXACT_RANGE);
                my_delta = q + (better < Rp ? 1 : 0);
                if (better == Rp - 1) {                            // this row holds the B-th best candidate
                    sm.found[0] = tot_q + strictly;
                    sm.found[1] = equal + 1;
                    sm.found[2] = Rp - strictly;
                    double lam_x = 0.0;
                    if (exact_gain_as_double(a_t, b_t, D_t, &lam_x)) sm.lam_exact = lam_x;
                    else atomicCAS(&sm.status, 0, (int)HORA_ERR_EXACT_RANGE);
                }
            } else {
                my_delta = q;
            }
            __syncthreads();
            if (B > 0 && sm.status == HORA_OK) {
                n_above = sm.found[0]; n_tied = sm.found[1]; n_taken = sm.found[2];
                lambda = sm.lam_exact;
            }
            __syncthreads();
        }
        // ---- 5: outputs and summary ----
        if (sm.redo) {                                         // (set before the barriers of step 4: the same in every thread)
            if (threadIdx.x == 0) redo[atomicAdd(n_redo, 1u)] = (int32_t)s;
            continue;
        }
        const int status = sm.status;
        const bool failed = status != HORA_OK;
        if (threadIdx.x < n) {
            delta[r0 + threadIdx.x] = failed ? 0 : my_delta;
            G[r0 + threadIdx.x] = failed ? 0 : G0 + my_delta;
        }
        double obj = 0.0;
        // U_i(Delta) from the row's own entry in shared memory: the product in U = 1 - prod_{j<Delta} (b+j)/(a+b+j)
        // is g_i(Delta) (b + Delta - 1) / a  (Eq. marginal); the product loop itself took up to Delta iterations of
        // the slowest lane
        if (!failed && !(flags & HORA_FLAG_SKIP_OBJECTIVE) && threadIdx.x < n && my_delta > 0)
            obj = 1.0 - __longlong_as_double((long long)HORA_AT(row, my_delta - 1, W)) *
                            (rw.b[threadIdx.x] + (double)(my_delta - 1)) / rw.a[threadIdx.x];
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) obj += __shfl_xor_sync(kFull, obj, d);
        __syncthreads();
        if (lane == 0) sm.obj_tmp[warp] = obj;
        __syncthreads();
        if (threadIdx.x == 0 && info != nullptr) {
            double tot = 0.0;
            for (int w = 0; w < kWarps; ++w) tot += sm.obj_tmp[w];
            hora_alloc_info o;
            o.status = status;
            o.first_pass_bits = 0;
            o.lambda = failed ? 0.0 : lambda;
            o.n_above = failed ? 0 : n_above;
            o.n_tied = failed ? 0 : n_tied;
            o.n_tied_taken = failed ? 0 : n_taken;
            o.objective = failed ? 0.0 : tot;
            o.sum_G = failed ? 0 : (long long)n * G0 + B;
            o.sum_cap = sum_cap;
            info[s] = o;
        }
    }
}

// ---- group offsets: exclusive scan of G over all prompts ----

__global__ void __launch_bounds__(kBThreads)
scan_block_sums(const int32_t *__restrict__ G, int64_t N, long long *bsum, int64_t NB, ScanHeader *hdr) {
    __shared__ long long s_warp[kBWarps];
    __shared__ bool s_last;
    const int64_t row0 = (int64_t)blockIdx.x * kScanRows;
    long long v = 0;
    for (int q = 0; q < kScanRows / kBThreads; ++q) {
        const int64_t row = row0 + q * kBThreads + threadIdx.x;
        if (row < N) v += G[row];
    }
    long long tot;
    block_exclusive_sum(v, &tot, s_warp);
    if (threadIdx.x == 0) bsum[blockIdx.x] = tot;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&hdr->ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    long long run = 0;
    for (int64_t b0 = 0; b0 < NB; b0 += kBThreads) {
        const int64_t b = b0 + threadIdx.x;
        const long long x = b < NB ? __ldcg(bsum + b) : 0;
        long long t;
        const long long e = block_exclusive_sum(x, &t, s_warp);
        if (b < NB) bsum[b] = run + e;
        run += t;
    }
}

__global__ void __launch_bounds__(kBThreads)
scan_write_offsets(const int32_t *__restrict__ G, int64_t N, const long long *__restrict__ bpre,
                   int64_t *__restrict__ offsets) {
    __shared__ long long s_warp[kBWarps];
    constexpr int kPer = kScanRows / kBThreads;
    const int64_t row0 = (int64_t)blockIdx.x * kScanRows + (int64_t)threadIdx.x * kPer;
    int g[kPer];
    long long v = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        g[q] = row0 + q < N ? G[row0 + q] : 0;
        v += g[q];
    }
    long long tot;
    long long pre = block_exclusive_sum(v, &tot, s_warp) + bpre[blockIdx.x];
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        if (row0 + q < N) offsets[row0 + q] = pre;
        pre += g[q];
        if (row0 + q == N - 1) offsets[N] = pre;
    }
}

// room for the rank tables of the shared-integer-prior route (its size does not depend on N or S)
constexpr size_t kBRankReserve = ((size_t)5 << 19) + 4096;     // 2.5 MiB: 2 MiB of positions + the per-type tables

// The hard-first rule (Sec. 4.2, "Comparison with the hard-first heuristic") per segment, a warp per segment: the
// segment's budget is dealt round-robin in prompt order to its prompts with c = 0 that are below their cap, the
// rest of it the same way to the other prompts.  Dealing round-robin fills the active class to a common level L
// (or each prompt's cap) and gives the first R prompts with cap > L one more:
//     f(L) = sum_i min(cap_i, L) <= budget of the class < f(L + 1),   R = budget - f(L);
// L comes out of a bisection whose step is one pass over the segment's caps and one warp sum.
__global__ void __launch_bounds__(kBThreads)
hard_first_batched_kernel(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                          int32_t ld, const int64_t *__restrict__ seg_off, const int64_t *__restrict__ budgets, int64_t S,
                          int32_t *__restrict__ delta, int32_t *__restrict__ G, hora_alloc_info *__restrict__ info) {
    const int lane = lane_id();
    const int64_t warp0 = (int64_t)blockIdx.x * kBWarps + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kBWarps;
    auto warp_sum = [](long long v) {
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
        return v;
    };
    for (int64_t s = warp0; s < S; s += n_warps) {
        const int64_t r0 = __ldg(seg_off + s);
        const int64_t n = __ldg(seg_off + s + 1) - r0;
        const long long B = __ldg(budgets + s);
        // prompt i of the segment: (tier, cap) with tier 0 for c = 0; -1 marks an invalid prompt
        auto fetch = [&](int64_t i, int *tier, int *cp) {
            const int ci = __ldg(c + r0 + i);
            *cp = cap ? __ldg(cap + r0 + i) : cap_scalar;
            *tier = (ci < 0 || ci > G0 || *cp < 0 || *cp > ld) ? -1 : (ci > 0);
        };
        long long cap0 = 0, cap1 = 0;
        bool bad = false;
        for (int64_t i = lane; i < n; i += kWarp) {
            int tier, cp;
            fetch(i, &tier, &cp);
            bad |= tier < 0;
            if (tier == 0) cap0 += cp; else if (tier == 1) cap1 += cp;
        }
        cap0 = warp_sum(cap0);
        cap1 = warp_sum(cap1);
        int status = HORA_OK;
        if (__any_sync(kFull, bad) || B < 0) status = HORA_ERR_INVALID_VALUE;
        else if (B > cap0 + cap1) status = HORA_ERR_INFEASIBLE;
        const int active = B <= cap0 ? 0 : 1;                  // the class in which the level is sought
        const long long Bt = active == 0 ? B : B - cap0;
        auto filled = [&](int L) {                             // f(L) over the active class
            long long part = 0;
            for (int64_t i = lane; i < n; i += kWarp) {
                int tier, cp;
                fetch(i, &tier, &cp);
                if (tier == active) part += cp < L ? cp : L;
            }
            return warp_sum(part);
        };
        int L = 0;
        long long used = 0;
        if (!status) {
            int lo = 0, hi = ld;                               // largest L with f(L) <= Bt
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (filled(mid) <= Bt) lo = mid; else hi = mid - 1;
            }
            L = lo;
            used = filled(L);
        }
        const long long R = Bt - used;
        long long before = 0, n_room = 0;                      // prompts with room above the level, in index order
        for (int64_t i0 = 0; i0 < n; i0 += kWarp) {
            const int64_t i = i0 + lane;
            int tier = -1, cp = 0;
            if (i < n) fetch(i, &tier, &cp);
            const bool in_active = !status && tier == active;
            const bool room = in_active && cp > L;
            const unsigned m = __ballot_sync(kFull, room);
            const long long rank = before + __popc(m & ((1u << lane) - 1u));
            int d = 0;
            if (in_active) d = (cp < L ? cp : L) + ((room && rank < R) ? 1 : 0);
            else if (!status && tier == 0) d = cp;            // the level is in the other class: c = 0 prompts are full
            if (i < n) {
                delta[r0 + i] = d;
                G[r0 + i] = status ? 0 : G0 + d;
            }
            before += __popc(m);
            n_room += __popc(m);
        }
        if (lane == 0 && info != nullptr) {
            hora_alloc_info o;
            o.status = status;
            o.first_pass_bits = 0;
            o.lambda = 0.0;
            o.n_above = status ? 0 : B - R;
            o.n_tied = status ? 0 : n_room;
            o.n_tied_taken = status ? 0 : R;
            o.objective = 0.0;
            o.sum_G = status ? 0 : n * (long long)G0 + B;
            o.sum_cap = cap0 + cap1;
            info[s] = o;
        }
    }
}

struct BatchedWorkspace {
    int64_t *seg_off, *budgets;
    long long *bsum;
    int32_t *redo;                 // [S] segments the narrow pass hands to the full pass
    ScanHeader *hdr;
    int32_t *table_status;
    void *tables;
    size_t bytes;
};

static BatchedWorkspace carve_batched(void *base, int64_t N, int64_t S) {
    BatchedWorkspace w{};
    size_t o = 0;
    char *p = static_cast<char *>(base);
    auto take = [&](size_t n) { char *q = p ? p + o : nullptr; o = (o + n + 255) & ~(size_t)255; return q; };
    const int64_t NB = (N + kScanRows - 1) / kScanRows;
    w.hdr = reinterpret_cast<ScanHeader *>(take(sizeof(ScanHeader)));
    w.seg_off = reinterpret_cast<int64_t *>(take(sizeof(int64_t) * (size_t)(S + 1)));
    w.budgets = reinterpret_cast<int64_t *>(take(sizeof(int64_t) * (size_t)(S > 0 ? S : 1)));
    w.bsum = reinterpret_cast<long long *>(take(sizeof(long long) * (size_t)(NB > 0 ? NB : 1)));
    w.redo = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (size_t)(S > 0 ? S : 1)));
    w.table_status = reinterpret_cast<int32_t *>(take(sizeof(int32_t)));
    w.tables = take(kBRankReserve);
    w.bytes = o;
    return w;
}

}  // namespace hora

extern "C" size_t hora_allocate_batched_workspace_bytes(int64_t N, int64_t S) {
    if (N < 0 || S < 0) return 0;
    return hora::carve_batched(nullptr, N, S).bytes;
}

extern "C" hora_status_t hora_allocate_batched(const double *alpha, const double *beta, double alpha0, double beta0,
                                               const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                                               int64_t N, int32_t ld, const int64_t *seg_offsets_host,
                                               const int64_t *budgets_host, int64_t S, uint32_t flags, int32_t *delta,
                                               int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev,
                                               void *workspace, size_t workspace_bytes, void *stream) {
    using namespace hora;
    if (N < 0 || S < 0 || ld < 1 || G0 < 0) return HORA_ERR_INVALID_ARG;
    if (S > 0x7FFFFFFFll) return HORA_ERR_INVALID_ARG;      // segment indices are kept in 32 bits
    if ((alpha == nullptr) != (beta == nullptr)) return HORA_ERR_INVALID_ARG;
    if (alpha == nullptr && !(alpha0 > 0.0 && beta0 > 0.0 && alpha0 < 1.0e300 && beta0 < 1.0e300))
        return HORA_ERR_INVALID_ARG;
    if (cap == nullptr && (cap_scalar < 0 || cap_scalar > ld)) return HORA_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(HORA_FLAG_EXACT_INT | HORA_FLAG_SKIP_OBJECTIVE | HORA_FLAG_SHARED_PRIOR | HORA_FLAG_HARD_FIRST))
        return HORA_ERR_INVALID_ARG;
    const bool hard_first = (flags & HORA_FLAG_HARD_FIRST) != 0;   // the comparison rule: the priors play no part
    if (seg_offsets_host == nullptr || (S > 0 && budgets_host == nullptr)) return HORA_ERR_INVALID_ARG;
    if (seg_offsets_host[0] != 0 || seg_offsets_host[S] != N) return HORA_ERR_INVALID_ARG;
    int64_t max_rows = 0;
    for (int64_t s = 0; s < S; ++s) {
        const int64_t n = seg_offsets_host[s + 1] - seg_offsets_host[s];
        if (n < 0 || budgets_host[s] < 0) return HORA_ERR_INVALID_ARG;
        max_rows = std::max(max_rows, n);
    }
    const int32_t rows_cap = (int32_t)((max_rows + 3) & ~(int64_t)3);
    const size_t smem = sizeof(BatchedSmemFixed) + (size_t)rows_cap * kBRowBytes +
                        (size_t)max_rows * batched_row_stride(ld) * sizeof(unsigned long long);
    // One prior for all prompts: the candidate values are ranked once for all segments (exactly, or as doubles,
    // by the tie mode) and every segment is solved on integer ranks by one warp (no shared-memory keys, no
    // segment size limit).
    const bool exact_ties = (flags & HORA_FLAG_EXACT_INT) != 0;
    const bool by_rank = alpha == nullptr && rank_route_applies(alpha0, beta0, G0, ld, exact_ties) &&
                         rank_pos_applies(G0, ld) && rank_tables_bytes(G0, ld, true) <= kBRankReserve;
    if (!by_rank && !hard_first && (max_rows > kBMaxRows || smem > kBMaxSmem))
        return HORA_ERR_WORKSPACE;                            // segment too large for one CTA
    if (N > 0 && (c == nullptr || delta == nullptr || G == nullptr)) return HORA_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HORA_ERR_WORKSPACE;
    const BatchedWorkspace w = carve_batched(workspace, N, S);
    if (workspace_bytes < w.bytes) return HORA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(w.hdr, 0, sizeof(ScanHeader), st) != cudaSuccess) return HORA_ERR_CUDA;
    if (cudaMemcpyAsync(w.seg_off, seg_offsets_host, sizeof(int64_t) * (size_t)(S + 1), cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return HORA_ERR_CUDA;
    if (S > 0 && cudaMemcpyAsync(w.budgets, budgets_host, sizeof(int64_t) * (size_t)S, cudaMemcpyHostToDevice, st) !=
                     cudaSuccess)
        return HORA_ERR_CUDA;
    int launches = 0;
    if (S > 0 && N > 0 && hard_first) {
        hard_first_batched_kernel<<<clamp_grid((S + kBWarps - 1) / kBWarps, 8), kBThreads, 0, st>>>(
            c, G0, cap, cap_scalar, ld, w.seg_off, w.budgets, S, delta, G, info_dev);
        if (cudaGetLastError() != cudaSuccess) return HORA_ERR_CUDA;
        ++launches;
    } else if (S > 0 && N > 0 && by_rank) {
        if (cudaMemsetAsync(w.table_status, 0, sizeof(int32_t), st) != cudaSuccess) return HORA_ERR_CUDA;
        const RankTables t = rank_tables_carve(w.tables, G0, ld, true);
        const int tl = launch_rank_tables(alpha0, beta0, G0, ld, exact_ties, t, w.table_status, st);
        if (tl < 0) return HORA_ERR_CUDA;
        if (launch_rank_batched(c, G0, cap, cap_scalar, ld, w.seg_off, w.budgets, S, flags, t, w.table_status, delta, G,
                                info_dev, st) != HORA_OK)
            return HORA_ERR_CUDA;
        launches += tl + 1;
    } else if (S > 0 && N > 0) {
        // Rows longer than 256 candidates: a narrow pass over every segment, then the full pass over the segments it
        // handed on (see the kernel).  227 KiB of shared memory per SM, 1 KiB of it reserved per resident CTA.
        const int threads = max_rows <= kWarp ? 128 : kBThreads;
        auto launch = [&](auto kernel, int cap_per_sm, int32_t W, const int32_t *todo, const unsigned int *n_todo) -> cudaError_t {
            const size_t sm_bytes = sizeof(BatchedSmemFixed) + (size_t)rows_cap * kBRowBytes +
                                    (size_t)max_rows * batched_row_stride(W) * sizeof(unsigned long long);
            const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(cap_per_sm, (227 * 1024) / (sm_bytes + 1024)));
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            kernel<<<clamp_grid(S, per_sm), threads, sm_bytes, st>>>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, W,
                                                                     w.seg_off, w.budgets, S, todo, n_todo, w.redo,
                                                                     &w.hdr->n_redo, flags, rows_cap, delta, G, info_dev);
            return cudaGetLastError();
        };
        // 8 entries a lane, as hora_gains; the narrow pass of small segments is compiled for six CTAs per SM (its
        // 31 KB of keys leave room for them), the others for five (128 threads) or three (256)
        cudaError_t e;
        if (ld > kBNarrow) {
            e = threads == 128 ? launch(allocate_batched_kernel<8, 128, 6>, 6, kBNarrow, nullptr, nullptr)
                               : launch(allocate_batched_kernel<8, kBThreads, 3>, 3, kBNarrow, nullptr, nullptr);
            if (e != cudaSuccess) return HORA_ERR_CUDA;
            ++launches;
            e = threads == 128 ? launch(allocate_batched_kernel<8, 128, 5>, 5, ld, w.redo, &w.hdr->n_redo)
                               : launch(allocate_batched_kernel<8, kBThreads, 3>, 3, ld, w.redo, &w.hdr->n_redo);
        } else {
            e = threads == 128 ? launch(allocate_batched_kernel<8, 128, 5>, 5, ld, nullptr, nullptr)
                               : launch(allocate_batched_kernel<8, kBThreads, 3>, 3, ld, nullptr, nullptr);
        }
        if (e != cudaSuccess) return HORA_ERR_CUDA;
        ++launches;
    }
    if (group_offsets != nullptr) {
        if (N == 0) {
            if (cudaMemsetAsync(group_offsets, 0, sizeof(int64_t), st) != cudaSuccess) return HORA_ERR_CUDA;
        } else {
            const int64_t NB = (N + kScanRows - 1) / kScanRows;
            scan_block_sums<<<(int)NB, kBThreads, 0, st>>>(G, N, w.bsum, NB, w.hdr);
            scan_write_offsets<<<(int)NB, kBThreads, 0, st>>>(G, N, w.bsum, group_offsets);
            launches += 2;
        }
    }
    count_launches(launches);
    return cuda_ok(cudaGetLastError());
}
