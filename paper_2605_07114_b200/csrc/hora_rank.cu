// Rank-based exact allocation for a shared integer prior (Proposition 1; Eq. marginal; Algorithm 1 Phase B).
//
// One Beta(alpha0, beta0) prior for every prompt leaves G0 + 1 posteriors (a, b) = (alpha0 + c, beta0 + G0 - c)
// and so at most T = (G0 + 1) * ld distinct candidate values g_c(Delta).  Greedy with lowest-index ties is then
// decided by (i) the exact order of those T values and (ii) how many prompts hold each of them — prompt i holds
// g_c(Delta) iff c_i = c and cap_i >= Delta.  Nothing per candidate is ever materialised:
//
//   tables   every type is ranked exactly: rank = number of types with a strictly larger gain.  Inside a class
//            the order is the order of Delta (rows decrease strictly); across classes a thread binary-searches
//            the other class's row, comparing fp64 values (same arithmetic as hora_gains) where they differ by
//            more than 2^-30 relative — two thousand times the evaluation error — and exact 512-bit fractions
//            where they do not.  Exactly equal types share a rank.
//   count    one pass over (c_i, cap_i): a histogram H[c][cap] (shared memory, one update per distinct bin per
//            warp); the last CTA turns it into instance counts per type (suffix sums over cap), adds them up by
//            rank, finds the rank r* at which the running count reaches B, and derives per class the number of
//            candidates above the threshold and whether the next one is tied with it.  The objective comes from
//            the same histogram (every prompt of bin (c, cap) gets the same Delta, up to the tied rollouts, each
//            of which adds exactly lambda).
//   sums/out two passes over (c_i, cap_i) again: sums of (above, tied) per 256 prompts and per CTA, then — every
//            CTA adding up the sums before its own — Delta, G and the CSR offsets, the first R tied prompts in
//            index order taking one more.  Neither pass has a barrier in its loop or a serial scan behind it.
//
// The batched form (hora_allocate_batched with the same kind of prior) ranks once for all segments and gives a
// warp to each segment: the threshold rank is bisected with a table pos[c][r] = #{Delta : rank_c(Delta) < r}, so
// one step costs one lookup per prompt and one warp reduction.
#include <cmath>

#define HORA_FILE_ID 4
#include "hora_block.cuh"
#include "hora_checked.cuh"
#include "hora_exact.cuh"
#include "hora_gains_chunk.cuh"
#include "hora_rank.cuh"

HORA_CHECKED_REGISTER()

namespace hora {

constexpr double kRankBand = 9.313225746154785e-10;       // 2^-30

static inline size_t rk_align(size_t x) { return (x + 255) & ~(size_t)255; }

bool rank_route_applies(double alpha0, double beta0, int32_t G0, int32_t ld, bool exact) {
    if (!(alpha0 > 0.0 && beta0 > 0.0) || G0 < 0 || ld < 1) return false;
    const double top = alpha0 + beta0 + (double)G0 + (double)ld;
    if (!(top < 1048576.0)) return false;
    if ((int64_t)(G0 + 1) * (int64_t)ld > kRankMaxTypes) return false;
    if (!exact) return true;                                // ties are equal doubles: nothing else to ask of the prior
    if (!(alpha0 >= 1.0 && beta0 >= 1.0 && alpha0 == std::floor(alpha0) && beta0 == std::floor(beta0))) return false;
    // every exact form a (b)_a / (b+Delta-1)_{a+1} or a (b)_{Delta-1} / (a+b)_Delta of the table fits 512 bits
    const double factors = std::fmin(alpha0 + (double)G0 + 1.0, (double)ld);
    return factors * std::log2(top) <= 500.0;
}

bool rank_pos_applies(int32_t G0, int32_t ld) {
    const int64_t C = G0 + 1, T = C * ld;
    return ld < 65536 && C * (T + 1) <= kRankMaxPos;
}

static size_t tables_layout(void *base, int32_t G0, int32_t ld, bool with_pos, RankTables *t) {
    const size_t C = (size_t)G0 + 1, T = C * (size_t)ld;
    size_t o = 0;
    char *p = static_cast<char *>(base);
    auto take = [&](size_t n) { char *q = p ? p + o : nullptr; o = rk_align(o + n); return q; };
    RankTables r{};
    r.rank = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * T));
    r.gain = reinterpret_cast<double *>(take(sizeof(double) * T));
    r.util = reinterpret_cast<double *>(take(sizeof(double) * C * ((size_t)ld + 1)));
    r.lam = reinterpret_cast<double *>(take(sizeof(double) * T));
    r.pos = with_pos ? reinterpret_cast<uint16_t *>(take(sizeof(uint16_t) * C * (T + 1))) : nullptr;
    if (t) *t = r;
    return o;
}

size_t rank_tables_bytes(int32_t G0, int32_t ld, bool with_pos) { return tables_layout(nullptr, G0, ld, with_pos, nullptr); }

RankTables rank_tables_carve(void *base, int32_t G0, int32_t ld, bool with_pos) {
    RankTables t;
    tables_layout(base, G0, ld, with_pos, &t);
    return t;
}

// ---------------------------------------------------------------------------------------------------
// Tables.

// Every CTA builds the whole table of fp64 gains in shared memory (a warp per class row: a few hundred
// instructions), then a thread ranks one type.
// EXACT: two types whose doubles are within 2^-30 of each other are compared as exact fractions (integer prior);
// otherwise the doubles themselves are the order and equal doubles are ties, which is how the key-based selection
// of hora_allocate treats a matrix of hora_gains without HORA_FLAG_EXACT_INT.
template <int E, bool EXACT>
__global__ void __launch_bounds__(kSelThreads)
rank_table_kernel(double alpha0, double beta0, int32_t G0, int32_t ld, RankTables t, int32_t *status) {
    pdl_enter();
    extern __shared__ __align__(16) unsigned char s_rank_tab[];
    double *s_g = reinterpret_cast<double *>(s_rank_tab);
    const int C = G0 + 1, T = C * ld;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    for (int row = warp; row < C; row += kSelThreads / kWarp) {
        const double a = alpha0 + (double)row, b = beta0 + (double)(G0 - row);
        double carry = 1.0;
        for (int32_t k0 = 0; k0 < ld; k0 += kWarp * E)
            gains_chunk<E, false, false>(a, b, a + b, ld, ld, k0, lane, carry, s_g + (size_t)row * ld, nullptr, nullptr);
    }
    __syncthreads();
    const int id = blockIdx.x * kSelThreads + threadIdx.x;
    if (id >= T) return;
    const int c = id / ld, j = id - c * ld;
    const double g0 = s_g[id];
    const double up = g0 * (1.0 + kRankBand), dn = g0 * (1.0 - kRankBand);
    const unsigned long long a = (unsigned long long)alpha0 + c, b = (unsigned long long)beta0 + (G0 - c);
    bool overflow = false, first_of_class = true;           // first: no class c2 < c holds an exactly equal type
    int rank = j;                                           // the entries before it in its own row
    for (int c2 = 0; c2 < C; ++c2) {
        if (c2 == c) continue;
        const double *row = s_g + (size_t)c2 * ld;
        const unsigned long long a2 = (unsigned long long)alpha0 + c2, b2 = (unsigned long long)beta0 + (G0 - c2);
        int lo = 0, hi = ld;                                // first column of row c2 that is not strictly above g0
        bool tie_seen = false;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            const double x = row[mid];
            bool above;
            if (!EXACT) {
                above = x > g0;
                tie_seen |= x == g0;
            } else if (x > up) above = true;
            else if (x < dn) above = false;
            else {
                const int sgn = exact_compare_types(a2, b2, (unsigned long long)mid + 1, a, b, (unsigned long long)j + 1, &overflow);
                above = sgn > 0;
                tie_seen |= sgn == 0;
            }
            if (above) lo = mid + 1; else hi = mid;
        }
        rank += lo;
        // the search ends on the equal entry if there is one (it is the first that is not above), but need not
        // have compared it: look at column lo itself
        if (c2 < c && lo < ld) {
            const double x = row[lo];
            if (!EXACT) {
                if (x == g0) first_of_class = false;
            } else if (x <= up && x >= dn) {
                if (tie_seen || exact_compare_types(a2, b2, (unsigned long long)lo + 1, a, b, (unsigned long long)j + 1, &overflow) == 0)
                    first_of_class = false;
            }
        }
    }
    if (overflow) raise_status(status, HORA_ERR_EXACT_RANGE);
    t.rank[id] = rank;
    t.gain[id] = g0;
    if (first_of_class) HORA_AT(t.lam, rank, T) = g0;
    t.util[(size_t)c * (ld + 1) + j + 1] = utility_from_gain(g0, alpha0 + (double)c, beta0 + (double)(G0 - c), j + 1);
    if (j == 0) t.util[(size_t)c * (ld + 1)] = 0.0;
}

// pos[c][r] = number of columns of row c whose rank is below r, r = 0..T
__global__ void __launch_bounds__(kSelThreads)
rank_pos_kernel(int32_t G0, int32_t ld, RankTables t) {
    const int64_t C = G0 + 1, T = C * ld;
    const int64_t id = (int64_t)blockIdx.x * kSelThreads + threadIdx.x;
    if (id >= C * (T + 1)) return;
    const int64_t c = id / (T + 1);
    const int32_t r = (int32_t)(id - c * (T + 1));
    const int32_t *row = t.rank + c * ld;
    int lo = 0, hi = ld;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(row + mid) < r) lo = mid + 1; else hi = mid;
    }
    t.pos[id] = (uint16_t)lo;
}

int launch_rank_tables(double alpha0, double beta0, int32_t G0, int32_t ld, bool exact, const RankTables &t,
                       int32_t *status, cudaStream_t s) {
    const int C = G0 + 1, T = C * ld;
    const size_t smem = sizeof(double) * (size_t)T;
    const int grid = (T + kSelThreads - 1) / kSelThreads;
    auto go = [&](auto kernel) -> bool {
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return false;
        kernel<<<grid, kSelThreads, smem, s>>>(alpha0, beta0, G0, ld, t, status);
        return cudaGetLastError() == cudaSuccess;
    };
    bool ok;
    if (exact) ok = go(rank_table_kernel<8, true>);          // 8 entries a lane at every ld, as hora_gains builds rows
    else ok = go(rank_table_kernel<8, false>);
    if (!ok) return -1;
    int launches = 1;
    if (t.pos != nullptr) {
        const int64_t n = (int64_t)C * ((int64_t)T + 1);
        rank_pos_kernel<<<(int)((n + kSelThreads - 1) / kSelThreads), kSelThreads, 0, s>>>(G0, ld, t);
        if (cudaGetLastError() != cudaSuccess) return -1;
        ++launches;
    }
    return launches;
}

// ---------------------------------------------------------------------------------------------------
// Single problem.

constexpr int kRankTask = 256;          // prompts a warp handles at a time in the sum / output passes (2 x 128)
constexpr int kRankMaxCtas = 4096;      // CTAs of those passes (each owns a contiguous run of tasks)

struct RankHeader {
    int32_t status;
    unsigned int ticket[3];
    int32_t rstar;                     // rank of the threshold; -1 when B == 0
    int32_t pad;
    long long R;                       // tied candidates to take
    unsigned long long n_above, n_tied, sum_cap;
    double lambda, objective;
};

struct RankWorkspace {
    RankHeader *hdr;
    unsigned long long *H;             // [C][ld+1] prompts per (c, cap)
    unsigned long long *bucket;        // [bins] instances by rank, stored top down: slot bins-1-rank
    int2 *tsum;                        // [NT] (above, tied) summed over each task of kRankTask prompts
    long long *super_hi, *super_t;     // [kRankMaxCtas] the same summed over each CTA's run of tasks
    int32_t *class_tab;                // [C] (candidates above the threshold << 1) | next one is tied
    RankTables tab;
    int32_t bins;
    size_t zero_bytes, bytes;
};

static int rank_bins(int32_t G0, int32_t ld) {
    const int T = (G0 + 1) * ld;
    int bins = kSelThreads;                                 // locate_rank wants a power of two in [256, 8192]
    while (bins < T) bins <<= 1;
    return bins;
}

static RankWorkspace rank_carve(void *base, int64_t N, int32_t G0, int32_t ld) {
    RankWorkspace w{};
    const size_t C = (size_t)G0 + 1;
    const int64_t NT = (N + kRankTask - 1) / kRankTask;
    w.bins = rank_bins(G0, ld);
    size_t o = 0;
    char *p = static_cast<char *>(base);
    auto take = [&](size_t n) { char *q = p ? p + o : nullptr; o = rk_align(o + n); return q; };
    w.hdr = reinterpret_cast<RankHeader *>(take(sizeof(RankHeader)));
    w.H = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * C * ((size_t)ld + 1)));
    w.bucket = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * (size_t)w.bins));
    w.zero_bytes = o;                                        // everything before this is cleared per call
    w.tsum = reinterpret_cast<int2 *>(take(sizeof(int2) * (size_t)(NT > 0 ? NT : 1)));
    w.super_hi = reinterpret_cast<long long *>(take(sizeof(long long) * kRankMaxCtas));
    w.super_t = reinterpret_cast<long long *>(take(sizeof(long long) * kRankMaxCtas));
    w.class_tab = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * C));
    const size_t tb = rank_tables_bytes(G0, ld, false);
    char *tbase = take(tb);
    w.tab = rank_tables_carve(tbase, G0, ld, false);
    if (!p) w.tab = RankTables{};
    w.bytes = o;
    return w;
}

size_t rank_allocate_workspace_bytes(int64_t N, int32_t G0, int32_t ld) { return rank_carve(nullptr, N, G0, ld).bytes; }

// Upper bound over every (G0, ld) the route accepts: what a caller reserves who only knows N.
size_t rank_allocate_workspace_bound(int64_t N) {
    const size_t T = kRankMaxTypes, NT = (size_t)((N + kRankTask - 1) / kRankTask) + 1;
    // C (ld + 1) <= 2 T, C <= T, bins <= T; each array rounded up to 256 bytes
    return rk_align(sizeof(RankHeader)) + rk_align(8 * 2 * T) + rk_align(8 * T) + rk_align(8 * NT) +
           2 * rk_align(8 * kRankMaxCtas) + rk_align(4 * T) +
           rk_align(4 * T) + rk_align(8 * T) + rk_align(8 * 2 * T) + rk_align(8 * T) + 4096;
}

// Four consecutive prompts, (c_i, cap_i) each: two 16-byte loads where the arrays allow (`vec`), else scalar loads.
// A prompt at or beyond N reads as c = -1 (no bin, not an error).
struct RankQuad { int32_t c[4], cap[4]; };

__device__ __forceinline__ void rank_load_quad(RankQuad &q, const int32_t *__restrict__ c, const int32_t *__restrict__ cap,
                                               int32_t cap_scalar, int64_t p, int64_t N, bool vec) {
    if (vec && p + 4 <= N) {
        const int4 cv = __ldg(reinterpret_cast<const int4 *>(c + p));
        q.c[0] = cv.x; q.c[1] = cv.y; q.c[2] = cv.z; q.c[3] = cv.w;
        if (cap) {
            const int4 pv = __ldg(reinterpret_cast<const int4 *>(cap + p));
            q.cap[0] = pv.x; q.cap[1] = pv.y; q.cap[2] = pv.z; q.cap[3] = pv.w;
        } else {
            q.cap[0] = q.cap[1] = q.cap[2] = q.cap[3] = cap_scalar;
        }
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            q.c[k] = p + k < N ? __ldg(c + p + k) : -1;
            q.cap[k] = (p + k < N && cap) ? __ldg(cap + p + k) : cap_scalar;
        }
    }
}

// (candidates above the threshold, tied candidate) of a prompt from its class entry; zeros for a missing prompt
__device__ __forceinline__ void rank_row_state(int32_t ci, int32_t cp, const int32_t *s_class, int n_class, int tiers,
                                               int *hi, int *tied) {
    *hi = 0;
    *tied = 0;
    if (ci < 0) return;
    const int e = HORA_AT(s_class, tiers ? (ci > 0) : ci, n_class), above = e >> 1;   // tiers: two classes only, c = 0 and c > 0
    *hi = cp < above ? cp : above;
    *tied = (e & 1) && cp > above;
}

// Tail of the hard-first heuristic (Sec. 4.2, "Comparison with the hard-first heuristic"), run by the last CTA of
// the counting pass over the two-class histogram H[tier][cap], tier 0 = prompts with c = 0.  The budget is dealt
// one rollout at a time, round-robin in prompt order, to the tier-0 prompts that are below their cap; what they
// cannot absorb is dealt the same way to the others.  Dealing round-robin fills every prompt of the active tier
// to a common level L (or its cap) and gives the first R prompts with cap > L one more:
//     f(L) = sum_i min(cap_i, L) <= budget of the tier < f(L + 1),   R = budget - f(L).
// The class table then reads exactly like the rank route's (level, "has a tied candidate"), so the same sum and
// output passes finish the job.
__device__ void hard_first_tail(const RankWorkspace &w, int32_t ld, int64_t B, long long *s_warp) {
    RankHeader *hdr = w.hdr;
    const unsigned long long *H0 = w.H, *H1 = w.H + (ld + 1);
    long long part0 = 0, part1 = 0;
    for (int cp = threadIdx.x; cp <= ld; cp += kSelThreads) {
        part0 += (long long)__ldcg(H0 + cp) * cp;
        part1 += (long long)__ldcg(H1 + cp) * cp;
    }
    long long cap0, cap1;
    block_exclusive_sum(part0, &cap0, s_warp);
    block_exclusive_sum(part1, &cap1, s_warp);
    if (threadIdx.x == 0) {
        hdr->sum_cap = (unsigned long long)(cap0 + cap1);
        if (B > cap0 + cap1) raise_status(&hdr->status, HORA_ERR_INFEASIBLE);
    }
    __syncthreads();
    if (*(volatile int32_t *)&hdr->status != 0) return;
    const int tier = B <= cap0 ? 0 : 1;                      // the tier the level is sought in
    const long long Bt = tier == 0 ? B : B - cap0;
    const unsigned long long *Ht = tier == 0 ? H0 : H1;
    auto filled = [&](int L) -> long long {                  // f(L), every thread gets it
        long long part = 0;
        for (int cp = threadIdx.x; cp <= ld; cp += kSelThreads) part += (long long)__ldcg(Ht + cp) * (cp < L ? cp : L);
        long long tot;
        block_exclusive_sum(part, &tot, s_warp);
        return tot;
    };
    int lo = 0, hi = ld;                                     // largest L with f(L) <= Bt  (f(0) = 0 <= Bt)
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (filled(mid) <= Bt) lo = mid; else hi = mid - 1;
    }
    const int L = lo;
    const long long used = filled(L);
    long long part = 0;
    for (int cp = threadIdx.x; cp <= ld; cp += kSelThreads)
        if (cp > L) part += (long long)__ldcg(Ht + cp);
    long long above_level;                                   // prompts of the tier that can take one more
    block_exclusive_sum(part, &above_level, s_warp);
    if (threadIdx.x == 0) {
        const int active = (L << 1) | (above_level > 0 ? 1 : 0);
        w.class_tab[tier] = active;
        w.class_tab[1 - tier] = tier == 0 ? 0 : (ld << 1);  // the others get nothing / tier 0 is filled to its caps
        hdr->rstar = L;
        hdr->R = Bt - used;
        hdr->n_above = (unsigned long long)(B - (Bt - used));
        hdr->n_tied = (unsigned long long)above_level;
        hdr->lambda = 0.0;
        hdr->objective = 0.0;
    }
}

// HARD: the hard-first heuristic instead of the hit-utility ranks — two classes only (c = 0, c > 0), and the tail
// finds a water level instead of a threshold rank (hard_first_tail).
template <bool HARD>
__global__ void __launch_bounds__(kSelThreads, 8)
rank_count_kernel(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                  int64_t N, int32_t ld, int64_t B, uint32_t flags, int vec, RankWorkspace w) {
    pdl_enter();
    extern __shared__ __align__(16) unsigned char s_rank_cnt[];
    unsigned int *s_hist = reinterpret_cast<unsigned int *>(s_rank_cnt);
    __shared__ long long s_warp[kSelThreads / kWarp];
    __shared__ double s_obj[kSelThreads / kWarp];
    const int C = HARD ? 2 : G0 + 1, n_h = C * (ld + 1);
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    for (int b = threadIdx.x; b < n_h; b += kSelThreads) s_hist[b] = 0;
    __syncthreads();
    bool bad = false;
    // a handful of bins: one shared-memory update per distinct bin per warp (the lanes would otherwise serialise
    // on a few addresses)
    const bool few_bins = n_h <= 64;
    auto tally = [&](const RankQuad &q, int64_t p) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            int bin = -1;
            if (p + k < N) {                                 // (a prompt beyond N was read as c = -1: not an error)
                if (q.c[k] < 0 || q.c[k] > G0 || q.cap[k] < 0 || q.cap[k] > ld) bad = true;
                else bin = (HARD ? (q.c[k] > 0) : q.c[k]) * (ld + 1) + q.cap[k];
            }
            if (few_bins) {                                  // (the match costs more than it saves on a wide table)
                const unsigned peers = __match_any_sync(kFull, bin);
                if (bin >= 0 && lane == __ffs(peers) - 1) atomicAdd(&HORA_AT(s_hist, bin, n_h), (unsigned)__popc(peers));
            } else if (bin >= 0) {
                atomicAdd(&HORA_AT(s_hist, bin, n_h), 1u);
            }
        }
    };
    // two quads in flight per thread
    const int64_t stride = (int64_t)gridDim.x * kSelThreads * 4;
    for (int64_t base = (int64_t)blockIdx.x * kSelThreads * 4; base < N; base += 2 * stride) {   // uniform per CTA
        const int64_t p = base + threadIdx.x * 4;
        RankQuad q0, q1;
        rank_load_quad(q0, c, cap, cap_scalar, p, N, vec != 0);
        rank_load_quad(q1, c, cap, cap_scalar, p + stride, N, vec != 0);
        tally(q0, p);
        tally(q1, p + stride);
    }
    if (bad) raise_status(&w.hdr->status, HORA_ERR_INVALID_VALUE);
    __syncthreads();
    for (int b = threadIdx.x; b < n_h; b += kSelThreads) {
        const unsigned int v = s_hist[b];
        if (v) atomicAdd(w.H + b, (unsigned long long)v);
    }
    if (!last_block(&w.hdr->ticket[0])) return;
    if (HARD) {
        hard_first_tail(w, ld, B, s_warp);
        return;
    }

    // ---- the last CTA: from the histogram to the threshold ----
    RankHeader *hdr = w.hdr;
    long long capsum = 0;
    for (int b = threadIdx.x; b < n_h; b += kSelThreads) capsum += (long long)__ldcg(w.H + b) * (b % (ld + 1));
    long long sum_cap;
    block_exclusive_sum(capsum, &sum_cap, s_warp);
    if (threadIdx.x == 0) {
        hdr->sum_cap = (unsigned long long)sum_cap;
        if (B > sum_cap) raise_status(&hdr->status, HORA_ERR_INFEASIBLE);
    }
    __syncthreads();
    if (*(volatile int32_t *)&hdr->status != 0) return;
    // instances per type: #{i : c_i = c, cap_i >= Delta} is a suffix sum of the class's histogram row; a warp per
    // class walks the row from the top, 32 values of Delta at a time, and adds each count to its rank's bucket
    for (int cls = warp; cls < C; cls += kSelThreads / kWarp) {
        const unsigned long long *Hrow = w.H + (size_t)cls * (ld + 1);
        const int32_t *rrow = w.tab.rank + (size_t)cls * ld;
        long long carry = 0;
        for (int top = ld; top >= 1; top -= kWarp) {
            const int D = top - lane;
            long long inc = D >= 1 ? (long long)__ldcg(Hrow + D) : 0;
#pragma unroll
            for (int d = 1; d < kWarp; d <<= 1) {
                const long long x = __shfl_up_sync(kFull, inc, d);
                if (lane >= d) inc += x;
            }
            const long long cnt = carry + inc;
            if (D >= 1 && cnt > 0) atomicAdd(&HORA_AT(w.bucket, w.bins - 1 - __ldg(rrow + D - 1), w.bins), (unsigned long long)cnt);
            carry += __shfl_sync(kFull, inc, kWarp - 1);
        }
    }
    __threadfence();
    __syncthreads();
    int rstar = -1;
    long long above = 0, count = 0;
    if (B > 0) {
        const int digit = locate_rank(w.bucket, w.bins, B, &above, &count, s_warp);
        if (digit < 0) {                                    // B <= sum of the buckets: an internal fault
            if (threadIdx.x == 0) raise_status(&hdr->status, HORA_ERR_INTERNAL);
            return;
        }
        rstar = w.bins - 1 - digit;
    }
    // per class: candidates above the threshold (ranks below r*), and whether the next one carries r*
    for (int cls = threadIdx.x; cls < C; cls += kSelThreads) {
        const int32_t *rrow = w.tab.rank + (size_t)cls * ld;
        int lo = 0, hi = rstar >= 0 ? ld : 0;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(rrow + mid) < rstar) lo = mid + 1; else hi = mid;
        }
        const int tied = rstar >= 0 && lo < ld && __ldg(rrow + lo) == rstar;
        w.class_tab[cls] = (lo << 1) | tied;
    }
    __syncthreads();
    const double lambda = rstar >= 0 ? __ldg(w.tab.lam + rstar) : 0.0;
    // objective: every prompt of bin (c, cap) ends at Delta = min(cap, above_c), plus the tied rollouts handed
    // out, each worth lambda (Eq. appendix-objective: U is the sum of the gains taken); fixed summation order
    double obj = 0.0;
    if (!(flags & HORA_FLAG_SKIP_OBJECTIVE)) {
        for (int b = threadIdx.x; b < n_h; b += kSelThreads) {
            const unsigned long long cnt = __ldcg(w.H + b);
            if (cnt == 0ull) continue;
            const int cls = b / (ld + 1), cp = b - cls * (ld + 1);
            const int hi_c = w.class_tab[cls] >> 1;
            obj += (double)cnt * __ldg(w.tab.util + (size_t)cls * (ld + 1) + (cp < hi_c ? cp : hi_c));
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) obj += __shfl_xor_sync(kFull, obj, d);
        if (lane == 0) s_obj[warp] = obj;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double total = 0.0;
        if (!(flags & HORA_FLAG_SKIP_OBJECTIVE)) {
            for (int k = 0; k < kSelThreads / kWarp; ++k) total += s_obj[k];
            total += (double)(B - above) * lambda;
        }
        hdr->rstar = rstar;
        hdr->R = B - above;
        hdr->n_above = (unsigned long long)above;
        hdr->n_tied = (unsigned long long)count;
        hdr->lambda = lambda;
        hdr->objective = total;
    }
}

// The prompts are cut into tasks of kRankTask; CTA k owns the contiguous tasks [k m, (k+1) m) and its warps take
// them in turn.  A lane holds 4 consecutive prompts of each 128 (two 16-byte loads), so a task is two steps.
__device__ __forceinline__ void rank_task_state(const RankQuad (&q)[2], const int32_t *s_class, int n_class, int tiers,
                                                int (&hi)[2][4], int (&tied)[2][4]) {
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int k = 0; k < 4; ++k) rank_row_state(q[h].c[k], q[h].cap[k], s_class, n_class, tiers, &hi[h][k], &tied[h][k]);
}

// Sums of (above, tied) per task and per CTA.  No barrier inside the loop, no ticket at the end.
__global__ void __launch_bounds__(kSelThreads, 4)
rank_sums_kernel(const int32_t *__restrict__ c, int32_t n_class, int tiers, const int32_t *__restrict__ cap,
                 int32_t cap_scalar, int64_t N, int vec, RankWorkspace w, int64_t NT, int64_t m) {
    pdl_enter();
    extern __shared__ __align__(16) unsigned char s_rank_cls[];
    int32_t *s_class = reinterpret_cast<int32_t *>(s_rank_cls);
    __shared__ long long s_acc[2][kSelThreads / kWarp];
    if (*(volatile int32_t *)&w.hdr->status != 0) return;    // the output pass writes zeros and reads none of this
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    for (int k = threadIdx.x; k < n_class; k += kSelThreads) s_class[k] = w.class_tab[k];
    __syncthreads();
    const int64_t t0 = (int64_t)blockIdx.x * m, t1 = t0 + m < NT ? t0 + m : NT;
    long long acc_hi = 0, acc_t = 0;
    for (int64_t t = t0 + warp; t < t1; t += kSelThreads / kWarp) {
        RankQuad q[2];
        rank_load_quad(q[0], c, cap, cap_scalar, t * kRankTask + lane * 4, N, vec != 0);
        rank_load_quad(q[1], c, cap, cap_scalar, t * kRankTask + 128 + lane * 4, N, vec != 0);
        int hi[2][4], tied[2][4], hs = 0, ts = 0;
        rank_task_state(q, s_class, n_class, tiers, hi, tied);
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int k = 0; k < 4; ++k) { hs += hi[h][k]; ts += tied[h][k]; }
        hs = __reduce_add_sync(kFull, hs);                   // at most 256 * ld < 2^31
        ts = __reduce_add_sync(kFull, ts);
        if (lane == 0) w.tsum[t] = make_int2(hs, ts);
        acc_hi += hs;
        acc_t += ts;
    }
    if (lane == 0) { s_acc[0][warp] = acc_hi; s_acc[1][warp] = acc_t; }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long a = 0, b = 0;
        for (int k = 0; k < kSelThreads / kWarp; ++k) { a += s_acc[0][k]; b += s_acc[1][k]; }
        w.super_hi[blockIdx.x] = a;
        w.super_t[blockIdx.x] = b;
    }
}

// Outputs.  CTA k adds up the sums of the CTAs before it, then each warp walks the CTA's tasks eight at a time:
// lanes 0..7 fetch the eight task sums, a 3-step scan gives the warp the prefix of its own task and the total
// of the eight, and the warp writes its 256 prompts (16-byte stores where the arrays allow: `vec_out`).
__global__ void __launch_bounds__(kSelThreads, 3)
rank_out_kernel(const int32_t *__restrict__ c, int32_t G0, int32_t n_class, int tiers, const int32_t *__restrict__ cap,
                int32_t cap_scalar, int64_t N, int64_t B, int vec, RankWorkspace w, int64_t NT, int64_t m,
                int32_t *__restrict__ delta,
                int32_t *__restrict__ G, int64_t *__restrict__ offsets, int vec_out, hora_alloc_info *info) {
    pdl_enter();
    extern __shared__ __align__(16) unsigned char s_rank_cls[];
    int32_t *s_class = reinterpret_cast<int32_t *>(s_rank_cls);
    __shared__ long long s_warp[kSelThreads / kWarp];
    const RankHeader *hdr = w.hdr;
    const int32_t status = *(volatile int32_t *)&hdr->status;
    const bool failed = status != 0;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    long long base_hi = 0, base_t = 0;
    if (!failed) {
        for (int k = threadIdx.x; k < n_class; k += kSelThreads) s_class[k] = w.class_tab[k];
        long long ph = 0, pt = 0;
        for (int k = threadIdx.x; k < (int)blockIdx.x; k += kSelThreads) { ph += w.super_hi[k]; pt += w.super_t[k]; }
        block_exclusive_sum(ph, &base_hi, s_warp);
        block_exclusive_sum(pt, &base_t, s_warp);
    }
    __syncthreads();
    const long long R = failed ? 0 : hdr->R;
    const int64_t t0 = (int64_t)blockIdx.x * m, t1 = t0 + m < NT ? t0 + m : NT;
    long long run_hi = base_hi, run_t = base_t;
    for (int64_t tc = t0; tc < t1; tc += kSelThreads / kWarp) {
        const int64_t t = tc + warp;
        RankQuad q[2];
        if (!failed && t < t1) {
            rank_load_quad(q[0], c, cap, cap_scalar, t * kRankTask + lane * 4, N, vec != 0);
            rank_load_quad(q[1], c, cap, cap_scalar, t * kRankTask + 128 + lane * 4, N, vec != 0);
        }
        int2 v = make_int2(0, 0);
        if (!failed && lane < kSelThreads / kWarp && tc + lane < t1) v = w.tsum[tc + lane];
        int2 inc = v;
#pragma unroll
        for (int d = 1; d < kSelThreads / kWarp; d <<= 1) {
            const int x = __shfl_up_sync(kFull, inc.x, d), y = __shfl_up_sync(kFull, inc.y, d);
            if (lane >= d) { inc.x += x; inc.y += y; }
        }
        const int before_hi = __shfl_sync(kFull, inc.x - v.x, warp), before_t = __shfl_sync(kFull, inc.y - v.y, warp);
        const int chunk_hi = __shfl_sync(kFull, inc.x, kSelThreads / kWarp - 1), chunk_t = __shfl_sync(kFull, inc.y, kSelThreads / kWarp - 1);
        if (t < t1) {
            long long pre_hi = run_hi + before_hi, pre_t = run_t + before_t;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t row0 = t * kRankTask + h * 128 + lane * 4;
                int hi[4], tied[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    hi[k] = tied[k] = 0;
                    if (!failed) rank_row_state(q[h].c[k], q[h].cap[k], s_class, n_class, tiers, &hi[k], &tied[k]);
                }
                const int hs = hi[0] + hi[1] + hi[2] + hi[3], ts = tied[0] + tied[1] + tied[2] + tied[3];
                // exclusive prefix over the lanes of (above, tied), packed: tied <= 4 per lane, 128 per step;
                // above <= 4 ld < 2^16 per lane, 2^21 per step
                const int packed = (hs << 8) | ts;
                int sc = packed;
#pragma unroll
                for (int d = 1; d < kWarp; d <<= 1) {
                    const int x = __shfl_up_sync(kFull, sc, d);
                    if (lane >= d) sc += x;
                }
                const int excl = sc - packed, total = __shfl_sync(kFull, sc, kWarp - 1);
                long long ph = pre_hi + (excl >> 8), pt = pre_t + (excl & 0xFF);
                int32_t d4[4];
                int64_t of[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    d4[k] = hi[k] + ((tied[k] && pt < R) ? 1 : 0);
                    of[k] = failed ? 0 : (row0 + k) * (int64_t)G0 + ph + (pt < R ? pt : R);
                    ph += hi[k];
                    pt += tied[k];
                }
                if (row0 + 4 <= N && vec_out) {
                    *reinterpret_cast<int4 *>(delta + row0) = make_int4(d4[0], d4[1], d4[2], d4[3]);
                    *reinterpret_cast<int4 *>(G + row0) =
                        failed ? make_int4(0, 0, 0, 0) : make_int4(G0 + d4[0], G0 + d4[1], G0 + d4[2], G0 + d4[3]);
                    if (offsets) {
                        *reinterpret_cast<longlong2 *>(offsets + row0) = make_longlong2(of[0], of[1]);
                        *reinterpret_cast<longlong2 *>(offsets + row0 + 2) = make_longlong2(of[2], of[3]);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (row0 + k < N) {
                            delta[row0 + k] = d4[k];
                            G[row0 + k] = failed ? 0 : G0 + d4[k];
                            if (offsets) offsets[row0 + k] = of[k];
                        }
                    }
                }
                pre_hi += total >> 8;
                pre_t += total & 0xFF;
            }
        }
        run_hi += chunk_hi;
        run_t += chunk_t;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (offsets) offsets[N] = failed ? 0 : N * (int64_t)G0 + B;
        if (info) {
            info->status = status;
            info->first_pass_bits = failed || B == 0 ? 0 : -1;   // no key pass at all on this route
            info->lambda = failed ? 0.0 : hdr->lambda;
            info->n_above = failed ? 0 : (int64_t)hdr->n_above;
            info->n_tied = failed ? 0 : (int64_t)hdr->n_tied;
            info->n_tied_taken = failed ? 0 : hdr->R;
            info->objective = failed ? 0.0 : hdr->objective;
            info->sum_G = failed ? 0 : N * (int64_t)G0 + B;
            info->sum_cap = (int64_t)hdr->sum_cap;
        }
    }
}

// The three passes over (c_i, cap_i) shared by the rank route and the hard-first heuristic.
template <bool HARD>
static hora_status_t launch_rank_passes(const RankWorkspace &w, const int32_t *c, int32_t G0, const int32_t *cap,
                                        int32_t cap_scalar, int64_t N, int32_t ld, int64_t B, uint32_t flags,
                                        int32_t *delta, int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev,
                                        cudaStream_t s, void (*mark)(int, cudaStream_t)) {
    const int C = HARD ? 2 : G0 + 1;
    const size_t smem_h = sizeof(unsigned int) * (size_t)C * ((size_t)ld + 1);
    if (smem_h > 48 * 1024 && cudaFuncSetAttribute(rank_count_kernel<HARD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)smem_h) != cudaSuccess)
        return HORA_ERR_CUDA;
    const int vec = ((reinterpret_cast<uintptr_t>(c) | reinterpret_cast<uintptr_t>(cap)) & 15u) == 0;
    const int per_sm = (int)std::fmax(1.0, std::fmin(8.0, std::floor(200.0 * 1024.0 / (double)(smem_h + 1024))));
    const int grid = clamp_grid((N + 8 * kSelThreads - 1) / (8 * kSelThreads), per_sm);
    launch_pdl(rank_count_kernel<HARD>, grid, kSelThreads, smem_h, s, c, G0, cap, cap_scalar, N, ld, B, flags, vec, w);
    if (mark) { mark(2, s); mark(3, s); }
    const size_t smem_c = sizeof(int32_t) * (size_t)C;
    const int warps = kSelThreads / kWarp;
    const int64_t NT = (N + kRankTask - 1) / kRankTask;
    int grid_b = clamp_grid((NT + warps - 1) / warps, 3);       // what the output pass keeps resident
    if (grid_b > kRankMaxCtas) grid_b = kRankMaxCtas;
    const int64_t m = (NT + grid_b - 1) / grid_b;            // tasks per CTA, a contiguous run
    launch_pdl(rank_sums_kernel, grid_b, kSelThreads, smem_c, s, c, C, HARD ? 1 : 0, cap, cap_scalar, N, vec, w, NT, m);
    if (mark) { mark(4, s); mark(5, s); }
    const int out_vec = ((reinterpret_cast<uintptr_t>(delta) | reinterpret_cast<uintptr_t>(G) |
                          reinterpret_cast<uintptr_t>(group_offsets)) & 15u) == 0;
    launch_pdl(rank_out_kernel, grid_b, kSelThreads, smem_c, s, c, G0, C, HARD ? 1 : 0, cap, cap_scalar, N, B, vec, w, NT, m,
               delta, G, group_offsets, out_vec, info_dev);
    if (mark) mark(6, s);
    return cuda_ok(cudaGetLastError());
}

hora_status_t launch_rank_allocate(double alpha0, double beta0, const int32_t *c, int32_t G0, const int32_t *cap,
                                   int32_t cap_scalar, int64_t N, int32_t ld, int64_t B, uint32_t flags, int32_t *delta,
                                   int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev, void *workspace,
                                   size_t workspace_bytes, cudaStream_t s, void (*mark)(int, cudaStream_t)) {
    const RankWorkspace w = rank_carve(workspace, N, G0, ld);
    if (workspace_bytes < w.bytes) return HORA_ERR_WORKSPACE;
    if (cudaMemsetAsync(w.hdr, 0, w.zero_bytes, s) != cudaSuccess) return HORA_ERR_CUDA;
    mark(0, s);
    const int tl = launch_rank_tables(alpha0, beta0, G0, ld, (flags & HORA_FLAG_EXACT_INT) != 0, w.tab, &w.hdr->status, s);
    if (tl < 0) return HORA_ERR_CUDA;
    mark(1, s);
    count_launches(tl + 3);
    return launch_rank_passes<false>(w, c, G0, cap, cap_scalar, N, ld, B, flags, delta, G, group_offsets, info_dev, s, mark);
}

// ---------------------------------------------------------------------------------------------------
// Batched: a warp per segment.

__global__ void __launch_bounds__(kSelThreads)
rank_batched_kernel(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                    int32_t ld, const int64_t *__restrict__ seg_off, const int64_t *__restrict__ budgets, int64_t S,
                    uint32_t flags, RankTables t, const int32_t *__restrict__ table_status, int32_t *__restrict__ delta,
                    int32_t *__restrict__ G, hora_alloc_info *__restrict__ info) {
    const int lane = lane_id();
    const int T = (G0 + 1) * ld;
    const int32_t tstat = table_status ? *table_status : 0;
    const int64_t warp0 = (int64_t)blockIdx.x * (kSelThreads / kWarp) + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * (kSelThreads / kWarp);
    for (int64_t s = warp0; s < S; s += n_warps) {
        const int64_t r0 = __ldg(seg_off + s);
        const int64_t n = __ldg(seg_off + s + 1) - r0;
        const long long B = __ldg(budgets + s);
        // prompts of the segment, 32 at a time; segments of at most 32 prompts (the paper's 15) stay in registers
        const bool small = n <= kWarp;
        int my_c = 0, my_cap = 0;
        bool bad = false;
        long long sum_cap = 0;
        for (int64_t i0 = 0; i0 < n; i0 += kWarp) {
            const int64_t i = i0 + lane;
            int ci = 0, cp = 0;
            if (i < n) {
                ci = __ldg(c + r0 + i);
                cp = cap ? __ldg(cap + r0 + i) : cap_scalar;
                if (ci < 0 || ci > G0 || cp < 0 || cp > ld) { bad = true; ci = 0; cp = 0; }
            }
            sum_cap += cp;
            if (small) { my_c = ci; my_cap = cp; }
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) sum_cap += __shfl_xor_sync(kFull, sum_cap, d);
        int status = tstat;
        if (!status && (__any_sync(kFull, bad) || B < 0)) status = HORA_ERR_INVALID_VALUE;
        if (!status && B > sum_cap) status = HORA_ERR_INFEASIBLE;
        // candidates of the segment whose rank is below r: sum_i min(cap_i, pos[c_i][r])
        auto count_below = [&](int r) -> long long {
            if (small) {
                const int p = (int)__ldg(&HORA_AT(t.pos, (size_t)my_c * (T + 1) + r, (size_t)(G0 + 1) * (T + 1)));
                return (long long)__reduce_add_sync(kFull, p < my_cap ? p : my_cap);
            }
            long long part = 0;
            for (int64_t i = lane; i < n; i += kWarp) {
                const int ci = __ldg(c + r0 + i);
                const int cp = cap ? __ldg(cap + r0 + i) : cap_scalar;
                const int p = (int)__ldg(&HORA_AT(t.pos, (size_t)ci * (T + 1) + r, (size_t)(G0 + 1) * (T + 1)));
                part += p < cp ? p : cp;
            }
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(kFull, part, d);
            return part;
        };
        int rstar = -1;
        long long above = 0, n_tied = 0;
        if (!status && B > 0) {
            int lo = 0, hi = T - 1;                          // smallest r with #{rank <= r} >= B
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (count_below(mid + 1) >= B) hi = mid; else lo = mid + 1;
            }
            rstar = lo;
            above = count_below(rstar);
            n_tied = count_below(rstar + 1) - above;
        }
        const long long R = B - above;
        // outputs: the first R tied prompts in index order take one more
        double obj = 0.0;
        long long pre_t = 0;
        for (int64_t i0 = 0; i0 < n; i0 += kWarp) {
            const int64_t i = i0 + lane;
            int ci = my_c, cp = my_cap;
            if (!small && i < n) {
                ci = __ldg(c + r0 + i);
                cp = cap ? __ldg(cap + r0 + i) : cap_scalar;
            }
            int hi_i = 0, tied_i = 0;
            if (i < n && rstar >= 0) {
                const int p0 = (int)__ldg(t.pos + (size_t)ci * (T + 1) + rstar);
                const int p1 = (int)__ldg(t.pos + (size_t)ci * (T + 1) + rstar + 1);
                hi_i = p0 < cp ? p0 : cp;
                tied_i = (p1 < cp ? p1 : cp) - hi_i;
            }
            const unsigned tmask = __ballot_sync(kFull, tied_i != 0);
            const long long before = pre_t + __popc(tmask & ((1u << lane) - 1u));
            const int d_i = hi_i + ((tied_i && before < R) ? 1 : 0);
            if (i < n) {
                delta[r0 + i] = status ? 0 : d_i;
                G[r0 + i] = status ? 0 : G0 + d_i;
                if (!status && !(flags & HORA_FLAG_SKIP_OBJECTIVE))
                    obj += __ldg(&HORA_AT(t.util, (size_t)ci * (ld + 1) + d_i, (size_t)(G0 + 1) * (ld + 1)));
            }
            pre_t += __popc(tmask);
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) obj += __shfl_xor_sync(kFull, obj, d);
        if (lane == 0 && info != nullptr) {
            hora_alloc_info o;
            o.status = status;
            o.first_pass_bits = 0;
            o.lambda = (status || rstar < 0) ? 0.0 : __ldg(t.lam + rstar);
            o.n_above = status ? 0 : above;
            o.n_tied = status ? 0 : n_tied;
            o.n_tied_taken = status ? 0 : R;
            o.objective = status ? 0.0 : obj;
            o.sum_G = status ? 0 : n * (long long)G0 + B;
            o.sum_cap = sum_cap;
            info[s] = o;
        }
    }
}

hora_status_t launch_rank_batched(const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar, int32_t ld,
                                  const int64_t *seg_off_dev, const int64_t *budgets_dev, int64_t S, uint32_t flags,
                                  const RankTables &t, const int32_t *table_status, int32_t *delta, int32_t *G,
                                  hora_alloc_info *info_dev, cudaStream_t s) {
    const int warps = kSelThreads / kWarp;
    const int grid = clamp_grid((S + warps - 1) / warps, 8);
    rank_batched_kernel<<<grid, kSelThreads, 0, s>>>(c, G0, cap, cap_scalar, ld, seg_off_dev, budgets_dev, S, flags, t,
                                                     table_status, delta, G, info_dev);
    return cuda_ok(cudaGetLastError());
}

// N == 0 for the hard-first call: nothing to hand out
__global__ void hard_first_empty(int64_t B, int64_t *offsets, hora_alloc_info *info) {
    if (offsets) offsets[0] = 0;
    if (info) {
        info->status = B > 0 ? HORA_ERR_INFEASIBLE : HORA_OK;
        info->first_pass_bits = 0;
        info->lambda = 0.0;
        info->n_above = info->n_tied = info->n_tied_taken = 0;
        info->objective = 0.0;
        info->sum_G = 0;
        info->sum_cap = 0;
    }
}

}  // namespace hora

extern "C" size_t hora_allocate_hard_first_workspace_bytes(int64_t N, int32_t ld) {
    if (N < 0 || ld < 1 || ld > hora::kRankMaxTypes) return 0;
    return hora::rank_carve(nullptr, N, 1, ld).bytes;       // two classes; the table area (a few KB) stays unused
}

extern "C" hora_status_t hora_allocate_hard_first(const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                                                  int64_t N, int32_t ld, int64_t B, int32_t *delta, int32_t *G,
                                                  int64_t *group_offsets, hora_alloc_info *info_dev, void *workspace,
                                                  size_t workspace_bytes, void *stream) {
    using namespace hora;
    if (N < 0 || N > 0x7FFFFFFFll || ld < 1 || ld > kRankMaxTypes || G0 < 0 || B < 0) return HORA_ERR_INVALID_ARG;
    if (cap == nullptr && (cap_scalar < 0 || cap_scalar > ld)) return HORA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (N == 0) {
        hard_first_empty<<<1, 1, 0, s>>>(B, group_offsets, info_dev);
        count_launches(1);
        return cuda_ok(cudaGetLastError());
    }
    if (c == nullptr || delta == nullptr || G == nullptr) return HORA_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HORA_ERR_WORKSPACE;
    const RankWorkspace w = rank_carve(workspace, N, 1, ld);
    if (workspace_bytes < w.bytes) return HORA_ERR_WORKSPACE;
    if (cudaMemsetAsync(w.hdr, 0, w.zero_bytes, s) != cudaSuccess) return HORA_ERR_CUDA;
    count_launches(3);
    return launch_rank_passes<true>(w, c, G0, cap, cap_scalar, N, ld, B, HORA_FLAG_SKIP_OBJECTIVE, delta, G, group_offsets,
                                    info_dev, s, nullptr);
}
