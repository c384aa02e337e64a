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
//   sums/out two passes over (c_i, cap_i) again: block sums of (above, tied) and their scan, then Delta, G and
//            the CSR offsets with the first R tied prompts in index order taking one more.
//
// The batched form (hora_allocate_batched with the same kind of prior) ranks once for all segments and gives a
// warp to each segment: the threshold rank is bisected with a table pos[c][r] = #{Delta : rank_c(Delta) < r}, so
// one step costs one lookup per prompt and one warp reduction.
#include <cmath>

#include "hora_block.cuh"
#include "hora_exact.cuh"
#include "hora_gains_chunk.cuh"
#include "hora_rank.cuh"

namespace hora {

constexpr double kRankBand = 9.313225746154785e-10;       // 2^-30

static inline size_t rk_align(size_t x) { return (x + 255) & ~(size_t)255; }

bool rank_route_applies(double alpha0, double beta0, int32_t G0, int32_t ld) {
    if (!(alpha0 >= 1.0 && beta0 >= 1.0 && alpha0 == std::floor(alpha0) && beta0 == std::floor(beta0))) return false;
    if (G0 < 0 || ld < 1) return false;
    const double top = alpha0 + beta0 + (double)G0 + (double)ld;
    if (top >= 1048576.0) return false;
    if ((int64_t)(G0 + 1) * (int64_t)ld > kRankMaxTypes) return false;
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

// sign of g_{a1,b1}(D1) - g_{a2,b2}(D2) on exact fractions; *overflow is set when 512 bits do not suffice
__device__ __noinline__ int exact_compare_types(unsigned long long a1, unsigned long long b1, unsigned long long D1,
                                                unsigned long long a2, unsigned long long b2, unsigned long long D2,
                                                bool *overflow) {
    UBig n1, d1, n2, d2;
    if (!exact_gain(a1, b1, D1, n1, d1) || !exact_gain(a2, b2, D2, n2, d2)) {
        *overflow = true;
        return 0;
    }
    return cmp_products(n1, d2, n2, d1);
}

// Every CTA builds the whole table of fp64 gains in shared memory (a warp per class row: a few hundred
// instructions), then a thread ranks one type.
template <int E>
__global__ void __launch_bounds__(kSelThreads)
rank_table_kernel(double alpha0, double beta0, int32_t G0, int32_t ld, RankTables t, int32_t *status) {
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
            if (x > up) above = true;
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
            if (x <= up && x >= dn) {
                if (tie_seen || exact_compare_types(a2, b2, (unsigned long long)lo + 1, a, b, (unsigned long long)j + 1, &overflow) == 0)
                    first_of_class = false;
            }
        }
    }
    if (overflow) raise_status(status, HORA_ERR_EXACT_RANGE);
    t.rank[id] = rank;
    t.gain[id] = g0;
    if (first_of_class) t.lam[rank] = g0;
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

int launch_rank_tables(double alpha0, double beta0, int32_t G0, int32_t ld, const RankTables &t, int32_t *status,
                       cudaStream_t s) {
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
    if (ld > 128) ok = go(rank_table_kernel<8>);
    else if (ld > 64) ok = go(rank_table_kernel<4>);
    else ok = go(rank_table_kernel<2>);
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
    long long *bsum_hi, *bsum_t;       // [NB]
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
    const int64_t NB = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    w.bins = rank_bins(G0, ld);
    size_t o = 0;
    char *p = static_cast<char *>(base);
    auto take = [&](size_t n) { char *q = p ? p + o : nullptr; o = rk_align(o + n); return q; };
    w.hdr = reinterpret_cast<RankHeader *>(take(sizeof(RankHeader)));
    w.H = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * C * ((size_t)ld + 1)));
    w.bucket = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * (size_t)w.bins));
    w.zero_bytes = o;                                        // everything before this is cleared per call
    w.bsum_hi = reinterpret_cast<long long *>(take(sizeof(long long) * (size_t)(NB > 0 ? NB : 1)));
    w.bsum_t = reinterpret_cast<long long *>(take(sizeof(long long) * (size_t)(NB > 0 ? NB : 1)));
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
    const size_t T = kRankMaxTypes, NB = (size_t)((N + kRowsPerBlock - 1) / kRowsPerBlock) + 1;
    // C (ld + 1) <= 2 T, C <= T, bins <= T; each array rounded up to 256 bytes
    return rk_align(sizeof(RankHeader)) + rk_align(8 * 2 * T) + rk_align(8 * T) + 2 * rk_align(8 * NB) + rk_align(4 * T) +
           rk_align(4 * T) + rk_align(8 * T) + rk_align(8 * 2 * T) + rk_align(8 * T) + 4096;
}

// (c_i, cap_i) of prompt i, validated; bin = -1 for an invalid or missing prompt
__device__ __forceinline__ int rank_bin(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap,
                                        int32_t cap_scalar, int32_t ld, int64_t i, int64_t N, bool *bad) {
    if (i >= N) return -1;
    const int32_t ci = __ldg(c + i);
    const int32_t cp = cap ? __ldg(cap + i) : cap_scalar;
    if (ci < 0 || ci > G0 || cp < 0 || cp > ld) { *bad = true; return -1; }
    return ci * (ld + 1) + cp;
}

__global__ void __launch_bounds__(kSelThreads)
rank_count_kernel(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                  int64_t N, int32_t ld, int64_t B, uint32_t flags, RankWorkspace w) {
    extern __shared__ __align__(16) unsigned char s_rank_cnt[];
    unsigned int *s_hist = reinterpret_cast<unsigned int *>(s_rank_cnt);
    __shared__ long long s_warp[kSelThreads / kWarp];
    __shared__ double s_obj[kSelThreads / kWarp];
    const int C = G0 + 1, n_h = C * (ld + 1);
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    for (int b = threadIdx.x; b < n_h; b += kSelThreads) s_hist[b] = 0;
    __syncthreads();
    bool bad = false;
    const int64_t stride = (int64_t)gridDim.x * kSelThreads * 4;
    for (int64_t base = (int64_t)blockIdx.x * kSelThreads * 4; base < N; base += stride) {
        int bin[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) bin[u] = rank_bin(c, G0, cap, cap_scalar, ld, base + u * kSelThreads + threadIdx.x, N, &bad);
#pragma unroll
        for (int u = 0; u < 4; ++u) {                       // one shared-memory update per distinct bin per warp
            const unsigned peers = __match_any_sync(kFull, bin[u]);
            if (bin[u] >= 0 && lane == __ffs(peers) - 1) atomicAdd(&s_hist[bin[u]], (unsigned)__popc(peers));
        }
    }
    if (bad) raise_status(&w.hdr->status, HORA_ERR_INVALID_VALUE);
    __syncthreads();
    for (int b = threadIdx.x; b < n_h; b += kSelThreads) {
        const unsigned int v = s_hist[b];
        if (v) atomicAdd(w.H + b, (unsigned long long)v);
    }
    if (!last_block(&w.hdr->ticket[0])) return;

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
            if (D >= 1 && cnt > 0) atomicAdd(w.bucket + (w.bins - 1 - __ldg(rrow + D - 1)), (unsigned long long)cnt);
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

// (candidates above the threshold, tied candidate) of a prompt from its class entry
__device__ __forceinline__ void rank_row_state(int bin, int32_t ld, const int32_t *s_class, int *hi, int *tied) {
    *hi = 0;
    *tied = 0;
    if (bin < 0) return;
    const int cls = bin / (ld + 1), cp = bin - cls * (ld + 1);
    const int e = s_class[cls], above = e >> 1;
    *hi = cp < above ? cp : above;
    *tied = (e & 1) && cp > above;
}

// Block sums of (above, tied) over blocks of kRowsPerBlock prompts; the last CTA scans them.
__global__ void __launch_bounds__(kSelThreads)
rank_sums_kernel(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                 int64_t N, int32_t ld, RankWorkspace w, int64_t NB) {
    extern __shared__ __align__(16) unsigned char s_rank_cls[];
    int32_t *s_class = reinterpret_cast<int32_t *>(s_rank_cls);
    __shared__ long long s_warp[kSelThreads / kWarp];
    const bool failed = *(volatile int32_t *)&w.hdr->status != 0;
    long long hi_sum = 0, t_sum = 0;
    if (!failed) {
        for (int k = threadIdx.x; k <= G0; k += kSelThreads) s_class[k] = w.class_tab[k];
        __syncthreads();
        const int64_t row0 = (int64_t)blockIdx.x * kRowsPerBlock + (int64_t)threadIdx.x * 4;
        bool bad = false;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int hi, tied;
            rank_row_state(rank_bin(c, G0, cap, cap_scalar, ld, row0 + q, N, &bad), ld, s_class, &hi, &tied);
            hi_sum += hi;
            t_sum += tied;
        }
    }
    long long tot_hi, tot_t;
    block_exclusive_sum(hi_sum, &tot_hi, s_warp);
    block_exclusive_sum(t_sum, &tot_t, s_warp);
    if (threadIdx.x == 0) { w.bsum_hi[blockIdx.x] = tot_hi; w.bsum_t[blockIdx.x] = tot_t; }
    if (last_block(&w.hdr->ticket[1])) {
        long long run_hi = 0, run_t = 0;
        scan_block_sums(w.bsum_hi, w.bsum_t, 0, NB, nullptr, nullptr, run_hi, run_t, s_warp);
    }
}

// Outputs: a thread owns four consecutive prompts (16-byte stores where the arrays allow: `vec`).
__global__ void __launch_bounds__(kSelThreads)
rank_out_kernel(const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                int64_t N, int32_t ld, int64_t B, RankWorkspace w, int32_t *__restrict__ delta, int32_t *__restrict__ G,
                int64_t *__restrict__ offsets, int vec, hora_alloc_info *info) {
    extern __shared__ __align__(16) unsigned char s_rank_cls[];
    int32_t *s_class = reinterpret_cast<int32_t *>(s_rank_cls);
    __shared__ long long s_warp[kSelThreads / kWarp];
    const RankHeader *hdr = w.hdr;
    const int32_t status = *(volatile int32_t *)&hdr->status;
    const bool failed = status != 0;
    if (!failed)
        for (int k = threadIdx.x; k <= G0; k += kSelThreads) s_class[k] = w.class_tab[k];
    __syncthreads();
    const int64_t row0 = (int64_t)blockIdx.x * kRowsPerBlock + (int64_t)threadIdx.x * 4;
    const bool whole = row0 + 4 <= N;
    int hi[4], tied[4];
    long long hi_sum = 0, t_sum = 0;
    bool bad = false;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        hi[q] = tied[q] = 0;
        if (!failed) rank_row_state(rank_bin(c, G0, cap, cap_scalar, ld, row0 + q, N, &bad), ld, s_class, &hi[q], &tied[q]);
        hi_sum += hi[q];
        t_sum += tied[q];
    }
    const long long blk_hi = failed ? 0 : w.bsum_hi[blockIdx.x], blk_t = failed ? 0 : w.bsum_t[blockIdx.x];
    const long long R = failed ? 0 : hdr->R;
    long long th, tt;
    long long pre_hi = blk_hi + block_exclusive_sum(hi_sum, &th, s_warp);
    long long pre_t = blk_t + block_exclusive_sum(t_sum, &tt, s_warp);
    int32_t d[4];
    int64_t of[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        d[q] = hi[q] + ((tied[q] && pre_t < R) ? 1 : 0);
        of[q] = failed ? 0 : (row0 + q) * (int64_t)G0 + pre_hi + (pre_t < R ? pre_t : R);
        pre_hi += hi[q];
        pre_t += tied[q];
    }
    if (whole && vec) {
        *reinterpret_cast<int4 *>(delta + row0) = make_int4(d[0], d[1], d[2], d[3]);
        *reinterpret_cast<int4 *>(G + row0) = failed ? make_int4(0, 0, 0, 0) : make_int4(G0 + d[0], G0 + d[1], G0 + d[2], G0 + d[3]);
        if (offsets) {
            *reinterpret_cast<longlong2 *>(offsets + row0) = make_longlong2(of[0], of[1]);
            *reinterpret_cast<longlong2 *>(offsets + row0 + 2) = make_longlong2(of[2], of[3]);
        }
    } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (row0 + q < N) {
                delta[row0 + q] = d[q];
                G[row0 + q] = failed ? 0 : G0 + d[q];
                if (offsets) offsets[row0 + q] = of[q];
            }
        }
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == kSelThreads - 1) {
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

hora_status_t launch_rank_allocate(double alpha0, double beta0, const int32_t *c, int32_t G0, const int32_t *cap,
                                   int32_t cap_scalar, int64_t N, int32_t ld, int64_t B, uint32_t flags, int32_t *delta,
                                   int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev, void *workspace,
                                   size_t workspace_bytes, cudaStream_t s, void (*mark)(int, cudaStream_t)) {
    const RankWorkspace w = rank_carve(workspace, N, G0, ld);
    if (workspace_bytes < w.bytes) return HORA_ERR_WORKSPACE;
    const int64_t NB = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    const int C = G0 + 1;
    if (cudaMemsetAsync(w.hdr, 0, w.zero_bytes, s) != cudaSuccess) return HORA_ERR_CUDA;
    mark(0, s);
    const int tl = launch_rank_tables(alpha0, beta0, G0, ld, w.tab, &w.hdr->status, s);
    if (tl < 0) return HORA_ERR_CUDA;
    mark(1, s);
    const size_t smem_h = sizeof(unsigned int) * (size_t)C * ((size_t)ld + 1);
    if (smem_h > 48 * 1024 &&
        cudaFuncSetAttribute(rank_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_h) != cudaSuccess)
        return HORA_ERR_CUDA;
    const int per_sm = smem_h > 32 * 1024 ? 2 : 4;
    const int grid = clamp_grid((N + 4 * kSelThreads - 1) / (4 * kSelThreads), per_sm);
    rank_count_kernel<<<grid, kSelThreads, smem_h, s>>>(c, G0, cap, cap_scalar, N, ld, B, flags, w);
    mark(2, s);
    mark(3, s);
    const size_t smem_c = sizeof(int32_t) * (size_t)C;
    rank_sums_kernel<<<(int)NB, kSelThreads, smem_c, s>>>(c, G0, cap, cap_scalar, N, ld, w, NB);
    mark(4, s);
    mark(5, s);
    const int out_vec = ((reinterpret_cast<uintptr_t>(delta) | reinterpret_cast<uintptr_t>(G) |
                          reinterpret_cast<uintptr_t>(group_offsets)) & 15u) == 0;
    rank_out_kernel<<<(int)NB, kSelThreads, smem_c, s>>>(c, G0, cap, cap_scalar, N, ld, B, w, delta, G, group_offsets,
                                                        out_vec, info_dev);
    mark(6, s);
    count_launches(tl + 3);
    return cuda_ok(cudaGetLastError());
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
                const int p = (int)__ldg(t.pos + (size_t)my_c * (T + 1) + r);
                return (long long)__reduce_add_sync(kFull, p < my_cap ? p : my_cap);
            }
            long long part = 0;
            for (int64_t i = lane; i < n; i += kWarp) {
                const int ci = __ldg(c + r0 + i);
                const int cp = cap ? __ldg(cap + r0 + i) : cap_scalar;
                const int p = (int)__ldg(t.pos + (size_t)ci * (T + 1) + r);
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
                if (!status && !(flags & HORA_FLAG_SKIP_OBJECTIVE)) obj += __ldg(t.util + (size_t)ci * (ld + 1) + d_i);
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

}  // namespace hora
