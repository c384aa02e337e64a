// hora_allocate: the B largest marginal gains over all (prompt, Delta) candidates, i.e. the result of
// Algorithm 1's Phase-B greedy loop (Proposition 1), found by selection instead of B sequential steps.
//
// Keys.  A gain is a non-negative finite double, so its bit pattern orders like the value.  The 64-bit
// key of the B-th largest gain is resolved from the top, a digit at a time:
//
//   estimate  every S-th row (about 4096 rows) is read and histogrammed on the top 13 bits; the scaled rank
//             says in which two adjacent 13-bit bins the threshold almost surely lies (the "window"), and,
//             interpolated inside its bin, roughly where: a guessed threshold.
//   level 0   one coalesced read of the whole matrix (a warp per row-item, two items in flight).  Only the
//             window is looked at closely: keys inside it are counted per 23-bit bin (2048 fine bins in
//             shared memory), keys above the guess are counted per row (stored for level 1) and in all.
//             The last CTA to finish knows from those counts whether the B-th key lies inside the window
//             and, if so, its 23-bit prefix.  If not (a sample that misleads), a plain pass histograms
//             every key on 13 bits and the selection goes on from there.  The full read also validates the
//             rows and sums the caps.
//   level 1   a thread per row: a row is non-increasing, so its keys with the resolved prefix form ONE
//             contiguous segment [p_hi, p_lo), and p_hi is within a key or two of the stored guess: the
//             thread reads the eight keys around the guess (widening, then a binary search over the row, if
//             they do not settle it) and stores the segment.  The same pass validates the priors and
//             evaluates the utility of every row whose segment is empty (its Delta is final).
//   tail      ONE cooperative launch finishes the threshold and the prefixes over prompts:
//     list    at most 65536 such keys (the usual case after a window hit): level 1 appended them to a list
//             and accumulated per-block sums of its provisional counts; one CTA resolves the remaining bits
//             over the list, corrects the block sums by the listed keys above / equal to the threshold and
//             scans them.  No further pass over rows.
//     digits  more than that (a missed window, or heavy ties): level 1 histogrammed the next 13 bits and
//             listed the rows whose segment is not empty; all CTAs narrow the listed rows' segments digit by
//             digit (13 bits at a time, a grid-wide barrier between levels), close them with the finished
//             threshold, form the block sums and scan them.  If level 1 found every key of the threshold's bin
//             to be one value (a mass tie), that value is the threshold and the digit levels are skipped.
//   out       p_hi = #keys > lambda, tied = #keys == lambda per row (segments left open by the list route are
//             closed here); Delta_i = p_hi + (tied candidates of row i that fall within the first
//             R = B - n_above tied candidates in prompt order); G_i, CSR offsets, objective.
//
// Outside the cooperative tail no kernel waits on another CTA: every "last CTA" step uses an atomic ticket
// after a fence; inside it the only waits are the runtime's grid-wide barriers.
//
// Exact mode (integer priors).  After the fp64 selection, candidates within a relative band of 2^-30
// around lambda (far wider than the fp64 evaluation error, far narrower than the gap between two
// entries of one row) are the only ones whose exact rank is in doubt.  Each row has at most one.
// Their types (a, b, Delta) are collected in a small hash table with instance counts, ranked exactly
// by cross multiplication in 1024-bit integers of num/den = a (b)_a / (b+Delta-1)_{a+1}  (or the equivalent
// a (b)_{Delta-1} / (a+b)_Delta when that has fewer factors), and the threshold class is found by
// walking the ranked types.  Rows are relabelled above / tied / below and the same sum/out steps run.
//
// One prior for all prompts and no matrix given: none of the above runs.  The at most
// (G0 + 1) * ld distinct candidate values are ranked once and the selection works on ranks and on counts of
// (c_i, cap_i): hora_rank.cu.
#include <cooperative_groups.h>

#include <atomic>
#include <type_traits>

#define HORA_FILE_ID 1
#include "hora_block.cuh"
#include "hora_checked.cuh"
#include "hora_common.cuh"
#include "hora_exact.cuh"
#include "hora_gains_chunk.cuh"
#include "hora_rank.cuh"

HORA_CHECKED_REGISTER()

namespace hora {

constexpr int kLevels = 5;                   // level 0 (full read) + four digit levels
constexpr int kListCap = 65536;              // candidates the single-CTA list selection accepts
constexpr int kListSmall = 1536;               // keys of the list that later sweeps keep in shared memory
constexpr int kTailPerSm = 4;                 // CTAs of the cooperative tail per SM
constexpr int kLevel1PerSm = 5;               // CTAs of level 1 per SM: the grid is exactly one resident wave (a sixth
                                              // CTA per SM that has to wait for a slot cost 25 us of 77 at 2^20 rows)
constexpr int kBins = 8192;                  // 13-bit digits
constexpr int kDigitBits = 13;
constexpr int kWinBins = 2;                  // coarse bins covered by the fine window of level 0
constexpr int kFineBits = 10;                // extra bits resolved inside the window
constexpr int kFinePerBin = 1 << kFineBits;
constexpr int kFineBins = kWinBins * kFinePerBin;
constexpr int kSampleRows = 4096;            // rows read by the estimate pass
constexpr int kTypeSlots = 4096;             // hash slots for exact tie types
constexpr int kMaxTypes = 1024;              // distinct types the exact ranking accepts
constexpr unsigned long long kKeyInf = 0x7FF0000000000000ull;

struct AllocHeader {
    int32_t status;
    int32_t resolved;                  // key bits resolved so far, from the top
    unsigned int ticket[16];
    unsigned long long sum_cap;
    unsigned long long sum_pguess;     // keys above the guessed threshold, over all rows
    unsigned long long prefix_key;     // the resolved bits in place (the threshold once all 64 are resolved)
    long long need;                    // rank of the threshold inside the current bin (1-based)
    int32_t lv_shift[8], lv_bits[8], sel_digit[8];   // per level: position, width and value of its digit
    int32_t win_lo;                    // first 13-bit bin of level 0's fine window
    unsigned int guess_hi;             // guessed threshold: a key counts as "above" when its high word exceeds this
    unsigned int n_active;             // rows with a non-empty segment after level 1
    int32_t l0_miss;                   // 1: the B-th key is not inside level 0's window (the plain 13-bit pass runs)
    unsigned long long sample_cap;     // sum of the caps of the sampled rows
    unsigned long long n_above, n_tied;
    long long R;                       // tied candidates to take
    double lambda;
    double objective;
    unsigned long long band_above;     // exact mode: candidates above the band
    unsigned int n_types;
    unsigned int n_cand;               // list mode: keys appended by level 1
    long long bin_count;               // keys that carry the prefix resolved so far
    int32_t list_mode;                 // 1: the keys of level 1's segments go to the candidate list
    int32_t pad1;
    unsigned long long seg_ref;        // digit route: the first segment key any thread of level 1 registered
    int32_t seg_differs;               // digit route: 1 if some segment key differs from seg_ref
    int32_t pad2;
};

struct Workspace {
    AllocHeader *hdr;
    unsigned long long *hist_est;      // [kBins] estimate pass
    unsigned long long *hist_coarse;   // [kBins] level 0, 13-bit bins outside the window
    unsigned long long *hist_fine;     // [kFineBins] level 0, 23-bit bins inside the window
    unsigned long long *hist_lv;       // [kLevels][kBins] levels 1..4 (slot 0 unused)
    int2 *rowstate;                    // [N] (p_hi, p_lo)
    unsigned int *pguess;              // [N] keys of the row above the guessed threshold
    int32_t *active;                   // [N] rows with a non-empty segment
    long long *bsum_hi, *bsum_t;       // [NB] sums over blocks of kRowsPerBlock prompts, overwritten by exclusive prefixes
    double *objpart;                   // [NB]
    unsigned long long *tkeys, *tcounts;   // [kTypeSlots]
    int32_t *tlabel;                   // [kTypeSlots]
    int32_t *rowslot;                  // [N]
    unsigned long long *cand_key;      // [kListCap] list mode: every key that carries level 0's prefix
    int32_t *cand_row;                 // [kListCap] and its row
    double *objrow;                    // [N] U_i(Delta_i) where level 1 could evaluate it, else negative
    double *gains;                     // [N*ld] when the caller passed none
    size_t bytes;
};

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static Workspace carve(void *base, int64_t N, int32_t ld, bool need_gains, bool exact) {
    Workspace w{};
    size_t o = 0;
    char *p = static_cast<char *>(base);
    const int64_t NB = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    auto take = [&](size_t n) { char *q = p ? p + o : nullptr; o = align256(o + n); return q; };
    w.hdr = reinterpret_cast<AllocHeader *>(take(sizeof(AllocHeader)));
    w.hist_est = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kBins));
    w.hist_coarse = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kBins));
    w.hist_fine = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kFineBins));
    w.hist_lv = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kLevels * kBins));
    w.bsum_hi = reinterpret_cast<long long *>(take(sizeof(long long) * (size_t)NB));
    w.bsum_t = reinterpret_cast<long long *>(take(sizeof(long long) * (size_t)NB));
    w.rowstate = reinterpret_cast<int2 *>(take(sizeof(int2) * (size_t)N));          // everything before this is zeroed per call
    w.pguess = reinterpret_cast<unsigned int *>(take(sizeof(unsigned int) * (size_t)N));
    w.active = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (size_t)N));
    w.objpart = reinterpret_cast<double *>(take(sizeof(double) * (size_t)NB));
    w.cand_key = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kListCap));
    w.cand_row = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * kListCap));
    w.objrow = reinterpret_cast<double *>(take(sizeof(double) * (size_t)N));
    if (exact) {
        w.tkeys = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kTypeSlots));
        w.tcounts = reinterpret_cast<unsigned long long *>(take(sizeof(unsigned long long) * kTypeSlots));
        w.tlabel = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * kTypeSlots));
        w.rowslot = reinterpret_cast<int32_t *>(take(sizeof(int32_t) * (size_t)N));
    }
    if (need_gains) w.gains = reinterpret_cast<double *>(take(sizeof(double) * (size_t)N * (size_t)ld));
    w.bytes = o;
    return w;
}

// Run by ONE CTA: select the next digit of the threshold from hist[0..bins), bins a power of two; the digit
// sits at bit `shift` of the key.  With `append` it extends the digit already recorded for `level` (the
// fine part of level 0) instead of starting a new one.
__device__ void find_digit(AllocHeader *hdr, const unsigned long long *hist, int bins, int bits, int shift, int level,
                           bool append, long long *s_warp) {
    long long above = 0, count = 0;
    const int digit = locate_rank(hist, bins, hdr->need, &above, &count, s_warp);
    if (digit >= 0 && threadIdx.x == 0) {
        hdr->sel_digit[level] = append ? ((hdr->sel_digit[level] << bits) | digit) : digit;
        hdr->lv_bits[level] = append ? hdr->lv_bits[level] + bits : bits;
        hdr->lv_shift[level] = shift;
        hdr->need -= above;
        hdr->prefix_key |= (unsigned long long)digit << shift;
        hdr->resolved += bits;
        hdr->bin_count = count;
    }
    __syncthreads();
}

__device__ __forceinline__ void flush_hist(const unsigned int *s_hist, unsigned long long *hist, int bins) {
    for (int b = threadIdx.x; b < bins; b += kSelThreads) {
        const unsigned int v = s_hist[b];
        if (v) atomicAdd(hist + b, (unsigned long long)v);
    }
}

// Width and position of the next digit once `resolved` bits are known.
__device__ __forceinline__ void next_digit(int resolved, int *bits, int *shift) {
    const int w = 64 - resolved < kDigitBits ? 64 - resolved : kDigitBits;
    *bits = w;
    *shift = 64 - resolved - w;
}

// Run by ONE CTA after the sample histogram is complete: scale the rank B to the sample and put the two-bin
// window around the bin it falls in — towards the upper neighbour when the rank falls in the upper half of
// that bin's count, else towards the lower one — and interpolate a guessed threshold inside that bin.  Both
// are hints: a poor one costs time, never correctness.
__device__ void place_window(AllocHeader *hdr, const unsigned long long *hist, int64_t B, int64_t n_sample, int64_t N,
                             long long *s_warp) {
    long long need = (long long)((double)B * (double)n_sample / (double)N + 0.5);
    const long long sample_cap = (long long)*(volatile unsigned long long *)&hdr->sample_cap;
    if (need < 1) need = 1;
    if (need > sample_cap) need = sample_cap;
    long long above = 0, count = 0;
    const int d = locate_rank(hist, kBins, need, &above, &count, s_warp);
    if (d >= 0 && threadIdx.x == 0) {
        const bool upper_half = 2 * (need - above) <= count;              // counting from the top of the bin
        int lo = upper_half ? d : d - 1;
        lo = lo < 0 ? 0 : (lo > kBins - kWinBins ? kBins - kWinBins : lo);
        hdr->win_lo = lo;
        // the guess: the rank's position inside bin d, counted from the top, on a linear scale of the key bits
        // (bin d holds the high words [d << 19, (d + 1) << 19))
        const double f = ((double)(need - above) - 0.5) / (double)(count > 0 ? count : 1);
        const unsigned int down = (unsigned int)(f * 524288.0);
        hdr->guess_hi = ((unsigned int)(d + 1) << 19) - (down < 524288u ? down : 524287u) - 1u;
    }
}

// ---------------------------------------------------------------------------------------------------
// Estimate: a warp per sampled row (every `every`-th row), histogram of the top 13 bits.  The last CTA
// scales the rank B to the sample and places the two-bin window around the bin it falls in: towards the
// upper neighbour when the rank falls in the upper half of that bin's count, else towards the lower one.
__global__ void __launch_bounds__(kSelThreads)
select_estimate(const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N, int32_t ld, int64_t every,
                const double *__restrict__ gains, int64_t B, AllocHeader *hdr, unsigned long long *hist) {
    pdl_enter();
    __shared__ unsigned int s_hist[kBins];
    __shared__ long long s_warp[kSelThreads / kWarp];
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) s_hist[b] = 0;
    __syncthreads();
    const int lane = lane_id();
    const int64_t n_sample = (N + every - 1) / every;
    const int64_t warp0 = (int64_t)blockIdx.x * (kSelThreads / kWarp) + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * (kSelThreads / kWarp);
    long long capsum = 0;
    for (int64_t sidx = warp0; sidx < n_sample; sidx += stride) {
        const int64_t row = sidx * every;
        int32_t capi = cap ? __ldg(cap + row) : cap_scalar;
        capi = capi < 0 ? 0 : (capi > ld ? ld : capi);
        if (lane == 0) capsum += capi;
        const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(gains) + row * (int64_t)ld;
        for (int32_t k0 = 0; k0 < capi; k0 += 8 * kWarp) {      // eight coalesced loads in flight per lane
            unsigned long long key[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int32_t j = k0 + u * kWarp + lane;
                key[u] = j < capi ? __ldg(keys + j) : 0ull;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (k0 + u * kWarp + lane < capi) atomicAdd(&s_hist[(int)(key[u] >> 51) & (kBins - 1)], 1u);
        }
    }
    __syncthreads();
    flush_hist(s_hist, hist, kBins);
    long long tot;
    block_exclusive_sum(capsum, &tot, s_warp);
    if (threadIdx.x == 0 && tot) atomicAdd(&hdr->sample_cap, (unsigned long long)tot);
    if (last_block(&hdr->ticket[15])) place_window(hdr, hist, B, n_sample, N, s_warp);
}

// ---------------------------------------------------------------------------------------------------
// Level 0: the one full read.  The matrix is cut into items of 32*E consecutive keys of one row; a warp
// takes one item at a time and a lane E consecutive keys of it, and the loads of the NEXT item are
// issued before the current one is processed.
//
// What is counted.  Only the window matters: the keys ABOVE it (one number) and the keys INSIDE it, per
// 23-bit bin (2048 fine bins in shared memory).  A row is sorted, so a 64-key slice of it lies wholly above the
// window, wholly below it, or (one or two slices of a 256-key row) needs a look at each key.  The per-key look
// also counts the keys above the guessed threshold; summed over the row that count is stored for level 1,
// and summed over everything it gives the number of keys above the window:
//     #above window = #above guess - #(window keys above the guess)      (the guess lies inside the window).
// The last CTA then knows whether the B-th key falls inside the window — almost always — and if so in which
// fine bin: 23 bits of the threshold.  If not, a second pass (select_level0_full) builds the plain 13-bit
// histogram of everything and the selection goes on from 13 bits.
// A histogram of all 8192 13-bit bins in the same pass was the first design; it cost an index computation and
// a shared-memory atomic for nearly every key (a row crosses some forty 13-bit bins), 2.4 times the
// instructions, and those, not memory, set the time.
// The pass also checks that the row is finite, non-negative and non-increasing and sums the caps.

// The window as the per-key code sees it: d = h - base is below `kFineBins << 9` exactly for the high words h of
// window keys (it wraps far above that for a key below the window; so does a key past the cap, which every caller
// presents as 0, unless the window is the lowest one: then such keys are kept out by their index), and a key is
// above the guess from the first pattern of the bin after the guess on.
struct WindowView {
    unsigned fine_shared;          // shared-window address of the fine histogram
    unsigned base;                 // first high word of the window
    unsigned above_from;           // first high word above the guess
    __device__ __forceinline__ void set(unsigned int *s_fine, unsigned W0, int t_guess) {
        fine_shared = (unsigned)__cvta_generic_to_shared(s_fine);
        base = W0 << 9;
        const unsigned long long g64 = ((unsigned long long)W0 + (unsigned)t_guess + 1ull) << 9;
        above_from = g64 > 0xFFFFFFFFull ? 0xFFFFFFFFu : (unsigned)g64;   // (no valid key is that high)
    }
};

// fine[d >> 9] += 1 where d < limit, as one predicated instruction (an `if` around the atomic compiled to a
// branch per key); the address is formed for every key and used only under the predicate
__device__ __forceinline__ void count_if_below(unsigned fine_shared, unsigned d, unsigned limit) {
    const unsigned addr = fine_shared + (d >> 9) * 4u;
    asm volatile("{\n .reg .pred p;\n setp.lt.u32 p, %1, %2;\n @p red.shared.add.u32 [%0], 1;\n}" ::"r"(addr), "r"(d), "r"(limit)
                 : "memory");
}

// E keys of one lane, as high words; the first `nvalid` exist, the rest are 0.  Counts the window keys in the fine
// histogram and returns how many keys are above the guess.  No branch but the one on the window's position.
template <int E>
__device__ __forceinline__ int window_count(const unsigned (&h)[E], int nvalid, const WindowView &wv) {
    int above = 0;
    auto count = [&](auto lowest) {
        constexpr bool kLowest = decltype(lowest)::value;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const unsigned d = h[j] - wv.base;
#ifdef HORA_CHECKED
            if ((!kLowest || j < nvalid) && d < ((unsigned)kFineBins << 9)) {
                unsigned int *fine = reinterpret_cast<unsigned int *>(__cvta_shared_to_generic(wv.fine_shared));
                atomicAdd(&HORA_AT(fine, d >> 9, kFineBins), 1u);
            }
#else
            count_if_below(wv.fine_shared, kLowest && j >= nvalid ? 0xFFFFFFFFu : d, (unsigned)kFineBins << 9);
#endif
            above += (h[j] >= wv.above_from) && (!kLowest || j < nvalid);
        }
    };
    if (wv.base != 0) count(std::false_type{}); else count(std::true_type{});
    return above;
}

// End of the full-read pass (shared by the pass that reads a materialised matrix and by the fused pass that
// produces the matrix): merge this CTA's window histogram, add up the caps and the counts above the guess, and
// let the last CTA locate the threshold's 23-bit prefix inside the window, or declare a miss.
__device__ void level0_finish(AllocHeader *hdr, unsigned long long *hist_fine, const unsigned int *s_fine, unsigned W0,
                              int t_guess, long long capsum, long long sum_pg, bool bad, int64_t B, long long *s_warp) {
    if (bad) raise_status(&hdr->status, HORA_ERR_INVALID_VALUE);
    __syncthreads();
    flush_hist(s_fine, hist_fine, kFineBins);
    long long tot;
    block_exclusive_sum(capsum, &tot, s_warp);
    if (threadIdx.x == 0 && tot) atomicAdd(&hdr->sum_cap, (unsigned long long)tot);
    block_exclusive_sum(sum_pg, &tot, s_warp);
    if (threadIdx.x == 0 && tot) atomicAdd(&hdr->sum_pguess, (unsigned long long)tot);
    if (last_block(&hdr->ticket[0])) {
        const unsigned long long sum_cap = *(volatile unsigned long long *)&hdr->sum_cap;
        const long long above_guess = (long long)*(volatile unsigned long long *)&hdr->sum_pguess;
        // window keys in all, and those above the guess
        long long part_all = 0, part_up = 0;
        for (int f = threadIdx.x; f < kFineBins; f += kSelThreads) {
            const long long v = (long long)__ldcg(hist_fine + f);
            part_all += v;
            if (f > t_guess) part_up += v;
        }
        long long in_window, up;
        block_exclusive_sum(part_all, &in_window, s_warp);
        block_exclusive_sum(part_up, &up, s_warp);
        const long long above_window = above_guess - up;
        const long long need_w = B - above_window;               // rank of the threshold inside the window
        const bool hit = B >= 1 && need_w >= 1 && need_w <= in_window;
        if (threadIdx.x == 0 && (unsigned long long)B > sum_cap) raise_status(&hdr->status, HORA_ERR_INFEASIBLE);
        long long above = 0, count = 0;
        const int t = hit ? locate_rank(hist_fine, kFineBins, need_w, &above, &count, s_warp) : -1;
        if (threadIdx.x == 0) {
            if (t >= 0) {
                const unsigned long long prefix23 = (unsigned long long)W0 + (unsigned long long)t;
                hdr->sel_digit[0] = (int32_t)prefix23;
                hdr->lv_bits[0] = kDigitBits + kFineBits;
                hdr->lv_shift[0] = 64 - (kDigitBits + kFineBits);
                hdr->need = need_w - above;
                hdr->prefix_key = prefix23 << (64 - (kDigitBits + kFineBits));
                hdr->resolved = kDigitBits + kFineBits;
                hdr->bin_count = count;
                hdr->list_mode = count <= (long long)kListCap ? 1 : 0;
            } else {
                hdr->need = B;
                hdr->l0_miss = B >= 1 ? 1 : 0;                   // the plain 13-bit pass takes over
            }
        }
    }
}

// One item in registers.  The item is cut into E/2 slices of 64 consecutive keys; of every slice a lane holds
// the pair of keys 2*lane, 2*lane + 1 (one 16-byte load, 512 contiguous bytes per warp instruction).  A slice is
// thus spread over all lanes, and one that lies wholly above or wholly below the window is settled by a vote
// instead of a look at each key; with E consecutive keys per lane the ten lanes of a row that intersect the
// window made every warp run the per-key code for all its keys (121 of 250 instructions per row).
template <int E>
struct Level0Item {
    ulonglong2 v[E / 2];           // slice p: keys k0 + 64 p + 2 lane, + 1
    unsigned long long before;     // lane 0 only: the key just before this item (or the largest finite key)
    int32_t capi;                  // the row's cap; -1 marks "no item"
};

template <int E, bool VEC2, bool ONE>
__device__ __forceinline__ void level0_fetch(Level0Item<E> &it, const int32_t *__restrict__ cap, int32_t cap_scalar,
                                             int64_t n_items, int32_t items_per_row, int32_t ld,
                                             const double *__restrict__ gains, int64_t item, int lane, bool *bad) {
    it.capi = -1;
    if (item >= n_items) return;
    const int64_t row = ONE ? item : item / items_per_row;     // ONE: an item is a whole row (no 64-bit division)
    const int32_t k0 = ONE ? 0 : (int32_t)(item - row * items_per_row) * (kWarp * E);
    int32_t capi = cap ? __ldg(cap + row) : cap_scalar;
    if (capi < 0 || capi > ld) { *bad = true; capi = 0; }
    it.capi = capi;
    const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(gains) + row * (int64_t)ld + k0 + 2 * lane;
    if (VEC2 && k0 + kWarp * E <= capi) {                      // the whole item lies below the cap: plain loads
#pragma unroll
        for (int p = 0; p < E / 2; ++p) it.v[p] = __ldg(reinterpret_cast<const ulonglong2 *>(keys) + 32 * p);
    } else {                                                   // ragged: keys past the cap read as 0
#pragma unroll
        for (int p = 0; p < E / 2; ++p) {
            const int32_t k = k0 + 64 * p + 2 * lane;
            it.v[p] = make_ulonglong2(0ull, 0ull);
            if (VEC2) {
                if (k < capi) {
                    it.v[p] = __ldg(reinterpret_cast<const ulonglong2 *>(keys) + 32 * p);
                    if (k + 1 >= capi) it.v[p].y = 0ull;
                }
            } else {
                if (k < capi) it.v[p].x = __ldg(keys + 64 * p);
                if (k + 1 < capi) it.v[p].y = __ldg(keys + 64 * p + 1);
            }
        }
    }
    it.before = kKeyInf - 1;
    if (lane == 0 && k0 > 0 && k0 < capi) it.before = __ldg(keys - 1);
}

// Exact order check of an item, on the values: !(next <= prev) also catches a NaN on either side.  Keys past the
// cap were read as 0.0, below every valid key.  Used for ragged items and wherever the quick check on the high
// words found two equal ones.
template <int E>
__device__ __forceinline__ bool level0_order_exact(const Level0Item<E> &it, int lane) {
    bool wrong = false;
    double prev_y = 0.0;                                       // lane 31: its y of the previous slice
#pragma unroll
    for (int p = 0; p < E / 2; ++p) {
        const double x = __longlong_as_double((long long)it.v[p].x), y = __longlong_as_double((long long)it.v[p].y);
        const double nx = __longlong_as_double((long long)__shfl_sync(kFull, it.v[p].x, (lane + 1) & 31));
        wrong |= !(y <= x);
        if (lane < 31) wrong |= !(nx <= y);                    // the next lane's x follows this lane's y
        else if (p > 0) wrong |= !(nx <= prev_y);              // lane 0's x of this slice follows lane 31's y of the last
        prev_y = y;
    }
    if (lane == 0) wrong |= !(__longlong_as_double((long long)it.v[0].x) <= __longlong_as_double((long long)it.before));
    return wrong;
}

template <int E, bool ONE>
__device__ __forceinline__ void level0_process(const Level0Item<E> &it, int64_t item, int32_t items_per_row,
                                               int lane, unsigned int *s_fine, unsigned W0, int t_guess,
                                               unsigned int *__restrict__ pguess, long long *capsum, long long *sum_pg,
                                               bool *bad) {
    const int64_t row = ONE ? item : item / items_per_row;
    const int32_t k0 = ONE ? 0 : (int32_t)(item - row * items_per_row) * (kWarp * E);
    const int32_t nvalid = it.capi - k0;                       // keys of this item below the cap (may be <= 0 or > 32 E)
    const bool full = nvalid >= kWarp * E;
    if (lane == 0 && k0 == 0) *capsum += it.capi;
    unsigned hx[E / 2], hy[E / 2];
#pragma unroll
    for (int p = 0; p < E / 2; ++p) {
        hx[p] = (unsigned)(it.v[p].x >> 32);
        hy[p] = (unsigned)(it.v[p].y >> 32);
    }
    // Order check.  The high words of valid keys order like the keys (a sign bit or a NaN shows as a high word
    // above its predecessor's, the first key being held against the largest finite double); only where two
    // neighbours have EQUAL high words do the low words matter, and then the exact check runs.  A row of
    // hora_gains never has such neighbours (consecutive entries differ by more than 1 part in 2^11).
    // Keys past the cap were read as 0: they can never show as a violation (0 is above nothing), and they are
    // kept out of the tie test by their index (a test that whole items skip).
    {
        bool viol = false, ties = false;
        auto quick = [&](auto whole) {
            constexpr bool kWhole = decltype(whole)::value;
            unsigned prev_hy = 0;
#pragma unroll
            for (int p = 0; p < E / 2; ++p) {
                const int32_t kk = 64 * p + 2 * lane;
                const unsigned nh = __shfl_sync(kFull, hx[p], (lane + 1) & 31);
                viol |= hy[p] > hx[p];
                ties |= hy[p] == hx[p] && (kWhole || kk + 1 < nvalid);
                // the key after this pair: the next lane's x; lane 31 holds lane 0's x against its last slice's y
                const unsigned mine = lane < 31 ? hy[p] : prev_hy;
                const int32_t next_k = lane < 31 ? kk + 2 : 64 * p;
                if (lane < 31 || p > 0) {
                    viol |= nh > mine;
                    ties |= nh == mine && (kWhole || next_k < nvalid);
                }
                prev_hy = hy[p];
            }
        };
        if (full) quick(std::true_type{}); else quick(std::false_type{});
        if (lane == 0) {
            const unsigned bh = (unsigned)(it.before >> 32);
            viol |= hx[0] > bh;
            ties |= hx[0] == bh && nvalid > 0;
        }
        if (__any_sync(kFull, ties)) viol |= level0_order_exact<E>(it, lane);
        *bad |= viol;
    }
    // Window: ts = prefix23 - W0 is negative below the window and >= kFineBins above it.  Slices come in
    // descending order, so after one that lies wholly below the window nothing is left to count.
    int above = 0;
#pragma unroll
    for (int p = 0; p < E / 2; ++p) {
        const int tsx = (int)(hx[p] >> 9) - (int)W0, tsy = (int)(hy[p] >> 9) - (int)W0;
        const int32_t kk = 64 * p + 2 * lane;
        const bool vx = full || kk < nvalid, vy = full || kk + 1 < nvalid;
        if (__all_sync(kFull, vy && tsy >= kFineBins)) {       // the slice lies above the window (hence above the guess)
            above += 2;
            continue;
        }
        if (__all_sync(kFull, !vx || tsx < 0)) break;          // ... or wholly below it
        if (vx) {
            if ((unsigned)tsx < (unsigned)kFineBins) atomicAdd(&HORA_AT(s_fine, tsx, kFineBins), 1u);
            above += tsx > t_guess;
        }
        if (vy) {
            if ((unsigned)tsy < (unsigned)kFineBins) atomicAdd(&HORA_AT(s_fine, tsy, kFineBins), 1u);
            above += tsy > t_guess;
        }
    }
    above = __reduce_add_sync(kFull, above);
    if (lane == 0) {
        *sum_pg += above;
        if (ONE) pguess[row] = (unsigned int)above;
        else if (above) atomicAdd(pguess + row, (unsigned int)above);   // several items per row: cleared by the host
    }
}

// CTAs per SM of the full-read pass: what the registers allow (two items of 16 E bytes per lane in flight)
template <int E>
constexpr int level0_per_sm() { return E == 8 ? 3 : 5; }

template <int E, bool VEC2, bool ONE>
__global__ void __launch_bounds__(kSelThreads, level0_per_sm<E>())
select_level0(const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N, int32_t ld,
              const double *__restrict__ gains, int64_t B, AllocHeader *hdr, unsigned long long *hist_fine,
              unsigned int *__restrict__ pguess) {
    pdl_enter();
    __shared__ unsigned int s_fine[kFineBins];             // the window's 23-bit bins
    __shared__ long long s_warp[kSelThreads / kWarp];
    for (int b = threadIdx.x; b < kFineBins; b += kSelThreads) s_fine[b] = 0;
    __syncthreads();
    const int lane = lane_id();
    const unsigned W0 = (unsigned)hdr->win_lo << kFineBits;
    int t_guess = (int)(hdr->guess_hi >> 9) - (int)W0;
    t_guess = t_guess < 0 ? 0 : (t_guess >= kFineBins ? kFineBins - 1 : t_guess);
    const int32_t items_per_row = (ld + kWarp * E - 1) / (kWarp * E);
    const int64_t n_items = N * items_per_row;
    const int64_t item0 = (int64_t)blockIdx.x * (kSelThreads / kWarp) + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * (kSelThreads / kWarp);
    long long capsum = 0, sum_pg = 0;
    bool bad = false;
    // two items in flight, in two fixed register sets (no copies): A is processed while B's loads land
    // (reading the matrix from its end, so that what the L2 still holds of the rows hora_gains wrote last is read
    // first, was tried: no difference in the step)
    Level0Item<E> A, Bq;
    level0_fetch<E, VEC2, ONE>(A, cap, cap_scalar, n_items, items_per_row, ld, gains, item0, lane, &bad);
    for (int64_t item = item0; item < n_items; item += 2 * stride) {
        level0_fetch<E, VEC2, ONE>(Bq, cap, cap_scalar, n_items, items_per_row, ld, gains, item + stride, lane, &bad);
        level0_process<E, ONE>(A, item, items_per_row, lane, s_fine, W0, t_guess, pguess, &capsum, &sum_pg, &bad);
        level0_fetch<E, VEC2, ONE>(A, cap, cap_scalar, n_items, items_per_row, ld, gains, item + 2 * stride, lane, &bad);
        if (Bq.capi >= 0)
            level0_process<E, ONE>(Bq, item + stride, items_per_row, lane, s_fine, W0, t_guess, pguess, &capsum, &sum_pg, &bad);
    }
    level0_finish(hdr, hist_fine, s_fine, W0, t_guess, capsum, sum_pg, bad, B, s_warp);
}

// ---------------------------------------------------------------------------------------------------
// The full-read pass for rows of at most 128 keys: LG = 16, 8 or 4 lanes take a row (of at most 8 LG keys) and a
// warp takes 32 / LG consecutive rows at a time, every row with its own cap, its own order check and its own count
// above the guess.  With a warp per row, a 64-key row cost as many warp instructions as a 256-key one (the cap,
// the votes, the reduction and the row's count are per row) and the pass read 2.4 TB/s.
// A lane holds 8 consecutive keys of its row, so all but one of its order checks stay inside the lane; the caps
// are fetched one item further ahead than the keys, whose loads they gate.
template <int LG>
struct Level0Short {
    unsigned long long key[8];     // keys 8 gl .. 8 gl + 7 of the lane's row (gl = its place among the row's lanes);
                                   // keys past the cap read as 0
    int32_t capi;                  // the cap of the lane's row (0 for a row past the end); -1 marks "no item"
};

// what every item of the pass needs, worked out once (items and rows are counted in 32 bits: N < 2^31)
struct Level0ShortPass {
    const int32_t *cap;
    int32_t cap_scalar, N, n_items, ld;
    const unsigned long long *keys;
    unsigned int *pguess;
    WindowView wv;
};

// 16 zero bytes: where a lane's chunk lies past the cap it reads these instead (a select on the address and an
// unconditional load, where a conditional load compiled to a branch of its own per chunk)
__device__ __align__(16) const unsigned long long g_zero_chunk[2] = {0ull, 0ull};

// the cap of the lane's row of `item`, without a branch: the load is taken at a row that exists
template <int LG>
__device__ __forceinline__ int32_t level0_short_cap(const Level0ShortPass &ps, int32_t item, int lane, unsigned *bad) {
    const int32_t row = item * (kWarp / LG) + lane / LG;
    const bool there = row < ps.N;                             // (an item past the end has no row that is)
    int32_t capi = ps.cap_scalar;
    if (ps.cap != nullptr) capi = __ldg(ps.cap + (there ? row : 0));
    const bool ok = (unsigned)capi <= (unsigned)ps.ld;
    *bad |= (unsigned)(there && !ok);
    capi = there && ok ? capi : 0;
    return item < ps.n_items ? capi : -1;
}

template <int LG, bool VEC2>
__device__ __forceinline__ void level0_short_fetch(Level0Short<LG> &it, const Level0ShortPass &ps, int32_t capi,
                                                   int32_t item, int lane) {
    it.capi = capi;
    const int gl = lane & (LG - 1);
    const int32_t row = item * (kWarp / LG) + lane / LG;
    const int32_t nvalid = capi - 8 * gl;                      // <= 0 for "no item" and for a row past the end
    const unsigned long long *keys = ps.keys + ((int64_t)row * ps.ld + 8 * gl);   // (used only where nvalid > 0)
#pragma unroll
    for (int j = 0; j < 8; j += 2) {
        if (VEC2) {
            const ulonglong2 t = __ldg(reinterpret_cast<const ulonglong2 *>(j < nvalid ? keys + j : g_zero_chunk));
            it.key[j] = t.x;
            it.key[j + 1] = j + 1 < nvalid ? t.y : 0ull;
        } else {
            it.key[j] = __ldg(j < nvalid ? keys + j : g_zero_chunk);
            it.key[j + 1] = __ldg(j + 1 < nvalid ? keys + j + 1 : g_zero_chunk);
        }
    }
}

template <int LG>
__device__ __forceinline__ void level0_short_process(const Level0Short<LG> &it, const Level0ShortPass &ps, int32_t item,
                                                     int lane, int32_t *capsum, int32_t *sum_pg, unsigned *bad) {
    const int gl = lane & (LG - 1);
    const int32_t row = item * (kWarp / LG) + lane / LG;
    const int32_t nvalid = it.capi - 8 * gl;
    // Order: the bit patterns of finite non-negative doubles order like the values, and anything else (a sign bit,
    // an infinity, a NaN) is a pattern above the largest finite one: it either exceeds its predecessor or is the
    // row's first key, which is held against that bound.  Keys past the cap are 0 and exceed nothing.
    {
        bool viol = false;
#pragma unroll
        for (int j = 0; j < 7; ++j) viol |= it.key[j + 1] > it.key[j];
        const unsigned long long nx = __shfl_down_sync(kFull, it.key[0], 1);
        viol |= gl < LG - 1 && nx > it.key[7];                 // the next lane of the same row
        viol |= gl == 0 && it.key[0] > kKeyInf - 1;
        *bad |= (unsigned)viol;
    }
    unsigned h[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) h[j] = (unsigned)(it.key[j] >> 32);
    int above = window_count<8>(h, nvalid, ps.wv);
#pragma unroll
    for (int d = 1; d < LG; d <<= 1) above += __shfl_xor_sync(kFull, above, d);
    if (gl == 0 && row < ps.N) {
        *capsum += it.capi;
        *sum_pg += above;
        ps.pguess[row] = (unsigned int)above;
    }
}

template <int LG, bool VEC2>
__global__ void __launch_bounds__(kSelThreads, 3)
select_level0_short(const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N, int32_t ld,
                    const double *__restrict__ gains, int64_t B, AllocHeader *hdr, unsigned long long *hist_fine,
                    unsigned int *__restrict__ pguess) {
    pdl_enter();
    __shared__ unsigned int s_fine[kFineBins];
    __shared__ long long s_warp[kSelThreads / kWarp];
    for (int b = threadIdx.x; b < kFineBins; b += kSelThreads) s_fine[b] = 0;
    __syncthreads();
    const int lane = lane_id();
    const unsigned W0 = (unsigned)hdr->win_lo << kFineBits;
    int t_guess = (int)(hdr->guess_hi >> 9) - (int)W0;
    t_guess = t_guess < 0 ? 0 : (t_guess >= kFineBins ? kFineBins - 1 : t_guess);
    constexpr int R = kWarp / LG;
    Level0ShortPass ps;
    ps.cap = cap;
    ps.cap_scalar = cap_scalar;
    ps.N = (int32_t)N;
    ps.n_items = (int32_t)((N + R - 1) / R);
    ps.ld = ld;
    ps.keys = reinterpret_cast<const unsigned long long *>(gains);
    ps.pguess = pguess;
    ps.wv.set(s_fine, W0, t_guess);
    const int32_t item0 = (int32_t)(blockIdx.x * (kSelThreads / kWarp) + (threadIdx.x >> 5));
    const int32_t stride = (int32_t)(gridDim.x * (kSelThreads / kWarp));   // (item + 3 stride stays far below 2^31)
    int32_t capsum = 0, sum_pg = 0;                            // per thread: at most 2^31 / (32 * a wave of warps)
    unsigned bad = 0;
    // two items in flight, in two fixed register sets, as in select_level0; caps one item further ahead
    Level0Short<LG> A, Bq;
    int32_t cap_b = level0_short_cap<LG>(ps, item0 + stride, lane, &bad);
    level0_short_fetch<LG, VEC2>(A, ps, level0_short_cap<LG>(ps, item0, lane, &bad), item0, lane);
    for (int32_t item = item0; item < ps.n_items; item += 2 * stride) {
        const int32_t cap_a = level0_short_cap<LG>(ps, item + 2 * stride, lane, &bad);
        level0_short_fetch<LG, VEC2>(Bq, ps, cap_b, item + stride, lane);
        level0_short_process<LG>(A, ps, item, lane, &capsum, &sum_pg, &bad);
        cap_b = level0_short_cap<LG>(ps, item + 3 * stride, lane, &bad);
        level0_short_fetch<LG, VEC2>(A, ps, cap_a, item + 2 * stride, lane);
        if (Bq.capi >= 0) level0_short_process<LG>(Bq, ps, item + stride, lane, &capsum, &sum_pg, &bad);
    }
    level0_finish(hdr, hist_fine, s_fine, W0, t_guess, capsum, sum_pg, bad != 0, B, s_warp);
}

// The plain pass, for the rare case that the window missed: a warp per row, every key counted on its top 13
// bits; the last CTA selects that digit and the selection goes on from there.  (The counts above the guess
// that level 0 stored mean little then; level 1 falls back to searching the rows.)
__global__ void __launch_bounds__(kSelThreads)
select_level0_full(const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N, int32_t ld,
                   const double *__restrict__ gains, AllocHeader *hdr, unsigned long long *hist) {
    pdl_enter();
    __shared__ unsigned int s_hist[kBins];
    __shared__ long long s_warp[kSelThreads / kWarp];
    if (*(volatile int32_t *)&hdr->status != 0 || hdr->l0_miss == 0) return;
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) s_hist[b] = 0;
    __syncthreads();
    const int lane = lane_id();
    const int64_t stride = (int64_t)gridDim.x * (kSelThreads / kWarp);
    for (int64_t row = (int64_t)blockIdx.x * (kSelThreads / kWarp) + (threadIdx.x >> 5); row < N; row += stride) {
        int32_t capi = cap ? __ldg(cap + row) : cap_scalar;
        capi = capi < 0 ? 0 : (capi > ld ? ld : capi);
        const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(gains) + row * (int64_t)ld;
        for (int32_t k0 = 0; k0 < capi; k0 += 8 * kWarp) {      // eight coalesced loads in flight per lane
            unsigned long long key[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int32_t j = k0 + u * kWarp + lane;
                key[u] = j < capi ? __ldg(keys + j) : 0ull;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (k0 + u * kWarp + lane < capi) atomicAdd(&s_hist[(int)(key[u] >> 51) & (kBins - 1)], 1u);
        }
    }
    __syncthreads();
    flush_hist(s_hist, hist, kBins);
    if (last_block(&hdr->ticket[14])) {
        find_digit(hdr, hist, kBins, kDigitBits, 51, 0, false, s_warp);
        if (threadIdx.x == 0) hdr->list_mode = (hdr->resolved > 0 && hdr->bin_count <= (long long)kListCap) ? 1 : 0;
    }
}

// ---------------------------------------------------------------------------------------------------
// Fused form of the full-read pass, used when the caller passes no gains matrix: the kernel that BUILDS the
// rows (same arithmetic, same bits as hora_gains) counts the keys while they are still in registers, so the
// matrix is written once and not read back in full.  The taps below plug into gains_chunk.

// counts every valid key of the lane on its top 13 bits only (the sampled estimate)
template <int E>
struct CoarseTap {
    unsigned long long key[E];
    unsigned int *s_hist;
    __device__ __forceinline__ void pair(int m, double g0, double g1) {
        key[m] = (unsigned long long)__double_as_longlong(g0);
        key[m + 1] = (unsigned long long)__double_as_longlong(g1);
    }
    __device__ __forceinline__ void finish(int32_t, int32_t k, int32_t capi, int32_t) {
        const int valid = capi - k;
#pragma unroll
        for (int m = 0; m < E; ++m)
            if (m < valid) atomicAdd(&s_hist[(unsigned)(key[m] >> 51)], 1u);
    }
    __device__ __forceinline__ void begin_row(int64_t, int32_t) {}
};

// the level-0 bookkeeping: window histogram and the count of keys above the guessed threshold.  LG lanes build a
// row (32 for long rows; 16, 8 or 4 when several short rows share the warp): the counts are summed over the
// row's own lanes, and the first lane of a row keeps its totals.
template <int E, int LG>
struct Level0Tap {
    unsigned long long key[E];
    WindowView wv;
    unsigned int *pguess;
    unsigned int *pg_row;          // the count of the prompt being built (null: the row does not exist)
    unsigned W0;
    int t_guess;
    unsigned int row_above;        // first lane of the row: keys above the guess in the chunks of this row so far
    long long sum_pg;              // first lane of a row: the same over all rows it led
    long long capsum;              // first lane of a row: caps of the rows it led
    __device__ __forceinline__ bool leader() const { return (threadIdx.x & (LG - 1)) == 0; }
    __device__ __forceinline__ void begin_row(int64_t row, int32_t capi) {
        pg_row = row >= 0 ? pguess + row : nullptr;
        row_above = 0;
        if (leader()) capsum += capi;
    }
    __device__ __forceinline__ void pair(int m, double g0, double g1) {
        key[m] = (unsigned long long)__double_as_longlong(g0);
        key[m + 1] = (unsigned long long)__double_as_longlong(g1);
    }
    __device__ __forceinline__ void finish(int32_t, int32_t k, int32_t capi, int32_t) {
        unsigned h[E];
#pragma unroll
        for (int m = 0; m < E; ++m) h[m] = (unsigned)(key[m] >> 32);
        int above = window_count<E>(h, capi - k, wv);
        if (LG == kWarp) {
            above = __reduce_add_sync(kFull, above);
        } else {
#pragma unroll
            for (int d = 1; d < LG; d <<= 1) above += __shfl_xor_sync(kFull, above, d);
        }
        row_above += (unsigned int)above;
        sum_pg += above;
        if (leader() && pg_row != nullptr) *pg_row = row_above;   // the row's chunks come one after another in these lanes
    }
};

// Estimate for the fused pass: the sampled rows are computed, not read.
template <int E>
__global__ void __launch_bounds__(kSelThreads)
select_estimate_fused(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
                      const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                      int64_t N, int32_t ld, int64_t every, int64_t B, AllocHeader *hdr, unsigned long long *hist) {
    pdl_enter();
    __shared__ unsigned int s_hist[kBins];
    __shared__ long long s_warp[kSelThreads / kWarp];
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) s_hist[b] = 0;
    __syncthreads();
    const int lane = lane_id();
    const int64_t n_sample = (N + every - 1) / every;
    const int64_t warp0 = (int64_t)blockIdx.x * (kSelThreads / kWarp) + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * (kSelThreads / kWarp);
    long long capsum = 0;
    CoarseTap<E> tap;
    tap.s_hist = s_hist;
    for (int64_t sidx = warp0; sidx < n_sample; sidx += stride) {
        const Posterior p = load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, sidx * every);
        if (lane == 0) capsum += p.cap;
        const double a = p.ok ? p.a : 1.0, b = p.ok ? p.b : 1.0;
        double carry = 1.0;
        for (int32_t k0 = 0; k0 < p.cap; k0 += kWarp * E)
            gains_chunk<E, false, false>(a, b, a + b, p.cap, ld, k0, lane, carry, nullptr, nullptr, nullptr, tap);
    }
    __syncthreads();
    flush_hist(s_hist, hist, kBins);
    long long tot;
    block_exclusive_sum(capsum, &tot, s_warp);
    if (threadIdx.x == 0 && tot) atomicAdd(&hdr->sample_cap, (unsigned long long)tot);
    if (last_block(&hdr->ticket[15])) place_window(hdr, hist, B, n_sample, N, s_warp);
}

// The fused full pass: the row loop of hora_gains (same staging, same arithmetic, same stores) with level 0's
// counting tapped in.  Rows are trusted to be sorted (they were just computed), so only the inputs are
// validated (the row loop raises the status for invalid priors, counts or caps).
template <int E, bool VEC2, int LG>
__global__ void __launch_bounds__(kSelThreads, 3)
gains_level0_fused(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
                   const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
                   int64_t N, int32_t ld, double *__restrict__ gains, int64_t B, AllocHeader *hdr,
                   unsigned long long *hist_fine, unsigned int *__restrict__ pguess) {
    pdl_enter();
    __shared__ unsigned int s_fine[kFineBins];
    __shared__ long long s_warp[kSelThreads / kWarp];
    for (int b = threadIdx.x; b < kFineBins; b += kSelThreads) s_fine[b] = 0;
    __syncthreads();
    Level0Tap<E, LG> tap;
    tap.pguess = pguess;
    tap.pg_row = pguess;
    tap.W0 = (unsigned)hdr->win_lo << kFineBits;
    const int t_guess = (int)(hdr->guess_hi >> 9) - (int)tap.W0;
    tap.t_guess = t_guess < 0 ? 0 : (t_guess >= kFineBins ? kFineBins - 1 : t_guess);
    tap.wv.set(s_fine, tap.W0, tap.t_guess);
    tap.row_above = 0;
    tap.sum_pg = 0;
    tap.capsum = 0;
    gains_rows_cta<E, VEC2, Level0Tap<E, LG>, LG>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, &hdr->status, tap);
    level0_finish(hdr, hist_fine, s_fine, tap.W0, tap.t_guess, tap.leader() ? tap.capsum : 0, tap.leader() ? tap.sum_pg : 0,
                  false, B, s_warp);
}

// ---------------------------------------------------------------------------------------------------
// Level 1: a thread per row.  r bits of the threshold are known (23 after a window hit, else 13); call P that
// prefix.  The row is non-increasing, so with p_hi = #keys above P and p_lo = #keys above or equal, the keys
// that carry P are the segment [p_hi, p_lo).  Level 0 left a guess of p_hi (the keys above a threshold
// interpolated from the sample); the thread reads the 8 keys around it — two sectors — and is done when the
// first of them is above P (or is the row's first key) and the last of them is below P (or is the row's
// last).  Otherwise it widens the range a few times, and after that two binary searches over the row find
// the segment.  The keys of the segment go to the candidate list (list mode: one slot reservation per warp
// that has any) or are histogrammed on the next digit, their rows appended to the active list.
// A per-row sketch of every 8th key, written by level 0 and scanned here, was the first design: the scan
// cost more issue slots (700 instructions per row) and memory (200 bytes per row) than the whole search here.

// prefix of a key: its top r bits, r <= 32
__device__ __forceinline__ unsigned key_prefix(unsigned long long key, int r) { return (unsigned)(key >> 32) >> (32 - r); }

// first index in [0, n) whose prefix is <= P (STRICT false) or < P (STRICT true); n if none
template <bool STRICT>
__device__ __forceinline__ int32_t first_not_above(const unsigned long long *__restrict__ keys, int32_t n, unsigned P, int r) {
    int32_t lo = 0, hi = n;
    while (lo < hi) {
        const int32_t mid = (lo + hi) >> 1;
        const unsigned kp = key_prefix(__ldg(&HORA_AT(keys, mid, n)), r);
        if (STRICT ? kp >= P : kp > P) lo = mid + 1; else hi = mid;
    }
    return lo;
}

template <bool VEC2>
__global__ void __launch_bounds__(kSelThreads, kLevel1PerSm)
select_level1(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
              const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N,
              int32_t ld, const double *__restrict__ gains, AllocHeader *hdr, unsigned long long *hist1,
              const unsigned int *__restrict__ pguess, int2 *__restrict__ rowstate,
              int32_t *__restrict__ active, unsigned long long *__restrict__ cand_key,
              int32_t *__restrict__ cand_row, long long *bsum_hi, double *__restrict__ objrow) {
    pdl_enter();
    __shared__ unsigned int s_hist[kBins];
    __shared__ long long s_warp[kSelThreads / kWarp];
    __shared__ unsigned long long s_ref;                         // digit route: the CTA's reference key, once it has one
    __shared__ int s_stop;
    // one reading of the status for the whole CTA: this kernel's own CTAs raise it when they finish, and the
    // threads of a CTA that read it one by one could disagree on whether to stay for the barriers below
    if (threadIdx.x == 0) s_stop = *(volatile int32_t *)&hdr->status != 0;
    const bool list = hdr->list_mode != 0;
    if (!list) {
        for (int b = threadIdx.x; b < kBins; b += kSelThreads) s_hist[b] = 0;
        if (threadIdx.x == 0) s_ref = 0ull;
    }

    bool differs = false;
    const int lane = lane_id();
    const int r = hdr->resolved;                                 // 13 or 23: the prefix lies in the key's high word
    const unsigned P = (unsigned)(hdr->prefix_key >> 32) >> (32 - r);
    int bits, shift;
    next_digit(r, &bits, &shift);
    const unsigned long long digit_mask = (1ull << bits) - 1ull;
    const int64_t stride = (int64_t)gridDim.x * kSelThreads;
    bool bad = false;
    // The inputs of a thread's NEXT row (guess, prior, count, cap) are fetched while the current row's keys are
    // being looked at.
    struct RowInputs { double al, be; int32_t ci, capi; unsigned int guess; };
    auto fetch_inputs = [&](int64_t row) {
        RowInputs in;
        in.al = alpha0; in.be = beta0; in.ci = 0; in.capi = cap_scalar; in.guess = 0;
        if (row < N) {
            in.guess = __ldg(pguess + row);
            if (alpha) { in.al = __ldg(alpha + row); in.be = __ldg(beta + row); }
            in.ci = __ldg(c + row);
            if (cap) in.capi = __ldg(cap + row);
        }
        return in;
    };
    RowInputs nxt = fetch_inputs((int64_t)blockIdx.x * kSelThreads + threadIdx.x);   // (in flight across the barrier)
    __syncthreads();
    if (s_stop) return;
    for (int64_t base = (int64_t)blockIdx.x * kSelThreads; base < N; base += stride) {
        const int64_t row = base + threadIdx.x;
        int32_t p_hi = 0, n_eq = 0;
        const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(gains);
        const RowInputs cur = nxt;
        nxt = fetch_inputs(row + stride);
        if (row < N) {
            const unsigned int guess = cur.guess;
            const Posterior post = make_posterior(cur.al, cur.be, cur.ci, cur.capi, G0, ld);
            bad |= !post.ok;
            const int32_t capi = post.cap;                       // 0 for an invalid row
            keys += row * (int64_t)ld;
            // the 8 keys around the guess, from a 4-key boundary (two whole sectors of an aligned row), at
            // least two keys on either side of it
            const int32_t j0 = guess < (unsigned)capi ? (int32_t)guess : capi;
            int32_t ws = (j0 > 2 ? j0 - 2 : 0) & ~3;
            int32_t we = ws + 8 < capi ? ws + 8 : capi;
            int32_t n_gt = 0;
            unsigned kp_first = 0, kp_last = 0;
            {
                unsigned kp[8];
                if (VEC2) {
#pragma unroll
                    for (int u = 0; u < 8; u += 2) {
                        ulonglong2 t = make_ulonglong2(0ull, 0ull);
                        if (ws + u < we) t = __ldg(reinterpret_cast<const ulonglong2 *>(&HORA_AT(keys, ws + u, ld - 1)));
                        kp[u] = key_prefix(t.x, r);
                        kp[u + 1] = key_prefix(t.y, r);
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < 8; ++u) kp[u] = ws + u < we ? key_prefix(__ldg(&HORA_AT(keys, ws + u, ld)), r) : 0u;
                }
                kp_first = kp[0];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const bool in = ws + u < we;
                    n_gt += in && kp[u] > P;
                    n_eq += in && kp[u] == P;
                    if (ws + u == we - 1) kp_last = kp[u];
                }
            }
            // done when everything before the keys read is above P and everything after them below it;
            // else widen by 8 keys on the open side, a few times, before falling back to a search of the row
            bool left_ok = ws == 0 || (we > ws && kp_first > P);
            bool right_ok = we == capi || kp_last < P;
            for (int widen = 0; widen < 3 && !(left_ok && right_ok); ++widen) {
                if (!left_ok) {                                  // the 8 keys before (independent loads)
                    unsigned kp[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) kp[u] = ws - 1 - u >= 0 ? key_prefix(__ldg(&HORA_AT(keys, ws - 1 - u, ld)), r) : 0u;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (ws - 1 - u >= 0) {
                            n_gt += kp[u] > P;
                            n_eq += kp[u] == P;
                            kp_first = kp[u];
                        }
                    }
                    ws = ws > 8 ? ws - 8 : 0;
                    left_ok = ws == 0 || kp_first > P;
                }
                if (!right_ok) {                                 // the 8 keys after
                    unsigned kp[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) kp[u] = we + u < capi ? key_prefix(__ldg(&HORA_AT(keys, we + u, ld)), r) : 0u;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (we + u < capi) {
                            n_gt += kp[u] > P;
                            n_eq += kp[u] == P;
                            kp_last = kp[u];
                        }
                    }
                    we = we + 8 < capi ? we + 8 : capi;
                    right_ok = we == capi || kp_last < P;
                }
            }
            if (left_ok && right_ok) {
                p_hi = ws + n_gt;
            } else {                                             // a poor guess, or a long segment
                p_hi = first_not_above<false>(keys, capi, P, r);
                n_eq = first_not_above<true>(keys + p_hi, capi - p_hi, P, r);
            }
            rowstate[row] = make_int2(p_hi, p_hi + n_eq);
            if (objrow != nullptr) {
                // no key in the threshold's bin: Delta_i = p_hi is final, and g_i(Delta_i) was just read (L1)
                double u = -1.0;                                 // otherwise: evaluated by the output pass
                if (n_eq == 0)
                    u = p_hi > 0 ? utility_from_gain(__longlong_as_double((long long)__ldg(&HORA_AT(keys, p_hi - 1, ld))), post.a, post.b, p_hi)
                                 : 0.0;
                objrow[row] = u;
            }
            if (!list) {
                // digit route: the segment's keys on the next digit.  This route means many keys in one bin — in the
                // extreme one value tied a million times — so every key is held against a reference key (the CTA's first
                // key, itself held against the first that any CTA put into the header; 0 stands for "none yet"): if
                // none differs, the threshold is known.  (Letting the lanes that meet in a bin send one update
                // between them made the pass slower.)
                for (int32_t j = 0; j < n_eq; ++j) {
                    const unsigned long long key = __ldg(&HORA_AT(keys, p_hi + j, ld));
                    unsigned long long ref = *(volatile unsigned long long *)&s_ref;
                    if (ref == 0ull) {                           // the CTA's first key becomes its reference ...
                        ref = atomicCAS(&s_ref, 0ull, key);
                        if (ref == 0ull) {                       // ... and is held against the header's, once per CTA
                            const unsigned long long g = atomicCAS(&hdr->seg_ref, 0ull, key);
                            differs |= g != 0ull && g != key;
                            ref = key;
                        }
                    }
                    differs |= key != ref || key == 0ull;      // (a caller's matrix may hold zeros: no shortcut then)
                    atomicAdd(&HORA_AT(s_hist, (key >> shift) & digit_mask, kBins), 1u);
                }
            }
        }
        if (list) {
            // per warp: one addition to the block sum of p_hi, one slot reservation for the warp's keys (the
            // order of the list does not matter to anything).  Nothing here waits for another warp.
            const int hi_sum = __reduce_add_sync(kFull, p_hi);
            if (lane == 0 && hi_sum != 0)
                atomicAdd(reinterpret_cast<unsigned long long *>(bsum_hi) + base / kRowsPerBlock, (unsigned long long)hi_sum);
            const unsigned has = __ballot_sync(kFull, n_eq > 0);
            if (has) {
                int inc = n_eq;                                  // inclusive scan of n_eq over the warp
#pragma unroll
                for (int d = 1; d < kWarp; d <<= 1) {
                    const int t = __shfl_up_sync(kFull, inc, d);
                    if (lane >= d) inc += t;
                }
                const int n_new = __shfl_sync(kFull, inc, kWarp - 1);
                unsigned int slot0 = 0;
                if (lane == 0) slot0 = atomicAdd(&hdr->n_cand, (unsigned int)n_new);
                slot0 = __shfl_sync(kFull, slot0, 0);
                const long long slot = (long long)slot0 + (inc - n_eq);
                for (int32_t j = 0; j < n_eq; ++j) {
                    const unsigned long long key = __ldg(&HORA_AT(keys, p_hi + j, ld));
                    if (slot + j < kListCap) {
                        HORA_AT(cand_key, slot + j, kListCap) = key;
                        HORA_AT(cand_row, slot + j, kListCap) = (int32_t)row;
                    }
                    atomicAdd(hist1 + ((key >> shift) & digit_mask), 1ull);   // few keys: straight to global memory
                }
            }
        } else {
            // append the rows that keep a segment: one counter update per warp
            const unsigned keep = __ballot_sync(kFull, n_eq > 0);
            if (keep) {
                unsigned int slot0 = 0;
                if (lane == 0) slot0 = atomicAdd(&hdr->n_active, (unsigned int)__popc(keep));
                slot0 = __shfl_sync(kFull, slot0, 0);
                if (n_eq > 0) HORA_AT(active, slot0 + __popc(keep & ((1u << lane) - 1u)), N) = (int32_t)row;
            }
        }
    }
    if (bad) raise_status(&hdr->status, HORA_ERR_INVALID_VALUE);
    if (list) return;
    if (differs) *(volatile int32_t *)&hdr->seg_differs = 1;
    __syncthreads();
    flush_hist(s_hist, hist1, 1 << bits);
    if (last_block(&hdr->ticket[1])) find_digit(hdr, hist1, 1 << bits, bits, shift, 1, false, s_warp);
}

// ---------------------------------------------------------------------------------------------------
// The tail: one cooperative launch (every CTA resident at once) that finishes the threshold and leaves, for
// the output pass, the exclusive prefixes of (#keys > lambda, #keys == lambda) over blocks of 1024 prompts.

// Close a row's segment with the finished threshold: keys above it, keys equal to it.
__device__ __forceinline__ int2 close_segment(const unsigned long long *__restrict__ keys, int2 st, unsigned long long lam,
                                              int32_t ld) {
    int32_t n_gt = 0, n_eq = 0;
    for (int32_t pp = st.x; pp < st.y; ++pp) {
        const unsigned long long key = __ldg(&HORA_AT(keys, pp, ld));
        if (key > lam) ++n_gt;
        else if (key == lam) ++n_eq;
        else break;
    }
    return make_int2(st.x + n_gt, st.x + n_gt + n_eq);
}

// List route, run by ONE CTA: the first digit comes from the histogram level 1 accumulated in global memory;
// the keys that carry it are usually a handful and are gathered into shared memory, over which the remaining
// digits are found 13 bits per sweep.  Should more than kListSmall keys share that digit (ties), the sweeps
// run over the list in global memory instead.  Then the block sums are corrected and scanned.
__device__ void tail_list(int64_t B, AllocHeader *hdr, const unsigned long long *hist1,
                          const unsigned long long *__restrict__ cand_key, const int32_t *__restrict__ cand_row,
                          long long *bsum_hi, long long *bsum_t, int64_t NB, unsigned int *s_hist,
                          unsigned long long *s_keys, long long *s_warp) {
    __shared__ long long s_pick[3];                              // digit, count above it, count of it
    __shared__ unsigned int s_fill;
    const int tid = threadIdx.x;
    unsigned int n_all = hdr->n_cand;
    n_all = n_all < (unsigned)kListCap ? n_all : (unsigned)kListCap;
    int resolved = hdr->resolved;
    long long need = hdr->need;
    unsigned long long prefix = hdr->prefix_key;
    const int r0 = resolved;                                     // every key of the list agrees on these bits
    long long left;                                              // keys that carry every digit found so far
    {
        int bits, shift;
        next_digit(resolved, &bits, &shift);
        long long above = 0, count = 0;
        const int digit = locate_rank(hist1, 1 << bits, need, &above, &count, s_warp);
        if (digit < 0) {                                         // the rank must lie within the list: an internal fault
            if (tid == 0) raise_status(&hdr->status, HORA_ERR_INTERNAL);
            return;
        }
        need -= above;
        prefix |= (unsigned long long)digit << shift;
        resolved += bits;
        left = count;
    }
    const unsigned long long *src = cand_key;
    unsigned int n = n_all;
    if (tid == 0) s_fill = 0;
    __syncthreads();
    if (left <= kListSmall && resolved < 64) {                   // gather them; the later sweeps stay in shared memory
        const int known = resolved - r0;
        const unsigned long long want = (prefix << r0) >> (64 - known);
        for (unsigned int i0 = 0; i0 < n_all; i0 += 8 * kSelThreads) {
            unsigned long long key[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned int i = i0 + u * kSelThreads + tid;
                key[u] = i < n_all ? cand_key[i] : 0ull;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned int i = i0 + u * kSelThreads + tid;
                if (i < n_all && (key[u] << r0) >> (64 - known) == want) {
                    const unsigned int slot = atomicAdd(&s_fill, 1u);
                    if (slot < (unsigned)kListSmall) HORA_AT(s_keys, slot, kListSmall) = key[u];
                }
            }
        }
        __syncthreads();
        n = s_fill < (unsigned)kListSmall ? s_fill : (unsigned)kListSmall;
        src = s_keys;
    }
    if (src == s_keys && n <= (unsigned)kSelThreads && resolved < 64) {
        // a handful of keys left: rank them directly — the threshold is the key k with
        // #(keys > k) < need <= #(keys >= k); equal keys write the same answer
        if (tid == 0) s_pick[0] = -1;
        __syncthreads();
        if ((unsigned)tid < n) {
            const unsigned long long mine = s_keys[tid];
            long long gt = 0, ge = 0;
            for (unsigned int j = 0; j < n; ++j) {
                const unsigned long long other = s_keys[j];
                gt += other > mine;
                ge += other >= mine;
            }
            if (gt < need && need <= ge) {
                s_pick[0] = (long long)mine;
                s_pick[1] = gt;
                s_pick[2] = ge - gt;
            }
        }
        __syncthreads();
        if (s_pick[0] < 0) {                                     // keys are non-negative doubles: an internal fault
            if (tid == 0) raise_status(&hdr->status, HORA_ERR_INTERNAL);
            return;
        }
        prefix = (unsigned long long)s_pick[0];
        need -= s_pick[1];
        left = s_pick[2];
        resolved = 64;
        __syncthreads();
    }
    while (resolved < 64) {
        int bits, shift;
        next_digit(resolved, &bits, &shift);
        const int bins = 1 << bits;
        for (int b = tid; b < bins; b += kSelThreads) s_hist[b] = 0;
        __syncthreads();
        // keys that agree with the digits found so far in this kernel (bits r0 .. resolved-1)
        const int known = resolved - r0;
        const unsigned long long want = (prefix << r0) >> (64 - known);
        for (unsigned int i0 = 0; i0 < n; i0 += 8 * kSelThreads) {
            unsigned long long key[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned int i = i0 + u * kSelThreads + tid;
                key[u] = i < n ? src[i] : 0ull;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned int i = i0 + u * kSelThreads + tid;
                if (i < n && (key[u] << r0) >> (64 - known) == want)
                    atomicAdd(&s_hist[(key[u] >> shift) & (unsigned long long)(bins - 1)], 1u);
            }
        }
        __syncthreads();
        locate_rank_shared(s_hist, bins, need, s_warp, s_pick);
        if (s_pick[0] < 0) {                                     // the rank left the histogram: an internal fault
            if (tid == 0) raise_status(&hdr->status, HORA_ERR_INTERNAL);
            return;
        }
        need -= s_pick[1];
        prefix |= (unsigned long long)s_pick[0] << shift;
        resolved += bits;
        left = s_pick[2];
        __syncthreads();
    }
    // The threshold is `prefix`; `need` of the `left` keys equal to it are taken.  Block sums: level 1 added up
    // its provisional p_hi (keys above the 23-bit prefix); the listed keys above / equal to the threshold
    // complete them, 4096 blocks at a time through shared-memory counters.
    unsigned int *s_fix_hi = s_hist, *s_fix_t = s_hist + kBins / 2;
    long long run_hi = 0, run_t = 0;
    for (int64_t b0 = 0; b0 < NB; b0 += kBins / 2) {
        const int64_t n_here = NB - b0 < kBins / 2 ? NB - b0 : kBins / 2;
        for (int b = tid; b < kBins; b += kSelThreads) s_hist[b] = 0;
        __syncthreads();
        for (unsigned int i0 = 0; i0 < n_all; i0 += 8 * kSelThreads) {
            unsigned long long key[8];
            int32_t row[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned int i = i0 + u * kSelThreads + tid;
                key[u] = i < n_all ? cand_key[i] : 0ull;
                row[u] = i < n_all ? cand_row[i] : 0;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned int i = i0 + u * kSelThreads + tid;
                const int64_t blk = (int64_t)row[u] / kRowsPerBlock - b0;
                if (i < n_all && blk >= 0 && blk < n_here) {
                    if (key[u] > prefix) atomicAdd(&HORA_AT(s_fix_hi, blk, kBins / 2), 1u);
                    else if (key[u] == prefix) atomicAdd(&HORA_AT(s_fix_t, blk, kBins / 2), 1u);
                }
            }
        }
        __syncthreads();
        scan_block_sums(bsum_hi, bsum_t, b0, n_here, s_fix_hi, s_fix_t, run_hi, run_t, s_warp);
        __syncthreads();
    }
    if (tid == 0) {
        hdr->prefix_key = prefix;
        hdr->need = need;
        hdr->resolved = resolved;
        hdr->n_above = (unsigned long long)run_hi;
        hdr->n_tied = (unsigned long long)run_t;
        hdr->R = B - run_hi;
        hdr->lambda = __longlong_as_double((long long)prefix);
    }
}

// Digit route, all CTAs: levels 2..4 (a thread per ACTIVE row narrows the stored segment by the digit selected
// one level up; the keys that remain are histogrammed on the next digit, which CTA 0 selects between two
// grid-wide barriers), then every segment is closed with the finished threshold, the block sums formed and
// scanned.  The active list is in no particular order; nothing here depends on it.
__device__ void tail_digits(int64_t N, int32_t ld, const double *__restrict__ gains, int64_t B, AllocHeader *hdr,
                            unsigned long long *hist_all, int2 *__restrict__ rowstate,
                            const int32_t *__restrict__ active, long long *bsum_hi, long long *bsum_t, int64_t NB,
                            unsigned int *s_hist, long long *s_warp) {
    cooperative_groups::grid_group grid = cooperative_groups::this_grid();
    const unsigned int n_active = hdr->n_active;
    const unsigned int stride = gridDim.x * kSelThreads;
    // Every key that carries level 0's prefix has the same value (a mass tie: one candidate type shared by a million
    // prompts): that value is the threshold, and the digit levels, a pass over the active rows each, are skipped.
    // (The rank `need` lies within those keys, so it stays as it is.)
    const unsigned long long seg_ref = hdr->seg_ref;
    const bool all_equal = seg_ref != 0ull && hdr->seg_differs == 0;
    if (all_equal) {
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            hdr->prefix_key = seg_ref;
            hdr->resolved = 64;
            __threadfence();
        }
        grid.sync();
    }
    for (int level = 2; level < kLevels && !all_equal; ++level) {
        int bits = 0, shift = 0;
        next_digit(*(volatile int32_t *)&hdr->resolved, &bits, &shift);
        const int bins = 1 << bits;
        for (int b = threadIdx.x; b < bins; b += kSelThreads) s_hist[b] = 0;
        __syncthreads();
        const int shift_prev = *(volatile int32_t *)&hdr->lv_shift[level - 1];
        const unsigned long long mask_prev = (1ull << *(volatile int32_t *)&hdr->lv_bits[level - 1]) - 1ull;
        const unsigned long long d_prev = (unsigned long long)*(volatile int32_t *)&hdr->sel_digit[level - 1];
        const unsigned long long mask_cur = (unsigned long long)bins - 1ull;
        for (unsigned int idx = blockIdx.x * kSelThreads + threadIdx.x; idx < n_active; idx += stride) {
            const int64_t row = HORA_AT(active, idx, N);
            const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(gains) + row * (int64_t)ld;
            const int2 st = __ldcg(&HORA_AT(rowstate, row, N));
            const int32_t p_hi = st.x, p_end = st.y;
            int32_t p = p_hi, new_hi = p_hi;
            while (p < p_end) {
                const unsigned long long key = __ldg(&HORA_AT(keys, p, ld));
                const unsigned long long dp = (key >> shift_prev) & mask_prev;
                if (dp > d_prev) {
                    new_hi = p + 1;
                } else if (dp == d_prev) {
                    atomicAdd(&HORA_AT(s_hist, (key >> shift) & mask_cur, kBins), 1u);
                } else {
                    break;
                }
                ++p;
            }
            if (new_hi != p_hi || p != p_end) HORA_AT(rowstate, row, N) = make_int2(new_hi, p);
        }
        __syncthreads();
        flush_hist(s_hist, hist_all + (size_t)level * kBins, bins);
        grid.sync();
        if (blockIdx.x == 0) {
            find_digit(hdr, hist_all + (size_t)level * kBins, bins, bits, shift, level, false, s_warp);
            __threadfence();
        }
        grid.sync();
    }
    // close every segment and add up blocks of kRowsPerBlock prompts
    const unsigned long long lam = *(volatile unsigned long long *)&hdr->prefix_key;
    for (int64_t blk = blockIdx.x; blk < NB; blk += gridDim.x) {
        long long hi_sum = 0, t_sum = 0;
#pragma unroll
        for (int q = 0; q < kRowsPerBlock / kSelThreads; ++q) {
            const int64_t row = blk * kRowsPerBlock + q * kSelThreads + threadIdx.x;
            if (row < N) {
                int2 st = __ldcg(rowstate + row);
                if (st.y > st.x) {
                    const int2 fin = close_segment(reinterpret_cast<const unsigned long long *>(gains) + row * (int64_t)ld, st, lam, ld);
                    if (fin.x != st.x || fin.y != st.y) rowstate[row] = fin;
                    st = fin;
                }
                hi_sum += st.x;
                t_sum += st.y - st.x;
            }
        }
        long long tot_hi, tot_t;
        block_exclusive_sum(hi_sum, &tot_hi, s_warp);
        block_exclusive_sum(t_sum, &tot_t, s_warp);
        if (threadIdx.x == 0) { bsum_hi[blk] = tot_hi; bsum_t[blk] = tot_t; }
    }
    grid.sync();
    if (blockIdx.x == 0) {
        long long run_hi = 0, run_t = 0;
        scan_block_sums(bsum_hi, bsum_t, 0, NB, nullptr, nullptr, run_hi, run_t, s_warp);
        if (threadIdx.x == 0) {
            hdr->n_above = (unsigned long long)run_hi;
            hdr->n_tied = (unsigned long long)run_t;
            hdr->R = B - run_hi;
            hdr->lambda = __longlong_as_double((long long)lam);
        }
    }
}

__global__ void __launch_bounds__(kSelThreads, kTailPerSm)
select_tail(int64_t N, int32_t ld, const double *__restrict__ gains, int64_t B, AllocHeader *hdr,
            unsigned long long *hist_all, int2 *__restrict__ rowstate, const int32_t *__restrict__ active,
            long long *bsum_hi, long long *bsum_t, int64_t NB, const unsigned long long *__restrict__ cand_key,
            const int32_t *__restrict__ cand_row) {
    pdl_enter();
    __shared__ unsigned int s_hist[kBins];
    __shared__ unsigned long long s_keys[kListSmall];
    __shared__ long long s_warp[2 * (kSelThreads / kWarp)];
    if (*(volatile int32_t *)&hdr->status != 0) return;         // the same answer in every CTA: nobody waits at a barrier
    if (hdr->list_mode != 0) {
        if (blockIdx.x == 0) tail_list(B, hdr, hist_all + kBins, cand_key, cand_row, bsum_hi, bsum_t, NB, s_hist, s_keys, s_warp);
        return;
    }
    tail_digits(N, ld, gains, B, hdr, hist_all, rowstate, active, bsum_hi, bsum_t, NB, s_hist, s_warp);
}

// (exact multi-word integer helpers: hora_exact.cuh)

__device__ __forceinline__ unsigned long long pack_type(unsigned long long a, unsigned long long b, unsigned long long D) {
    return (a << 43) | (b << 22) | D;   // a, b < 2^21, D < 2^22
}

// ---------------------------------------------------------------------------------------------------
// Exact mode, step 1: per row, find the (at most one) candidate inside the band around the fp64
// threshold, register its type, and store the provisional state (everything above the band is taken).
__global__ void __launch_bounds__(kSelThreads)
exact_collect(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
              const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
              int64_t N, int32_t ld, const double *__restrict__ gains, AllocHeader *hdr, int2 *__restrict__ rowstate,
              int32_t *__restrict__ rowslot, unsigned long long *tkeys, unsigned long long *tcounts,
              double *__restrict__ objrow) {
    pdl_enter();
    __shared__ long long s_warp[kSelThreads / kWarp];
    // instances per table slot, added up in the CTA first: with one type tied a million times every warp of the
    // grid would otherwise update the same global counter
    __shared__ unsigned int s_cnt[kTypeSlots];
    __shared__ int s_stop;                                       // one reading of the status for the whole CTA
    if (threadIdx.x == 0) s_stop = *(volatile int32_t *)&hdr->status != 0;
    for (int h = threadIdx.x; h < kTypeSlots; h += kSelThreads) s_cnt[h] = 0u;
    __syncthreads();
    if (s_stop) return;
    const unsigned long long lam_key = hdr->prefix_key;
    const bool list = hdr->list_mode != 0;
    const double lam = __longlong_as_double((long long)lam_key);
    const double delta_rel = 9.313225746154785e-10;   // 2^-30
    const unsigned long long k_hi = (unsigned long long)__double_as_longlong(lam * (1.0 + delta_rel));
    const unsigned long long k_lo = (unsigned long long)__double_as_longlong(lam * (1.0 - delta_rel));
    const int lane = lane_id();
    const int64_t stride = (int64_t)gridDim.x * kSelThreads;
    long long above = 0;
    int32_t err = 0;
    for (int64_t base = (int64_t)blockIdx.x * kSelThreads; base < N; base += stride) {
        const int64_t row = base + threadIdx.x;
        unsigned long long tkey = 0;
        int32_t q = 0;
        if (row < N) {
            const double al = alpha ? __ldg(alpha + row) : alpha0, be = beta ? __ldg(beta + row) : beta0;
            const int32_t ci = __ldg(c + row);
            const int32_t capi = cap ? __ldg(cap + row) : cap_scalar;
            if (!(al >= 1.0 && be >= 1.0 && al == floor(al) && be == floor(be))) err = HORA_ERR_NOT_INTEGER;
            else if (al + be + (double)G0 + (double)ld >= 1048576.0) err = err ? err : HORA_ERR_EXACT_RANGE;
            const unsigned long long *keys = reinterpret_cast<const unsigned long long *>(gains) + row * (int64_t)ld;
            int2 st = rowstate[row];
            const bool had_segment = st.y > st.x;             // (level 1 evaluated the row's utility only if not)
            const int32_t p_level1 = st.x;
            if (list && st.y > st.x) st = close_segment(keys, st, lam_key, ld);   // the list route leaves segments open
            q = st.x;                                         // #keys > lambda
            if (q > 0 && __ldg(&HORA_AT(keys, q - 1, ld)) <= k_hi) {
                --q;
                if (q > 0 && __ldg(&HORA_AT(keys, q - 1, ld)) <= k_hi) err = err ? err : HORA_ERR_EXACT_RANGE;
            }
            const bool has = (q < capi) && (__ldg(&HORA_AT(keys, q, ld)) >= k_lo);
            if (has && q + 1 < capi && __ldg(&HORA_AT(keys, q + 1, ld)) >= k_lo) err = err ? err : HORA_ERR_EXACT_RANGE;
            if (has && !err)
                tkey = pack_type((unsigned long long)al + ci, (unsigned long long)be + (G0 - ci), (unsigned long long)q + 1);
            // Level 1 left U_i(p_hi) for the rows without a key in the threshold's bin.  It stands unless the exact
            // ranking can still move the row's Delta: a candidate inside the band, or a count that the band changed.
            if (objrow != nullptr && !had_segment && (has || q != p_level1)) objrow[row] = -1.0;
            above += q;
        }
        // one table update per distinct type per warp
        const unsigned int peers = __match_any_sync(kFull, tkey);
        int32_t slot = -1;
        if (tkey != 0) {
            const int leader = __ffs(peers) - 1;
            if (lane == leader) {
                unsigned int h = (unsigned int)((tkey * 0x9E3779B97F4A7C15ull) >> 52) & (kTypeSlots - 1);
                for (int probe = 0; probe < kTypeSlots; ++probe) {
                    // a slot once taken never changes: look before trying to take it
                    unsigned long long old = *(volatile unsigned long long *)&HORA_AT(tkeys, h, kTypeSlots);
                    if (old == 0ull) old = atomicCAS(&HORA_AT(tkeys, h, kTypeSlots), 0ull, tkey);
                    if (old == 0ull || old == tkey) {
                        if (old == 0ull) atomicAdd(&hdr->n_types, 1u);
                        slot = (int32_t)h;
                        break;
                    }
                    h = (h + 1) & (kTypeSlots - 1);
                }
                if (slot >= 0) atomicAdd(&HORA_AT(s_cnt, slot, kTypeSlots), (unsigned int)__popc(peers));
                else err = err ? err : HORA_ERR_EXACT_RANGE;
            }
            slot = __shfl_sync(peers, slot, leader);
        }
        if (row < N) {
            rowslot[row] = slot;
            rowstate[row] = make_int2(q, q);
        }
    }
    if (err) raise_status(&hdr->status, err);
    long long tot;
    block_exclusive_sum(above, &tot, s_warp);                   // (its barriers also put the CTA's counts in place)
    if (threadIdx.x == 0 && tot) atomicAdd(&hdr->band_above, (unsigned long long)tot);
    for (int h = threadIdx.x; h < kTypeSlots; h += kSelThreads) {
        const unsigned int v = s_cnt[h];
        if (v) atomicAdd(&HORA_AT(tcounts, h, kTypeSlots), (unsigned long long)v);
    }
}

// Exact mode, step 2 (one CTA): rank the collected types exactly and label them.
//   label 2: strictly better than the threshold class (taken)   1: threshold class   0: worse
// Numerators and denominators (512 bits each) live in dynamic shared memory: kExactRankSmem bytes.
constexpr int kExactRankThreads = 256;
constexpr size_t kExactRankSmem = (size_t)kMaxTypes * (2 * sizeof(UBig) + sizeof(unsigned long long) + sizeof(int));

__global__ void __launch_bounds__(kExactRankThreads)
exact_rank(int64_t B, AllocHeader *hdr, const unsigned long long *__restrict__ tkeys,
           const unsigned long long *__restrict__ tcounts, int32_t *__restrict__ tlabel) {
    pdl_enter();
    extern __shared__ __align__(16) unsigned char s_rank_raw[];
    UBig *s_num = reinterpret_cast<UBig *>(s_rank_raw);
    UBig *s_den = s_num + kMaxTypes;
    unsigned long long *s_cnt = reinterpret_cast<unsigned long long *>(s_den + kMaxTypes);
    int *s_slot = reinterpret_cast<int *>(s_cnt + kMaxTypes);
    __shared__ int s_n;
    __shared__ int s_err;
    __shared__ unsigned long long s_writer;
    if (hdr->status != 0) return;
    if (threadIdx.x == 0) { s_n = 0; s_err = 0; s_writer = ~0ull; }
    __syncthreads();
    for (int h = threadIdx.x; h < kTypeSlots; h += blockDim.x) {
        tlabel[h] = 0;
        const unsigned long long key = tkeys[h];
        if (key != 0ull) {
            const int j = atomicAdd(&s_n, 1);
            if (j < kMaxTypes) {
                UBig nu, de;
                if (!exact_gain(key >> 43, (key >> 22) & 0x1FFFFFull, key & 0x3FFFFFull, nu, de)) s_err = 1;
                s_num[j] = nu;
                s_den[j] = de;
                s_cnt[j] = tcounts[h];
                s_slot[j] = h;
            }
        }
    }
    __syncthreads();
    const int n = s_n;
    if (n > kMaxTypes || s_err) {
        if (threadIdx.x == 0) raise_status(&hdr->status, HORA_ERR_EXACT_RANGE);
        return;
    }
    const long long Rp = B - (long long)hdr->band_above;     // rollouts to hand out inside the band
    for (int t = threadIdx.x; t < n; t += blockDim.x) {
        long long above = 0, equal = 0;
        for (int u = 0; u < n; ++u) {
            const int s = cmp_products(s_num[u], s_den[t], s_num[t], s_den[u]);   // sign(val_u - val_t)
            if (s > 0) above += (long long)s_cnt[u];
            else if (s == 0) equal += (long long)s_cnt[u];
        }
        int label = 0;
        if (above + equal < Rp) label = 2;
        else if (above < Rp) label = 1;
        HORA_AT(tlabel, s_slot[t], kTypeSlots) = label;
        if (label == 1) {
            // Members of the threshold class agree on R, but their unreduced num/den differ, and so may the
            // last bit of the quotient below: the member with the smallest packed type (a, b, Delta) alone
            // reports lambda (table slots depend on the insertion order, types do not).
            hdr->R = Rp - above;
            atomicMin(&s_writer, tkeys[s_slot[t]]);
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < n; t += blockDim.x)
        if (tkeys[s_slot[t]] == s_writer) hdr->lambda = ratio_double(s_num[t], s_den[t]);
}

// ---------------------------------------------------------------------------------------------------
// Block sums of (p_hi, tied) in prompt order, and their exclusive scan by the last CTA; used where the tail
// did not run (B == 0: mode 0) or its result is relabelled (exact mode: mode 2, apply the labels first).
// With `validate` the priors and counts of every prompt are checked here (level 1 checks them otherwise).
__global__ void __launch_bounds__(kSelThreads)
select_sum(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
           const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar, int validate,
           int64_t N, int32_t ld, const double *__restrict__ gains, int mode, int64_t B, AllocHeader *hdr,
           int2 *__restrict__ rowstate, const int32_t *__restrict__ rowslot, const int32_t *__restrict__ tlabel,
           long long *bsum_hi, long long *bsum_t, int64_t NB) {
    pdl_enter();
    __shared__ long long s_warp[2 * (kSelThreads / kWarp)];
    const bool failed = *(volatile int32_t *)&hdr->status != 0;
    long long hi_sum = 0, t_sum = 0;
    if (!failed) {
        const int64_t row0 = (int64_t)blockIdx.x * kRowsPerBlock;
        constexpr int kPer = kRowsPerBlock / kSelThreads;
        int2 st[kPer];
        int32_t slot[kPer];
        bool ok = true;
#pragma unroll
        for (int q = 0; q < kPer; ++q) {                      // every load of the thread is issued before any is used
            const int64_t row = row0 + q * kSelThreads + threadIdx.x;
            const int64_t rr = row < N ? row : N - 1;
            st[q] = rowstate[rr];
            slot[q] = mode == 2 ? rowslot[rr] : -1;
            if (validate) ok &= load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, rr).ok;
        }
        if (!ok) raise_status(&hdr->status, HORA_ERR_INVALID_VALUE);   // seen by the kernels that follow
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int64_t row = row0 + q * kSelThreads + threadIdx.x;
            if (row < N) {
                if (mode == 2) {
                    const int label = slot[q] >= 0 ? HORA_AT(tlabel, slot[q], kTypeSlots) : 0;
                    st[q] = make_int2(st[q].x + (label == 2), st[q].x + (label == 2) + (label == 1));
                    rowstate[row] = st[q];
                }
                hi_sum += st[q].x;
                t_sum += st[q].y - st[q].x;
            }
        }
    }
    long long tot_hi, tot_t, e_hi, e_t;
    block_exclusive_sum2(hi_sum, t_sum, e_hi, e_t, tot_hi, tot_t, s_warp);
    if (threadIdx.x == 0) { bsum_hi[blockIdx.x] = tot_hi; bsum_t[blockIdx.x] = tot_t; }
    if (last_block(&hdr->ticket[8 + mode])) {
        long long run_hi = 0, run_t = 0;
        scan_block_sums(bsum_hi, bsum_t, 0, NB, nullptr, nullptr, run_hi, run_t, s_warp);
        if (threadIdx.x == 0 && !failed) {
            hdr->n_above = (unsigned long long)run_hi;
            hdr->n_tied = (unsigned long long)run_t;
            hdr->R = B - run_hi;
            if (mode != 2) hdr->lambda = B > 0 ? __longlong_as_double((long long)hdr->prefix_key) : 0.0;
        }
    }
}

// Outputs.  A CTA owns kRowsPerBlock consecutive prompts, a thread four consecutive ones (16-byte loads and
// stores where the caller's arrays are 16-byte aligned: `vec`).  `objrow` (may be null) holds the utilities
// level 1 already evaluated; a negative entry, or no array, means "evaluate here".
__global__ void __launch_bounds__(kSelThreads)
select_out(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
           const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N,
           int32_t ld, const double *__restrict__ gains, int64_t B, uint32_t flags, AllocHeader *hdr,
           const int2 *__restrict__ rowstate, const double *__restrict__ objrow, const long long *__restrict__ bpre_hi,
           const long long *__restrict__ bpre_t, double *objpart, int64_t NB, int32_t *__restrict__ delta,
           int32_t *__restrict__ G, int64_t *__restrict__ offsets, int vec, hora_alloc_info *info) {
    pdl_enter();
    __shared__ long long s_warp[2 * (kSelThreads / kWarp)];
    __shared__ double s_obj[kSelThreads / kWarp];
    constexpr int kPer = kRowsPerBlock / kSelThreads;
    static_assert(kPer == 4, "a thread owns four consecutive prompts");
    const int64_t row0 = (int64_t)blockIdx.x * kRowsPerBlock + (int64_t)threadIdx.x * kPer;
    const bool whole = row0 + kPer <= N;                      // all four prompts exist
    // Every load that does not depend on another is issued here, before the first is used: the header's fields,
    // the block prefixes, the rows' states and utilities (the arrays are read whether or not the call has failed;
    // they lie inside the workspace either way).
    const int32_t status = hdr->status;                       // (raised by earlier kernels only)
    const int32_t list_mode = hdr->list_mode;
    const unsigned long long lam_key = hdr->prefix_key;
    const long long R_hdr = hdr->R;
    const long long blk_hi_raw = bpre_hi[blockIdx.x], blk_t_raw = bpre_t[blockIdx.x];
    const bool use_objrow = objrow != nullptr && !(flags & HORA_FLAG_SKIP_OBJECTIVE);
    int2 st[kPer];
    double o[kPer];
    if (whole) {
        const int4 s01 = *reinterpret_cast<const int4 *>(rowstate + row0), s23 = *reinterpret_cast<const int4 *>(rowstate + row0 + 2);
        st[0] = make_int2(s01.x, s01.y); st[1] = make_int2(s01.z, s01.w);
        st[2] = make_int2(s23.x, s23.y); st[3] = make_int2(s23.z, s23.w);
    } else {
#pragma unroll
        for (int q = 0; q < kPer; ++q) st[q] = row0 + q < N ? rowstate[row0 + q] : make_int2(0, 0);
    }
#pragma unroll
    for (int q = 0; q < kPer; ++q) o[q] = -1.0;
    if (use_objrow) {
        if (whole) {
            const double2 o01 = *reinterpret_cast<const double2 *>(objrow + row0), o23 = *reinterpret_cast<const double2 *>(objrow + row0 + 2);
            o[0] = o01.x; o[1] = o01.y; o[2] = o23.x; o[3] = o23.y;
        } else {
#pragma unroll
            for (int q = 0; q < kPer; ++q) if (row0 + q < N) o[q] = objrow[row0 + q];
        }
    }
    const bool failed = status != 0;
    // the list route of the tail leaves the segments as level 1 found them (exact mode has closed them since)
    const bool open = !failed && list_mode != 0 && !(flags & HORA_FLAG_EXACT_INT);
    const bool want_obj = !failed && !(flags & HORA_FLAG_SKIP_OBJECTIVE);
    const long long blk_hi = failed ? 0 : blk_hi_raw, blk_t = failed ? 0 : blk_t_raw;
    const long long R = failed ? 0 : R_hdr;
    int32_t hi[kPer], tied[kPer];
    long long hi_sum = 0, t_sum = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        if (failed) st[q] = make_int2(0, 0);
        if (open && st[q].y > st[q].x)
            st[q] = close_segment(reinterpret_cast<const unsigned long long *>(gains) + (row0 + q) * (int64_t)ld, st[q], lam_key, ld);
        hi[q] = st[q].x;
        tied[q] = st[q].y - st[q].x;
        hi_sum += hi[q];
        t_sum += tied[q];
    }
    long long th, tt, pre_hi, pre_t;
    block_exclusive_sum2(hi_sum, t_sum, pre_hi, pre_t, th, tt, s_warp);
    pre_hi += blk_hi;
    pre_t += blk_t;
    int32_t d[kPer];
    int64_t of[kPer];
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        long long take = R - pre_t;
        take = take < 0 ? 0 : (take > tied[q] ? tied[q] : take);
        d[q] = hi[q] + (int32_t)take;
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
        for (int q = 0; q < kPer; ++q) {
            if (row0 + q < N) {
                delta[row0 + q] = d[q];
                G[row0 + q] = failed ? 0 : G0 + d[q];
                if (offsets) offsets[row0 + q] = of[q];
            }
        }
    }
    // Objective: level 1's values where they stand (the row had no key in the threshold's bin, so its Delta was
    // final there); the other rows are evaluated here, from the row's own entry g_i(Delta).
    double obj = 0.0;
    if (want_obj) {
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            if (row0 + q < N && d[q] > 0) {
                double u = o[q];
                if (u < 0.0) {
                    const Posterior p = load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, row0 + q);
                    u = utility_from_gain(__ldg(&HORA_AT(gains, (row0 + q) * (int64_t)ld + (d[q] - 1), N * (int64_t)ld)), p.a, p.b, d[q]);
                }
                obj += u;
            }
        }
    }
    if (offsets && blockIdx.x == gridDim.x - 1 && threadIdx.x == kSelThreads - 1)
        offsets[N] = failed ? 0 : N * (int64_t)G0 + B;
    // objective: fixed-order tree (lanes by butterfly, then warps and blocks in index order)
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) obj += __shfl_xor_sync(kFull, obj, d);
    if (lane_id() == 0) s_obj[threadIdx.x >> 5] = obj;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < kSelThreads / kWarp; ++w) s += s_obj[w];
        objpart[blockIdx.x] = s;
    }
    if (last_block(&hdr->ticket[12])) {
        double part = 0.0;
        for (int64_t b = threadIdx.x; b < NB; b += kSelThreads) part += __ldcg(objpart + b);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(kFull, part, d);
        __syncthreads();
        if (lane_id() == 0) s_obj[threadIdx.x >> 5] = part;
        __syncthreads();
        if (threadIdx.x == 0) {
            double s = 0.0;
            for (int w = 0; w < kSelThreads / kWarp; ++w) s += s_obj[w];
            hdr->objective = s;
            if (info) {
                info->status = status;
                info->first_pass_bits = failed ? 0 : hdr->lv_bits[0];
                info->lambda = failed ? 0.0 : hdr->lambda;
                info->n_above = failed ? 0 : (int64_t)hdr->n_above;
                info->n_tied = failed ? 0 : (int64_t)hdr->n_tied;
                info->n_tied_taken = failed ? 0 : hdr->R;
                info->objective = failed ? 0.0 : s;
                info->sum_G = failed ? 0 : N * (int64_t)G0 + B;
                info->sum_cap = (int64_t)hdr->sum_cap;
            }
        }
    }
}

// Marks the call failed from the host's side (a launch that could not be made after others were enqueued).
__global__ void fail_call(AllocHeader *hdr, int32_t code) { raise_status(&hdr->status, code); }

// N == 0: nothing to select; still produce a well-defined summary.
__global__ void write_empty(int64_t B, int64_t *offsets, hora_alloc_info *info) {
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

// Optional profiling aids (see hora_allocate_profile_events / hora_allocate_profile_stages): events recorded
// around the full-read pass, and after each stage of the call.
// The handles are kept per host thread: only calls issued by the thread that set them record anything, so calls
// running concurrently from other threads (on other streams) are left alone.
static thread_local cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;
constexpr int kStageEvents = 7;
static thread_local cudaEvent_t g_stage_ev[kStageEvents] = {};

static inline void mark_stage(int k, cudaStream_t s) {
    const cudaEvent_t ev = g_stage_ev[k];
    if (ev != nullptr) cudaEventRecord(ev, s);
}

template <int E>
static void launch_level0(bool vec2, int grid, cudaStream_t s, const int32_t *cap, int32_t cap_scalar, int64_t N,
                          int32_t ld, const double *gains, int64_t B, const Workspace &w) {
    const bool one = ld <= kWarp * E;                     // an item is a whole row
    grid = clamp_grid((N * ((ld + kWarp * E - 1) / (kWarp * E)) + kSelThreads / kWarp - 1) / (kSelThreads / kWarp),
                      level0_per_sm<E>());                // exactly what is resident at once
    auto go = [&](auto kernel) { launch_pdl(kernel, grid, kSelThreads, 0, s, cap, cap_scalar, N, ld, gains, B, w.hdr, w.hist_fine, w.pguess); };
    if (vec2) { if (one) go(select_level0<E, true, true>); else go(select_level0<E, true, false>); }
    else { if (one) go(select_level0<E, false, true>); else go(select_level0<E, false, false>); }
}

template <int E>
static cudaError_t launch_fused(bool vec2, bool estimate, int grid_est, int64_t every, int grid, cudaStream_t s,
                                const double *alpha, const double *beta, double alpha0, double beta0, const int32_t *c,
                                int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N, int32_t ld, int64_t B,
                                const Workspace &w) {
    if (estimate)
        launch_pdl(select_estimate_fused<E>, grid_est, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar,
                   N, ld, every, B, w.hdr, w.hist_est);
    auto go = [&](auto kernel) {
        launch_pdl(kernel, grid, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, w.gains, B, w.hdr,
                   w.hist_fine, w.pguess);
    };
    // lanes per row as in hora_gains: short rows share a warp
    if (ld > 128) { if (vec2) go(gains_level0_fused<E, true, kWarp>); else go(gains_level0_fused<E, false, kWarp>); }
    else if (ld > 64) { if (vec2) go(gains_level0_fused<E, true, 16>); else go(gains_level0_fused<E, false, 16>); }
    else if (ld > 32) { if (vec2) go(gains_level0_fused<E, true, 8>); else go(gains_level0_fused<E, false, 8>); }
    else { if (vec2) go(gains_level0_fused<E, true, 4>); else go(gains_level0_fused<E, false, 4>); }
    return cudaGetLastError();
}

// CTAs of the cooperative tail on the current device: what fits at once, at most kTailPerSm per SM (0 on failure).
// Looked up once per device.
static int tail_grid_size() {
    constexpr int kMaxDev = 64;
    static std::atomic<int> cached[kMaxDev];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return 0;
    int g = cached[dev].load(std::memory_order_acquire);
    if (g > 0) return g;
    int coop = 0, sms = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_tail, kSelThreads, 0) != cudaSuccess || per_sm <= 0)
        return 0;
    g = sms * (per_sm < kTailPerSm ? per_sm : kTailPerSm);
    cached[dev].store(g, std::memory_order_release);
    return g;
}

}  // namespace hora

extern "C" void hora_allocate_profile_events(void *start_event, void *stop_event) {
    hora::g_prof_start = static_cast<cudaEvent_t>(start_event);
    hora::g_prof_stop = static_cast<cudaEvent_t>(stop_event);
}

extern "C" void hora_allocate_profile_stages(void *const *events_host, int32_t n) {
    for (int k = 0; k < hora::kStageEvents; ++k)
        hora::g_stage_ev[k] = events_host != nullptr && k < n ? static_cast<cudaEvent_t>(events_host[k]) : nullptr;
}

extern "C" size_t hora_allocate_workspace_bytes(int64_t N, int32_t ld, int32_t gains_is_null, uint32_t flags) {
    if (N < 0 || ld < 1) return 0;
    // the caller promises a shared integer prior, exact ties and no matrix: the rank-based route, which needs
    // neither the matrix nor anything per candidate
    if ((flags & HORA_FLAG_SHARED_PRIOR) && gains_is_null != 0)
        return hora::rank_allocate_workspace_bound(N);
    return hora::carve(nullptr, N, ld, gains_is_null != 0, (flags & HORA_FLAG_EXACT_INT) != 0).bytes;
}

extern "C" hora_status_t hora_allocate(const double *alpha, const double *beta, double alpha0, double beta0,
                                       const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N,
                                       int32_t ld, const double *gains, int64_t B, uint32_t flags, int32_t *delta,
                                       int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev, void *workspace,
                                       size_t workspace_bytes, void *stream) {
    using namespace hora;
    if (N < 0 || ld < 1 || G0 < 0 || B < 0) return HORA_ERR_INVALID_ARG;
    if (N > 0x7FFFFFFFll) return HORA_ERR_INVALID_ARG;     // row indices are kept in 32 bits
    if ((alpha == nullptr) != (beta == nullptr)) return HORA_ERR_INVALID_ARG;
    if (alpha == nullptr && !(alpha0 > 0.0 && beta0 > 0.0 && alpha0 < 1.0e300 && beta0 < 1.0e300))
        return HORA_ERR_INVALID_ARG;
    if (cap == nullptr && (cap_scalar < 0 || cap_scalar > ld)) return HORA_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(HORA_FLAG_EXACT_INT | HORA_FLAG_SKIP_OBJECTIVE | HORA_FLAG_SHARED_PRIOR))
        return HORA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (N == 0) {
        write_empty<<<1, 1, 0, s>>>(B, group_offsets, info_dev);
        count_launches(1);
        return cuda_ok(cudaGetLastError());
    }
    if (c == nullptr || delta == nullptr || G == nullptr) return HORA_ERR_INVALID_ARG;
    if (gains != nullptr && (reinterpret_cast<uintptr_t>(gains) & 7u)) return HORA_ERR_INVALID_ARG;
    const bool exact = (flags & HORA_FLAG_EXACT_INT) != 0;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HORA_ERR_WORKSPACE;
    // One prior for all prompts and no matrix given: at most (G0 + 1) * ld distinct candidate values, ranked once
    // (exactly for an integer prior with HORA_FLAG_EXACT_INT, else as the doubles hora_gains would write); the
    // selection runs on ranks and on counts of (c_i, cap_i) and builds no matrix.
    if (alpha == nullptr && gains == nullptr && rank_route_applies(alpha0, beta0, G0, ld, exact))
        return launch_rank_allocate(alpha0, beta0, c, G0, cap, cap_scalar, N, ld, B, flags, delta, G, group_offsets,
                                    info_dev, workspace, workspace_bytes, s, mark_stage);
    const Workspace w = carve(workspace, N, ld, gains == nullptr, exact);
    if (workspace_bytes < w.bytes) return HORA_ERR_WORKSPACE;
    const int64_t NB = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    // the cooperative tail: every CTA must be resident at once, so the grid is what the device can hold; asked
    // before anything is enqueued, so that a device without cooperative launch leaves the outputs untouched
    const int tail_grid = B > 0 ? tail_grid_size() : 0;
    if (B > 0 && tail_grid <= 0) return HORA_ERR_CUDA;
    bool launch_failed = false;

    // header and histograms are contiguous at the start of the workspace
    const size_t zero_bytes = reinterpret_cast<char *>(w.rowstate) - reinterpret_cast<char *>(w.hdr);
    if (cudaMemsetAsync(w.hdr, 0, zero_bytes, s) != cudaSuccess) return HORA_ERR_CUDA;
    if (exact) {
        const size_t tb = reinterpret_cast<char *>(w.rowslot) - reinterpret_cast<char *>(w.tkeys);
        if (cudaMemsetAsync(w.tkeys, 0, tb, s) != cudaSuccess) return HORA_ERR_CUDA;
    }
    const bool fused = gains == nullptr;                  // no matrix given: build it and count its keys in one pass
    if (!fused && ld > 256 && B > 0)                      // rows of several items add up their counts with atomics
        if (cudaMemsetAsync(w.pguess, 0, sizeof(unsigned int) * (size_t)N, s) != cudaSuccess) return HORA_ERR_CUDA;
    if (fused) gains = w.gains;
    const bool vec2 = (ld % 2 == 0) && ((reinterpret_cast<uintptr_t>(gains) & 15u) == 0);
    const int rows_per_cta = kSelThreads / kWarp;
    const int64_t every = (N + kSampleRows - 1) / kSampleRows;
    const int64_t n_sample = (N + every - 1) / every;
    // two rows per warp: half as many CTAs flush their histogram into the same few hundred global bins
    const int grid_est = clamp_grid((n_sample + 2 * rows_per_cta - 1) / (2 * rows_per_cta), 2);
    mark_stage(0, s);
    if (B > 0 && !fused)
        launch_pdl(select_estimate, grid_est, kSelThreads, 0, s, cap, cap_scalar, N, ld, every, gains, B, w.hdr, w.hist_est);
    const int grid0 = clamp_grid((N + rows_per_cta - 1) / rows_per_cta, 3);
    const int grid1 = clamp_grid((N + kSelThreads - 1) / kSelThreads, kLevel1PerSm);
    const cudaEvent_t prof_start = g_prof_start, prof_stop = g_prof_stop;
    if (!fused) mark_stage(1, s);                         // (the fused pass launches its own estimate)
    if (prof_start != nullptr && prof_stop != nullptr) cudaEventRecord(prof_start, s);
    if (fused) {
        const int gridf = clamp_grid((N + kCtaRows - 1) / kCtaRows, 3);
        if (launch_fused<8>(vec2, B > 0, grid_est, every, gridf, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld,
                            B, w) != cudaSuccess)
            return HORA_ERR_CUDA;
    } else if (ld > 256 || (ld > 128 && cap == nullptr && cap_scalar == ld)) {
        // long rows, and whole rows of up to 256 keys (slices settled by votes: 0.35 against 0.37 ms at 2^20 x 256)
        launch_level0<8>(vec2, grid0, s, cap, cap_scalar, N, ld, gains, B, w);
    } else {                                              // short rows share a warp; ragged ones of up to 256 keys
        auto go = [&](auto kernel, int lg) {
            const int64_t items = (N + kWarp / lg - 1) / (kWarp / lg);
            launch_pdl(kernel, clamp_grid((items + rows_per_cta - 1) / rows_per_cta, 3), kSelThreads, 0, s, cap, cap_scalar, N,
                       ld, gains, B, w.hdr, w.hist_fine, w.pguess);
        };
        if (ld > 128) { if (vec2) go(select_level0_short<32, true>, 32); else go(select_level0_short<32, false>, 32); }
        else if (ld > 64) { if (vec2) go(select_level0_short<16, true>, 16); else go(select_level0_short<16, false>, 16); }
        else if (ld > 32) { if (vec2) go(select_level0_short<8, true>, 8); else go(select_level0_short<8, false>, 8); }
        else { if (vec2) go(select_level0_short<4, true>, 4); else go(select_level0_short<4, false>, 4); }
    }
    if (prof_start != nullptr && prof_stop != nullptr) cudaEventRecord(prof_stop, s);
    if (B > 0)                                            // stands down at once unless the window missed
        launch_pdl(select_level0_full, grid0, kSelThreads, 0, s, cap, cap_scalar, N, ld, gains, w.hdr, w.hist_coarse);
    mark_stage(2, s);
    const int grid_rows = clamp_grid((N + kSelThreads - 1) / kSelThreads, 6);
    // utilities of the rows without a key in the threshold's bin are evaluated by level 1, which has the row's
    // entry at hand (in exact mode exact_collect withdraws those that the tie ranking can still move)
    double *objrow = (B > 0 && !(flags & HORA_FLAG_SKIP_OBJECTIVE)) ? w.objrow : nullptr;
    if (B > 0) {
        if (vec2)
            launch_pdl(select_level1<true>, grid1, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld,
                       gains, w.hdr, w.hist_lv + kBins, w.pguess, w.rowstate, w.active, w.cand_key, w.cand_row, w.bsum_hi,
                       objrow);
        else
            launch_pdl(select_level1<false>, grid1, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld,
                       gains, w.hdr, w.hist_lv + kBins, w.pguess, w.rowstate, w.active, w.cand_key, w.cand_row, w.bsum_hi,
                       objrow);
        mark_stage(3, s);
        {
            int64_t N_ = N, B_ = B, NB_ = NB;
            int32_t ld_ = ld;
            AllocHeader *hdr_ = w.hdr;
            unsigned long long *hist_ = w.hist_lv;
            int2 *rowstate_ = w.rowstate;
            const int32_t *active_ = w.active;
            long long *bhi_ = w.bsum_hi, *bt_ = w.bsum_t;
            const unsigned long long *ck_ = w.cand_key;
            const int32_t *cr_ = w.cand_row;
            void *args[] = {&N_, &ld_, &gains, &B_, &hdr_, &hist_, &rowstate_, &active_, &bhi_, &bt_, &NB_, &ck_, &cr_};
            if (cudaLaunchCooperativeKernel(reinterpret_cast<void *>(select_tail), dim3(tail_grid), dim3(kSelThreads), args,
                                            0, s) != cudaSuccess) {
                // the passes before it are already enqueued: mark the call failed on the device, so that the
                // output pass below leaves zeroed outputs and the status in info_dev
                (void)cudaGetLastError();
                fail_call<<<1, 1, 0, s>>>(w.hdr, HORA_ERR_CUDA);
                launch_failed = true;
            }
        }
        mark_stage(4, s);
        if (exact) {
            launch_pdl(exact_collect, grid_rows, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld,
                       gains, w.hdr, w.rowstate, w.rowslot, w.tkeys, w.tcounts, objrow);
            if (cudaFuncSetAttribute(exact_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kExactRankSmem) !=
                cudaSuccess)
                launch_failed = true;
            launch_pdl(exact_rank, 1, kExactRankThreads, kExactRankSmem, s, B, w.hdr, w.tkeys, w.tcounts, w.tlabel);
            launch_pdl(select_sum, (int)NB, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, 0, N, ld, gains,
                       2, B, w.hdr, w.rowstate, w.rowslot, w.tlabel, w.bsum_hi, w.bsum_t, NB);
        }
    } else {
        if (cudaMemsetAsync(w.rowstate, 0, sizeof(int2) * (size_t)N, s) != cudaSuccess) return HORA_ERR_CUDA;
        launch_pdl(select_sum, (int)NB, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, 1, N, ld, gains, 0,
                   B, w.hdr, w.rowstate, nullptr, nullptr, w.bsum_hi, w.bsum_t, NB);
    }
    mark_stage(5, s);
    const int out_vec = ((reinterpret_cast<uintptr_t>(delta) | reinterpret_cast<uintptr_t>(G) |
                          reinterpret_cast<uintptr_t>(group_offsets)) & 15u) == 0;
    launch_pdl(select_out, (int)NB, kSelThreads, 0, s, alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, B, flags,
               w.hdr, w.rowstate, objrow, w.bsum_hi, w.bsum_t, w.objpart, NB, delta, G, group_offsets, out_vec, info_dev);
    mark_stage(6, s);
    count_launches(B > 0 ? (exact ? 9 : 6) : 3);
    if (launch_failed) return HORA_ERR_CUDA;
    return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------------
// hora_allocate_static: the same allocation with the scratch held by the library itself.
//
// The scratch is a file-scope device array, so it exists on every GPU that loads this library from the
// moment the module is loaded until the process ends, and no allocation call is ever made on its behalf.
// Host code cannot hand the array's NAME to a kernel: on the host that name is only a stand-in for the
// symbol, not an address the GPU understands.  The device address is looked up once per device with
// cudaGetSymbolAddress and cached.
namespace hora {

constexpr size_t kStaticScratchBytes = (size_t)8 << 20;     // 8 MiB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::atomic<void *> g_static_scratch_addr[kMaxDevices];

// Device address of the scratch array on the current device (nullptr on failure).
static void *static_scratch_address() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void *p = g_static_scratch_addr[dev].load(std::memory_order_acquire);
    if (p != nullptr) return p;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return nullptr;
    g_static_scratch_addr[dev].store(p, std::memory_order_release);
    return p;
}

}  // namespace hora

extern "C" size_t hora_allocate_static_capacity(void) { return hora::kStaticScratchBytes; }

extern "C" hora_status_t hora_allocate_static(const double *alpha, const double *beta, double alpha0, double beta0,
                                              const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                                              int64_t N, int32_t ld, const double *gains, int64_t B, uint32_t flags,
                                              int32_t *delta, int32_t *G, int64_t *group_offsets,
                                              hora_alloc_info *info_dev, void *stream) {
    using namespace hora;
    if (N < 0 || ld < 1) return HORA_ERR_INVALID_ARG;
    // the problem must fit the built-in scratch; say so before touching the device
    const size_t need = hora_allocate_workspace_bytes(N, ld, gains == nullptr ? 1 : 0, flags);
    if (need > kStaticScratchBytes) return HORA_ERR_WORKSPACE;
    void *scratch = static_scratch_address();
    if (scratch == nullptr) return HORA_ERR_CUDA;
    return hora_allocate(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, B, flags, delta, G,
                         group_offsets, info_dev, scratch, kStaticScratchBytes, stream);
}
