// Shared pieces of the token-axis kernels (hora_token_broadcast, hora_group_advantage_tokens): the chunking
// constants, the block-wide offset search and the loop that writes the tokens of the staged rollouts.
#pragma once
#include "hora_common.cuh"

namespace hora {

constexpr int kBcThreads = 256;
constexpr int kBcWarps = kBcThreads / kWarp;
constexpr int kStage = 1024;                            // rollouts staged per round
constexpr int kWarpTokens = 128;                        // tokens one warp writes per step
constexpr int kStepTokens = kBcWarps * kWarpTokens;     // tokens the CTA writes per step
constexpr int64_t kMaxChunk = 1 << 30;                  // keeps chunk-relative offsets in 32 bits
constexpr int64_t kFrontChunk = 1 << 16;                // tokens per CTA when there are enough of them

// Tokens per CTA.  CTAs start in index order, so the ones resident at any moment write one moving front of
// adjacent chunks; with 256 KiB chunks that front stays within a few DRAM pages per channel, and the measured
// write rate is 6.3 TB/s against 5.5 TB/s for one long chunk per CTA slot (the same bytes spread over 1184
// distant streams).  Short token axes fall back to one chunk per CTA slot.
inline int64_t token_chunk(int64_t T) {
    const int64_t max_ctas = (int64_t)sm_count() * 8;
    int64_t chunk = (T + max_ctas - 1) / max_ctas;
    if (chunk > kFrontChunk) chunk = kFrontChunk;
    chunk = (chunk + kStepTokens - 1) / kStepTokens * kStepTokens;
    return chunk > kMaxChunk ? kMaxChunk : chunk;
}

// Largest r in [0, R] with off[r] <= t (off is non-decreasing, off[0] <= t).  All threads return it.
static __device__ int64_t block_find_rollout(const int64_t *__restrict__ off, int64_t R, int64_t t,
                                      unsigned long long *s_bounds) {
    int64_t lo = 0, hi = R;
    while (hi > lo) {
        __syncthreads();
        if (threadIdx.x == 0) { s_bounds[0] = (unsigned long long)lo; s_bounds[1] = (unsigned long long)hi; }
        __syncthreads();
        const int64_t step = (hi - lo + kBcThreads - 1) / kBcThreads;
        const int64_t probe = lo + (int64_t)(threadIdx.x + 1) * step;
        if (probe <= hi) {
            if (__ldg(off + probe) <= t) atomicMax(&s_bounds[0], (unsigned long long)probe);
            else atomicMin(&s_bounds[1], (unsigned long long)(probe - 1));
        }
        __syncthreads();
        lo = (int64_t)s_bounds[0];
        hi = (int64_t)s_bounds[1];
    }
    __syncthreads();
    return lo;
}

// Writes s_val[j] over the tokens of staged rollout j, for the chunk-relative tokens [t, t_end) (t_end =
// s_rel[n_stage]).  Tokens are visited in 128-token windows on an absolute 128-aligned grid; each warp takes a
// contiguous run of windows, so that it stays inside one rollout for many windows in a row: there the loop is
// one broadcast 16-byte store per lane and window and nothing else.  Only the window in which a rollout ends
// walks the offsets.
template <bool VEC4>
__device__ __forceinline__ void write_staged(const int32_t *s_rel, const float *s_val, int n_stage, int32_t t,
                                             int32_t t_end, int warp, int lane, float *__restrict__ dst) {
    const int32_t first = t & ~(kWarpTokens - 1);
    const int32_t n_win = (t_end - first + kWarpTokens - 1) / kWarpTokens;
    const int32_t share = (n_win + kBcWarps - 1) / kBcWarps;
    int32_t w0 = first + warp * share * kWarpTokens;
    int32_t w_end = w0 + share * kWarpTokens;                    // end of this warp's run of windows
    if (w_end > first + n_win * kWarpTokens) w_end = first + n_win * kWarpTokens;
    if (w0 >= w_end) return;
    int cur = 0;                                                 // warp-uniform: largest j with s_rel[j] <= w0 (else 0)
    for (int lo = 0, hi = n_stage - 1; lo <= hi;) {
        const int mid = (lo + hi) >> 1;
        if (s_rel[mid] <= w0) { cur = mid; lo = mid + 1; } else { hi = mid - 1; }
    }
    while (w0 < w_end) {
        while (cur + 1 < n_stage && s_rel[cur + 1] <= w0) ++cur;
        // whole windows inside rollout `cur` (and inside [t, t_end)), starting at w0
        int32_t stop = s_rel[cur + 1] < t_end ? s_rel[cur + 1] : t_end;
        if (stop > w_end) stop = w_end;
        int32_t n_full = (VEC4 && w0 >= t && stop > w0) ? (stop - w0) / kWarpTokens : 0;
        if (n_full > 0) {
            const float v = s_val[cur];
            const float4 vv = make_float4(v, v, v, v);
            float4 *p = reinterpret_cast<float4 *>(dst + w0) + lane;
            w0 += n_full * kWarpTokens;
            for (; n_full >= 4; n_full -= 4, p += 4 * (kWarpTokens / 4)) {
                __stcs(p, vv);
                __stcs(p + kWarpTokens / 4, vv);
                __stcs(p + 2 * (kWarpTokens / 4), vv);
                __stcs(p + 3 * (kWarpTokens / 4), vv);
            }
            for (; n_full > 0; --n_full, p += kWarpTokens / 4) __stcs(p, vv);
            continue;
        }
        // the window at w0 holds a rollout boundary, or an end of [t, t_end): every lane finds its own rollouts
        const int32_t t0 = w0 + lane * 4;
        int r = cur;
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            while (r + 1 < n_stage && s_rel[r + 1] <= t0 + q) ++r;
            v[q] = s_val[r];
        }
        if (VEC4 && t0 >= t && t0 + 4 <= t_end) {
            __stcs(reinterpret_cast<float4 *>(dst + t0), make_float4(v[0], v[1], v[2], v[3]));
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (t0 + q >= t && t0 + q < t_end) dst[t0 + q] = v[q];
        }
        w0 += kWarpTokens;
    }
}

}  // namespace hora
