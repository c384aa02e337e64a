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
// s_rel[n_stage]).  Tokens are visited in 128-token windows on an absolute 128-aligned grid, one window per warp
// per step; a window that lies inside one rollout is one broadcast 16-byte store per lane.
template <bool VEC4>
__device__ __forceinline__ void write_staged(const int32_t *s_rel, const float *s_val, int n_stage, int32_t t,
                                             int32_t t_end, int warp, int lane, float *__restrict__ dst) {
    int cur = 0;                                    // warp-uniform, forward only: s_rel[cur] <= window start
    for (int32_t w0 = (t & ~(kWarpTokens - 1)) + warp * kWarpTokens; w0 < t_end; w0 += kStepTokens) {
        while (cur + 1 < n_stage && s_rel[cur + 1] <= w0) ++cur;
        const int32_t t0 = w0 + lane * 4;
        if (w0 >= t && w0 + kWarpTokens <= t_end && s_rel[cur + 1] >= w0 + kWarpTokens) {
            const float v = s_val[cur];             // the whole window lies inside rollout `cur`
            if (VEC4) {
                __stcs(reinterpret_cast<float4 *>(dst + t0), make_float4(v, v, v, v));
            } else {
                dst[t0] = v; dst[t0 + 1] = v; dst[t0 + 2] = v; dst[t0 + 3] = v;
            }
            continue;
        }
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
    }
}

}  // namespace hora
