// hora_group_advantage_tokens: per-token advantages (and, optionally, per-token loss weights) straight from the
// rewards, without the per-rollout advantage array in between (Sec. 3.1 and Eq. grpo-objective: the advantage is
// computed over the prompt's group and is the same for every token of a rollout; Sec. 3.2, variable-size groups:
// the 1/G factor becomes 1/G_i).
//
// Same output-centric scheme as hora_token_broadcast: one contiguous token chunk per CTA, rollouts staged in
// shared memory round by round, 128-token windows written with 16-byte streaming stores.  What differs is where
// the staged values come from: the CTA finds the group of its first staged rollout with the same block-wide
// search (over the group offsets), and its warps take the groups that intersect the staged rollouts one each:
// a warp reads the whole group's rewards (they are a few KB and come from L2), forms mean and scale in fp64, and
// fills the advantage — and the weight 1/(G_g * len_r) or 1/(G_g * L) — of the group's staged rollouts.  A group
// that straddles two chunks has its statistics computed by both CTAs; that costs reward reads (4 B per rollout
// against ~4 KB of tokens written per rollout), no synchronisation, and the result is the same on both sides.
#include "hora_broadcast.cuh"
#include "hora_group_stats.cuh"

namespace hora {

template <bool VEC4, bool WEIGHT>
__global__ void __launch_bounds__(kBcThreads)
advantage_tokens_kernel(const float *__restrict__ rewards, const int64_t *__restrict__ goff, int64_t N,
                        const int64_t *__restrict__ off, int64_t R, int64_t T, int64_t chunk, int32_t mode, double eps,
                        int32_t ddof, int32_t weight_mode, double length_const, float *__restrict__ out,
                        float *__restrict__ out_w, int32_t *status_dev) {
    pdl_enter();
    __shared__ int32_t s_rel[kStage + 1];
    __shared__ float s_adv[kStage];
    __shared__ float s_w[WEIGHT ? kStage : 1];
    __shared__ unsigned long long s_bounds[2];
    __shared__ int s_need;
    const int64_t t_all = __ldg(off + R);
    if (t_all < T) T = t_all;
    const int64_t c0 = (int64_t)blockIdx.x * chunk;
    if (c0 >= T) return;
    const int32_t len = (int32_t)((c0 + chunk < T ? c0 + chunk : T) - c0);
    const int lane = lane_id(), warp = threadIdx.x >> 5;

    int64_t r_base = block_find_rollout(off, R, c0, s_bounds);
    int32_t t = 0;
    while (t < len && r_base < R) {
        const int n_stage = (int)((R - r_base < kStage) ? R - r_base : kStage);
        __syncthreads();
        if (threadIdx.x == 0) s_need = 0;
        for (int j = threadIdx.x; j <= n_stage; j += kBcThreads) {
            const int64_t d = __ldg(off + r_base + j) - c0;
            s_rel[j] = d < 0 ? -1 : (d > len ? len : (int32_t)d);
        }
        __syncthreads();
        // staged rollouts that start before the chunk ends: the only ones whose values are read below
        for (int j = threadIdx.x; j < n_stage; j += kBcThreads)
            if (s_rel[j] < len && (j + 1 == n_stage || s_rel[j + 1] >= len)) s_need = j + 1;
        __syncthreads();
        const int n_need = s_need;
        if (n_need == 0) break;                                            // cannot happen for valid offsets
        const int64_t r_end = r_base + n_need;
        // group of the first staged rollout: the largest g with goff[g] <= r_base (skips empty groups before it)
        const int64_t g_first = block_find_rollout(goff, N, r_base, s_bounds);
        for (int j = threadIdx.x; j < n_need; j += kBcThreads) {           // rollouts beyond the last group
            s_adv[j] = 0.0f;
            if (WEIGHT) s_w[j] = 0.0f;
        }
        __syncthreads();
        for (int64_t g = g_first + warp; g < N; g += kBcWarps) {
            const int64_t s = __ldg(goff + g), e = __ldg(goff + g + 1);
            if (s >= r_end) break;
            if (e < s || s < 0) { raise_status(status_dev, HORA_ERR_INVALID_VALUE); continue; }
            if (e == s || e <= r_base) continue;
            double mean, scale;
            group_mean_scale(rewards, s, e, mode, eps, ddof, lane, mean, scale);
            const int64_t j0 = s > r_base ? s : r_base, j1 = e < r_end ? e : r_end;
            for (int64_t j = j0 + lane; j < j1; j += kWarp) {
                s_adv[j - r_base] = (float)(((double)__ldg(rewards + j) - mean) * scale);
                if (WEIGHT) {
                    double denom = (double)(e - s) * length_const;
                    if (weight_mode == HORA_WEIGHT_PER_TOKEN) denom = (double)(e - s) * (double)(__ldg(off + j + 1) - __ldg(off + j));
                    s_w[j - r_base] = denom > 0.0 ? (float)(1.0 / denom) : 0.0f;
                }
            }
        }
        __syncthreads();
        const int32_t t_end = s_rel[n_need];                               // tokens covered by the needed rollouts
        write_staged<VEC4>(s_rel, s_adv, n_need, t, t_end, warp, lane, out + c0);
        if (WEIGHT) write_staged<VEC4>(s_rel, s_w, n_need, t, t_end, warp, lane, out_w + c0);
        r_base += n_need;
        t = t_end > t ? t_end : t;
    }
}

}  // namespace hora

extern "C" hora_status_t hora_group_advantage_tokens(const float *rewards, const int64_t *group_offsets, int64_t N,
                                                     const int64_t *token_offsets, int64_t R, int64_t T, int32_t mode,
                                                     float eps, int32_t ddof, int32_t weight_mode, float length_const,
                                                     float *token_adv, float *token_weight, int32_t *status_dev,
                                                     void *stream) {
    using namespace hora;
    if (N < 0 || R < 0 || T < 0 || (mode != HORA_ADV_GRPO && mode != HORA_ADV_RLOO) || (ddof != 0 && ddof != 1) ||
        !(eps >= 0.0f))
        return HORA_ERR_INVALID_ARG;
    if (token_weight != nullptr) {
        if (weight_mode != HORA_WEIGHT_PER_TOKEN && weight_mode != HORA_WEIGHT_CONST_LENGTH) return HORA_ERR_INVALID_ARG;
        if (weight_mode == HORA_WEIGHT_CONST_LENGTH && !(length_const > 0.0f)) return HORA_ERR_INVALID_ARG;
    }
    if (R == 0 || T == 0) return HORA_OK;
    if (rewards == nullptr || group_offsets == nullptr || token_offsets == nullptr || token_adv == nullptr)
        return HORA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(token_adv) & 3u) || (reinterpret_cast<uintptr_t>(token_weight) & 3u))
        return HORA_ERR_INVALID_ARG;
    const int64_t chunk = token_chunk(T);
    const int64_t grid = (T + chunk - 1) / chunk;
    if (grid > 0x7FFFFFFF) return HORA_ERR_INVALID_ARG;
    const bool vec4 = ((reinterpret_cast<uintptr_t>(token_adv) | reinterpret_cast<uintptr_t>(token_weight)) & 15u) == 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#define HORA_LAUNCH_AT(V, W)                                                                                        \
    launch_pdl(advantage_tokens_kernel<V, W>, (int)grid, kBcThreads, 0, st, rewards, group_offsets, N, token_offsets, \
               R, T, chunk, mode, (double)eps, ddof, weight_mode, (double)length_const, token_adv, token_weight,      \
               status_dev)
    if (token_weight != nullptr) { if (vec4) HORA_LAUNCH_AT(true, true); else HORA_LAUNCH_AT(false, true); }
    else                         { if (vec4) HORA_LAUNCH_AT(true, false); else HORA_LAUNCH_AT(false, false); }
#undef HORA_LAUNCH_AT
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
