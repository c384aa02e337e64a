// hora_token_broadcast: replicate each rollout's advantage over its tokens (Eq. grpo-objective: the
// per-token advantage has no dependence on the token position).
//
// Output-centric streaming write.  The token axis is cut into one contiguous chunk per CTA (a
// multiple of 1024 tokens, so every 16-byte store is aligned).  A CTA locates the rollout that
// contains its first token with a block-wide k-ary search over the CSR offsets, then repeatedly
// stages the next kStage+1 offsets in shared memory and writes the tokens they cover: a warp
// writes 128 consecutive tokens per step (one float4 per lane, st.global.cs), keeping a rollout
// cursor that only moves forward.  Cost per token is independent of the length mix; the only
// global reads are the offsets (8 B per rollout, once) and the advantages (4 B per rollout).
// Runs of very short rollouts that outrun the staged window are still handled (the cursor then
// reads offsets from global memory), only more slowly.
#include "hora_common.cuh"

namespace hora {

constexpr int kBcThreads = 256;
constexpr int kBcWarps = kBcThreads / kWarp;
constexpr int kStage = 1024;                            // rollouts staged per round (plus the closing offset)
constexpr int kWarpTokens = 128;                        // tokens one warp writes per step
constexpr int kStepTokens = kBcWarps * kWarpTokens;     // tokens the CTA writes per step

// Largest r in [0, R] with off[r] <= t (off is non-decreasing, off[0] <= t).  All threads return it.
__device__ int64_t block_find_rollout(const int64_t *__restrict__ off, int64_t R, int64_t t,
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

template <bool VEC4>
__global__ void __launch_bounds__(kBcThreads)
token_broadcast_kernel(const float *__restrict__ adv, const int64_t *__restrict__ off, int64_t R, int64_t T,
                       int64_t chunk, float *__restrict__ out) {
    __shared__ int64_t s_off[kStage + 1];
    __shared__ unsigned long long s_bounds[2];
    const int64_t t_all = __ldg(off + R);
    if (t_all < T) T = t_all;                           // never write past the last rollout
    const int64_t c0 = (int64_t)blockIdx.x * chunk;
    if (c0 >= T) return;
    const int64_t c1 = (c0 + chunk < T) ? c0 + chunk : T;
    const int lane = lane_id(), warp = threadIdx.x >> 5;

    int64_t r_base = block_find_rollout(off, R, c0, s_bounds);
    if (r_base >= R) r_base = R - 1;                    // cannot happen while c0 < off[R]; keeps reads in range
    int64_t t = c0;
    while (t < c1) {
        const int64_t n_stage = (R - r_base < kStage) ? R - r_base : kStage;
        __syncthreads();
        for (int64_t j = threadIdx.x; j <= n_stage; j += kBcThreads) s_off[j] = __ldg(off + r_base + j);
        __syncthreads();
        // offset of rollout r (r_base <= r <= R): shared memory inside the staged window, global beyond it
        auto off_at = [&](int64_t r) -> int64_t {
            const int64_t j = r - r_base;
            return (j <= n_stage) ? s_off[j] : __ldg(off + r);
        };
        const int64_t staged_end = s_off[n_stage] / kWarpTokens * kWarpTokens;
        int64_t t_end = (staged_end > t + kStepTokens) ? staged_end : t + kStepTokens;
        if (t_end > c1) t_end = c1;

        int64_t cur = r_base;                           // warp-uniform: off[cur] <= every token this warp still writes
        for (int64_t w0 = t + (int64_t)warp * kWarpTokens; w0 < t_end; w0 += kStepTokens) {
            while (cur + 1 < R && off_at(cur + 1) <= w0) ++cur;
            const int64_t t0 = w0 + lane * 4;
            if (t0 >= t_end) continue;
            int64_t r = cur;
            while (r + 1 < R && off_at(r + 1) <= t0) ++r;
            float v0 = __ldg(adv + r), v1 = v0, v2 = v0, v3 = v0;
            if (r + 1 < R && off_at(r + 1) < t0 + 4) {   // a rollout boundary falls inside these four tokens
                while (r + 1 < R && off_at(r + 1) <= t0 + 1) ++r;
                v1 = __ldg(adv + r);
                while (r + 1 < R && off_at(r + 1) <= t0 + 2) ++r;
                v2 = __ldg(adv + r);
                while (r + 1 < R && off_at(r + 1) <= t0 + 3) ++r;
                v3 = __ldg(adv + r);
            }
            if (VEC4 && t0 + 4 <= t_end) {
                __stcs(reinterpret_cast<float4 *>(out + t0), make_float4(v0, v1, v2, v3));
            } else {
                if (t0 < t_end) out[t0] = v0;
                if (t0 + 1 < t_end) out[t0 + 1] = v1;
                if (t0 + 2 < t_end) out[t0 + 2] = v2;
                if (t0 + 3 < t_end) out[t0 + 3] = v3;
            }
        }
        if (t_end >= c1) break;
        // rollout containing t_end: binary search inside the stage, forward walk beyond it
        int64_t nr;
        if (t_end < s_off[n_stage]) {
            int64_t lo = 0, hi = n_stage - 1;           // s_off[0] <= t < t_end
            while (lo < hi) {
                const int64_t mid = (lo + hi + 1) >> 1;
                if (s_off[mid] <= t_end) lo = mid; else hi = mid - 1;
            }
            nr = r_base + lo;
        } else {
            nr = r_base + n_stage - 1;
            while (nr + 1 < R && __ldg(off + nr + 1) <= t_end) ++nr;
        }
        r_base = nr;
        t = t_end;
    }
}

}  // namespace hora

extern "C" hora_status_t hora_token_broadcast(const float *adv, const int64_t *token_offsets, int64_t R, int64_t T,
                                              float *token_adv, void *stream) {
    using namespace hora;
    if (R < 0 || T < 0) return HORA_ERR_INVALID_ARG;
    if (R == 0 || T == 0) return HORA_OK;
    if (adv == nullptr || token_offsets == nullptr || token_adv == nullptr) return HORA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(token_adv) & 3u) return HORA_ERR_INVALID_ARG;
    const int64_t max_ctas = (int64_t)kSmCount * 8;
    int64_t chunk = (T + max_ctas - 1) / max_ctas;
    chunk = (chunk + kStepTokens - 1) / kStepTokens * kStepTokens;
    const int grid = (int)((T + chunk - 1) / chunk);
    const bool vec4 = (reinterpret_cast<uintptr_t>(token_adv) & 15u) == 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (vec4)
        token_broadcast_kernel<true><<<grid, kBcThreads, 0, s>>>(adv, token_offsets, R, T, chunk, token_adv);
    else
        token_broadcast_kernel<false><<<grid, kBcThreads, 0, s>>>(adv, token_offsets, R, T, chunk, token_adv);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
