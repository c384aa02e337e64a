// hora_token_broadcast: replicate each rollout's advantage over its tokens (Eq. grpo-objective: the
// per-token advantage has no dependence on the token position).
//
// Output-centric streaming write.  The token axis is cut into contiguous chunks, one per CTA (a
// multiple of 1024 tokens, at most 65536).  A CTA locates the rollout that contains its first token with a
// block-wide k-ary search over the CSR offsets, then works in rounds: it stages the next kStage
// rollouts in shared memory — offsets as 32-bit distances from the chunk start, advantages as they
// are — and writes every token those rollouts cover.  Tokens are visited in 128-token windows on an
// absolute 128-aligned grid, one 16-byte st.global.cs per lane and window; a warp takes a contiguous run
// of windows, so while it is inside one rollout (the usual case for responses of tens to thousands of
// tokens) it stores one broadcast value window after window and never looks at the offsets.  Cost per token does not depend on the length mix; the only global
// reads are 8 B of offset and 4 B of advantage per rollout.
#include "hora_broadcast.cuh"

namespace hora {

template <bool VEC4>
__global__ void __launch_bounds__(kBcThreads)
token_broadcast_kernel(const float *__restrict__ adv, const int64_t *__restrict__ off, int64_t R, int64_t T,
                       int64_t chunk, float *__restrict__ out) {
    pdl_enter();
    __shared__ int32_t s_rel[kStage + 1];               // offsets relative to the chunk start, clamped to [-1, len]
    __shared__ float s_adv[kStage];
    __shared__ unsigned long long s_bounds[2];
    const int64_t t_all = __ldg(off + R);
    if (t_all < T) T = t_all;                           // never write past the last rollout
    const int64_t c0 = (int64_t)blockIdx.x * chunk;
    if (c0 >= T) return;
    const int32_t len = (int32_t)((c0 + chunk < T ? c0 + chunk : T) - c0);   // tokens of this chunk
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    float *__restrict__ dst = out + c0;

    int64_t r_base = block_find_rollout(off, R, c0, s_bounds);   // off[r_base] <= c0
    int32_t t = 0;                                      // next token (chunk-relative) not yet written
    while (t < len && r_base < R) {
        const int n_stage = (int)((R - r_base < kStage) ? R - r_base : kStage);
        __syncthreads();
        for (int j = threadIdx.x; j <= n_stage; j += kBcThreads) {
            const int64_t d = __ldg(off + r_base + j) - c0;
            s_rel[j] = d < 0 ? -1 : (d > len ? len : (int32_t)d);
            if (j < n_stage) s_adv[j] = __ldg(adv + r_base + j);
        }
        __syncthreads();
        const int32_t t_end = s_rel[n_stage];           // the staged rollouts cover tokens [t, t_end)
        write_staged<VEC4>(s_rel, s_adv, n_stage, t, t_end, warp, lane, dst);
        r_base += n_stage;
        t = t_end > t ? t_end : t;
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
    const int64_t chunk = token_chunk(T);
    const int64_t grid = (T + chunk - 1) / chunk;
    if (grid > 0x7FFFFFFF) return HORA_ERR_INVALID_ARG;
    const bool vec4 = (reinterpret_cast<uintptr_t>(token_adv) & 15u) == 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (vec4)
        launch_pdl(token_broadcast_kernel<true>, (int)grid, kBcThreads, 0, s, adv, token_offsets, R, T, chunk, token_adv);
    else
        launch_pdl(token_broadcast_kernel<false>, (int)grid, kBcThreads, 0, s, adv, token_offsets, R, T, chunk, token_adv);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
