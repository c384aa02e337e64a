// hora_rollout_weights: the loss weight of every rollout under variable-size groups (Sec. 3.2, "Training
// objective with variable-size groups": 1/G is replaced by 1/G_i so that each prompt weighs the same however
// many rollouts it received; Eq. grpo-objective has the further factor 1/|o| per response).
//
// A warp takes 32 consecutive groups (lane i reads group i's two offsets, coalesced), then walks each group
// with all lanes: weight = 1 / (G_g * len_r) or 1 / (G_g * length_const), computed in fp64 with one division
// and rounded to fp32.  Memory bound and tiny next to the rest of the path (12 bytes per rollout).
#include "hora_common.cuh"

namespace hora {

constexpr int kWWarps = 8;

__global__ void __launch_bounds__(kWWarps *kWarp)
rollout_weights_kernel(const int64_t *__restrict__ goff, int64_t N, const int64_t *__restrict__ toff, int32_t mode,
                       double length_const, float *__restrict__ weights, int32_t *status_dev) {
    const int lane = lane_id();
    const int64_t warp0 = (int64_t)blockIdx.x * kWWarps + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * kWWarps;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    for (int64_t blk = warp0; blk < n_blocks; blk += stride) {
        const int64_t g0 = blk * kWarp;
        const int ng = (int)((N - g0 < kWarp) ? N - g0 : kWarp);
        int64_t my_s = 0, my_e = 0;
        if (lane < ng) {
            my_s = __ldg(goff + g0 + lane);
            my_e = __ldg(goff + g0 + lane + 1);
        }
        if (my_e < my_s || my_s < 0) {
            raise_status(status_dev, HORA_ERR_INVALID_VALUE);
            my_e = my_s;
        }
        for (int i = 0; i < ng; ++i) {
            const int64_t s = __shfl_sync(kFull, my_s, i), e = __shfl_sync(kFull, my_e, i);
            const double G = (double)(e - s);
            for (int64_t r = s + lane; r < e; r += kWarp) {
                double denom = G * length_const;
                if (mode == HORA_WEIGHT_PER_TOKEN) {
                    const int64_t len = __ldg(toff + r + 1) - __ldg(toff + r);
                    if (len < 0) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
                    denom = G * (double)len;
                }
                weights[r] = denom > 0.0 ? (float)(1.0 / denom) : 0.0f;
            }
        }
    }
}

}  // namespace hora

extern "C" hora_status_t hora_rollout_weights(const int64_t *group_offsets, int64_t N, const int64_t *token_offsets,
                                              int32_t mode, float length_const, float *weights, int32_t *status_dev,
                                              void *stream) {
    using namespace hora;
    if (N < 0 || (mode != HORA_WEIGHT_PER_TOKEN && mode != HORA_WEIGHT_CONST_LENGTH)) return HORA_ERR_INVALID_ARG;
    if (mode == HORA_WEIGHT_CONST_LENGTH && !(length_const > 0.0f)) return HORA_ERR_INVALID_ARG;
    if (N == 0) return HORA_OK;
    if (group_offsets == nullptr || weights == nullptr) return HORA_ERR_INVALID_ARG;
    if (mode == HORA_WEIGHT_PER_TOKEN && token_offsets == nullptr) return HORA_ERR_INVALID_ARG;
    const int64_t n_blocks = (N + kWarp - 1) / kWarp;
    const int grid = clamp_grid((n_blocks + kWWarps - 1) / kWWarps, 8);
    rollout_weights_kernel<<<grid, kWWarps * kWarp, 0, static_cast<cudaStream_t>(stream)>>>(
        group_offsets, N, token_offsets, mode, (double)length_const, weights, status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
