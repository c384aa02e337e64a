// hora_allocation_share: the statistic behind Fig. 3 — for every Phase-A success count k = 0..G0 the number of
// prompts with c_i = k and the Phase-B rollouts they received (Sec. 4.1).  Integer histogram: per-CTA bins in
// shared memory, one 64-bit global atomic per non-empty bin per CTA; the result does not depend on the order.
#include "hora_common.cuh"

namespace hora {

constexpr int kShareThreads = 256;
constexpr int kShareMaxG0 = 2047;                      // 2 x 2048 64-bit bins in shared memory

__global__ void __launch_bounds__(kShareThreads)
allocation_share_kernel(const int32_t *__restrict__ c, const int32_t *__restrict__ delta, int64_t N, int32_t G0,
                        unsigned long long *prompts, unsigned long long *budget, int32_t *status_dev) {
    __shared__ unsigned long long s_prompts[kShareMaxG0 + 1], s_budget[kShareMaxG0 + 1];
    for (int k = threadIdx.x; k <= G0; k += kShareThreads) { s_prompts[k] = 0; s_budget[k] = 0; }
    __syncthreads();
    // A warp folds equal counts together before it touches the bins: with G0 = 8 there are nine classes, and
    // 32 lanes hammering nine shared-memory words would serialise.
    const int lane = lane_id();
    const int64_t stride = (int64_t)gridDim.x * kShareThreads;
    for (int64_t base = (int64_t)blockIdx.x * kShareThreads + (threadIdx.x & ~(kWarp - 1)); base < N; base += stride) {
        const int64_t i = base + lane;
        int32_t ci = -1, di = 0;
        if (i < N) { ci = __ldg(c + i); di = __ldg(delta + i); }
        bool ok = i < N;
        if (ok && (ci < 0 || ci > G0 || di < 0)) { raise_status(status_dev, HORA_ERR_INVALID_VALUE); ok = false; }
        unsigned remaining = __ballot_sync(kFull, ok);
        while (remaining) {
            const int leader = __ffs(remaining) - 1;
            const int32_t k = __shfl_sync(kFull, ci, leader);
            const bool mine = ok && ci == k;
            const unsigned m = __ballot_sync(kFull, mine);
            const unsigned lo = __reduce_add_sync(kFull, mine ? (unsigned)di & 0xFFFFu : 0u);
            const unsigned hi = __reduce_add_sync(kFull, mine ? (unsigned)di >> 16 : 0u);
            if (lane == leader) {
                atomicAdd(&s_prompts[k], (unsigned long long)__popc(m));
                const unsigned long long sum = (unsigned long long)lo + ((unsigned long long)hi << 16);
                if (sum) atomicAdd(&s_budget[k], sum);
            }
            remaining &= ~m;
        }
    }
    __syncthreads();
    for (int k = threadIdx.x; k <= G0; k += kShareThreads) {
        if (s_prompts[k]) atomicAdd(prompts + k, s_prompts[k]);
        if (s_budget[k]) atomicAdd(budget + k, s_budget[k]);
    }
}

}  // namespace hora

extern "C" hora_status_t hora_allocation_share(const int32_t *c, const int32_t *delta, int64_t N, int32_t G0,
                                               int64_t *prompts, int64_t *budget, int32_t *status_dev, void *stream) {
    using namespace hora;
    if (N < 0 || G0 < 0 || G0 > kShareMaxG0) return HORA_ERR_INVALID_ARG;
    if (prompts == nullptr || budget == nullptr || (N > 0 && (c == nullptr || delta == nullptr))) return HORA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t bytes = sizeof(int64_t) * ((size_t)G0 + 1);
    if (cudaMemsetAsync(prompts, 0, bytes, s) != cudaSuccess || cudaMemsetAsync(budget, 0, bytes, s) != cudaSuccess)
        return HORA_ERR_CUDA;
    if (N == 0) return HORA_OK;
    allocation_share_kernel<<<clamp_grid((N + kShareThreads - 1) / kShareThreads, 4), kShareThreads, 0, s>>>(
        c, delta, N, G0, reinterpret_cast<unsigned long long *>(prompts), reinterpret_cast<unsigned long long *>(budget),
        status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
