// hora_pass_at_k: the unbiased Pass@K estimator of Eq. pass-k, averaged over prompts, for a grid of K:
//     Pass@K = mean_q [ 1 - C(n - c_q, K) / C(n, K) ],   c_q correct samples out of n.
// Two small kernels: a histogram of the counts c_q (values 0..n), then one CTA per K that evaluates
// 1 - prod_{i<K} (n - c - i)/(n - i) for every count value and sums value * multiplicity in a fixed order
// (so the mean is bitwise reproducible).  C(n-c, K) = 0 when n - c < K: the product then meets a zero factor.
#include "hora_common.cuh"

namespace hora {

constexpr int kPkThreads = 256;

__global__ void __launch_bounds__(kPkThreads)
passk_histogram(const int32_t *__restrict__ c, int64_t Q, int32_t n, unsigned long long *hist, int32_t *status_dev) {
    const int64_t stride = (int64_t)gridDim.x * kPkThreads;
    for (int64_t q = (int64_t)blockIdx.x * kPkThreads + threadIdx.x; q < Q; q += stride) {
        const int32_t v = __ldg(c + q);
        if (v < 0 || v > n) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
        else atomicAdd(hist + v, 1ull);
    }
}

__global__ void __launch_bounds__(kPkThreads)
passk_evaluate(const unsigned long long *__restrict__ hist, int64_t Q, int32_t n, const int32_t *__restrict__ K,
               double *__restrict__ out, int32_t *status_dev) {
    __shared__ double s_part[kPkThreads];
    const int32_t k = __ldg(K + blockIdx.x);
    if (k < 0 || k > n) {                                    // uniform over the CTA
        if (threadIdx.x == 0) { raise_status(status_dev, HORA_ERR_INVALID_VALUE); out[blockIdx.x] = 0.0; }
        return;
    }
    double part = 0.0;
    for (int32_t cv = threadIdx.x; cv <= n; cv += kPkThreads) {
        const unsigned long long cnt = hist[cv];
        if (cnt == 0) continue;
        double ratio = 1.0;                                  // C(n - cv, k) / C(n, k)
        for (int32_t i = 0; i < k; ++i) {
            const int32_t num = n - cv - i;
            if (num <= 0) { ratio = 0.0; break; }
            ratio *= (double)num / (double)(n - i);
        }
        part += (1.0 - ratio) * (double)cnt;
    }
    s_part[threadIdx.x] = part;
    __syncthreads();
    for (int d = kPkThreads / 2; d >= 1; d >>= 1) {
        if (threadIdx.x < d) s_part[threadIdx.x] += s_part[threadIdx.x + d];
        __syncthreads();
    }
    if (threadIdx.x == 0) out[blockIdx.x] = Q > 0 ? s_part[0] / (double)Q : 0.0;
}

}  // namespace hora

extern "C" size_t hora_pass_at_k_workspace_bytes(int32_t n_samples) {
    return n_samples < 0 ? 0 : sizeof(unsigned long long) * ((size_t)n_samples + 1);
}

extern "C" hora_status_t hora_pass_at_k(const int32_t *c, int64_t Q, int32_t n_samples, const int32_t *K_dev,
                                        int32_t n_K, double *pass_at_k, int32_t *status_dev, void *workspace,
                                        size_t workspace_bytes, void *stream) {
    using namespace hora;
    if (Q < 0 || n_samples < 1 || n_K < 0) return HORA_ERR_INVALID_ARG;
    if (n_K == 0) return HORA_OK;
    if ((Q > 0 && c == nullptr) || K_dev == nullptr || pass_at_k == nullptr) return HORA_ERR_INVALID_ARG;
    if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 7u) ||
        workspace_bytes < hora_pass_at_k_workspace_bytes(n_samples))
        return HORA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long *hist = static_cast<unsigned long long *>(workspace);
    if (cudaMemsetAsync(hist, 0, hora_pass_at_k_workspace_bytes(n_samples), s) != cudaSuccess) return HORA_ERR_CUDA;
    if (Q > 0) passk_histogram<<<clamp_grid((Q + kPkThreads - 1) / kPkThreads, 8), kPkThreads, 0, s>>>(c, Q, n_samples, hist, status_dev);
    passk_evaluate<<<n_K, kPkThreads, 0, s>>>(hist, Q, n_samples, K_dev, pass_at_k, status_dev);
    count_launches(Q > 0 ? 2 : 1);
    return cuda_ok(cudaGetLastError());
}
