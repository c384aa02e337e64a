// Learned-prior front end (appendix "Prior-design predictor details", Eq. posterior-learned): a predictor gives a
// success-rate estimate p_hat_i and, for the dual-head variants, a confidence s_i (softplus of a raw head output,
// clamped to [0.25, 16]; the single-head variants use a fixed s = 2).  The prior is Beta(s p_hat, s (1 - p_hat));
// the posterior of Eq. posterior-learned follows when hora_gains / hora_allocate add the Phase-A counts.
// Also the per-prompt Beta-Binomial negative log-likelihood those predictors are trained with.
// Both are one thread per prompt; the probes themselves are outside this library.
#include "hora_common.cuh"

namespace hora {

constexpr double kSMin = 0.25, kSMax = 16.0;

__device__ __forceinline__ double confidence(const double *s_raw, double s_fixed, int64_t i) {
    if (s_raw == nullptr) return s_fixed;
    const double x = __ldg(s_raw + i);
    const double sp = x > 0.0 ? x + log1p(exp(-x)) : log1p(exp(x));      // softplus, overflow-free
    return sp < kSMin ? kSMin : (sp > kSMax ? kSMax : sp);
}

__global__ void learned_prior_kernel(const double *__restrict__ p_hat, const double *__restrict__ s_raw, double s_fixed,
                                     int64_t N, double *__restrict__ alpha, double *__restrict__ beta,
                                     int32_t *status_dev) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const double p = __ldg(p_hat + i);
    const double s = confidence(s_raw, s_fixed, i);
    const bool ok = p > 0.0 && p < 1.0 && s > 0.0 && s < 1.0e300;
    if (!ok) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
    alpha[i] = ok ? s * p : 0.0;
    beta[i] = ok ? s * (1.0 - p) : 0.0;
}

// log B(x, y)
__device__ __forceinline__ double lbeta(double x, double y) { return lgamma(x) + lgamma(y) - lgamma(x + y); }

__global__ void beta_binomial_nll_kernel(const double *__restrict__ p_hat, const double *__restrict__ s_raw,
                                         double s_fixed, const int32_t *__restrict__ c, int32_t G0, int64_t N,
                                         double *__restrict__ nll, int32_t *status_dev) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const double p = __ldg(p_hat + i);
    const double s = confidence(s_raw, s_fixed, i);
    const int32_t ci = __ldg(c + i);
    const bool ok = p > 0.0 && p < 1.0 && s > 0.0 && s < 1.0e300 && ci >= 0 && ci <= G0;
    if (!ok) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
    const double a = s * p, b = s * (1.0 - p);
    nll[i] = ok ? -(lbeta((double)ci + a, (double)(G0 - ci) + b) - lbeta(a, b)) : 0.0;
}

}  // namespace hora

extern "C" hora_status_t hora_learned_prior(const double *p_hat, const double *s_raw, double s_fixed, int64_t N,
                                            double *alpha, double *beta, int32_t *status_dev, void *stream) {
    using namespace hora;
    if (N < 0 || (s_raw == nullptr && !(s_fixed > 0.0 && s_fixed < 1.0e300))) return HORA_ERR_INVALID_ARG;
    if (N == 0) return HORA_OK;
    if (p_hat == nullptr || alpha == nullptr || beta == nullptr) return HORA_ERR_INVALID_ARG;
    const int64_t grid = (N + 255) / 256;
    if (grid > 0x7FFFFFFF) return HORA_ERR_INVALID_ARG;
    learned_prior_kernel<<<(int)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(p_hat, s_raw, s_fixed, N, alpha, beta,
                                                                               status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}

extern "C" hora_status_t hora_beta_binomial_nll(const double *p_hat, const double *s_raw, double s_fixed,
                                                const int32_t *c, int32_t G0, int64_t N, double *nll,
                                                int32_t *status_dev, void *stream) {
    using namespace hora;
    if (N < 0 || G0 < 0 || (s_raw == nullptr && !(s_fixed > 0.0 && s_fixed < 1.0e300))) return HORA_ERR_INVALID_ARG;
    if (N == 0) return HORA_OK;
    if (p_hat == nullptr || c == nullptr || nll == nullptr) return HORA_ERR_INVALID_ARG;
    const int64_t grid = (N + 255) / 256;
    if (grid > 0x7FFFFFFF) return HORA_ERR_INVALID_ARG;
    beta_binomial_nll_kernel<<<(int)grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(p_hat, s_raw, s_fixed, c, G0, N, nll,
                                                                                   status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}
