// hora_gains: fp64 marginal-gain rows by a warp-level prefix product (Eq. marginal and its recurrence).
//
// With k = Delta-1 the row is an inclusive prefix product of factors phi_k = num_k / den_k,
//     num_0 = a,  num_k = b + k - 1 (k >= 1),   den_k = a + b + k,
// so g[0] = a/(a+b) and g[k+1] = g[k] (b+k)/(a+b+k+1), which is the paper's recurrence.
// One warp owns one row at a time.  A lane takes E consecutive factors, multiplies numerators forwards and
// denominators backwards, and needs ONE reciprocal for its E entries (1/(d_0..d_m) = (d_{m+1}..d_{E-1}) / (d_0..d_{E-1})).
// The lanes' E-factor products are combined by a multiplicative warp scan; rows longer than 32*E
// carry the running product from chunk to chunk.  The value of an entry depends on (a, b, k, E) only,
// never on the row index, so equal posteriors give bitwise equal rows.
#include "hora_common.cuh"
#include "hora_gains_chunk.cuh"

namespace hora {

// The kernel is the shared row loop with no tap attached.
// LG: lanes per row.  Rows of at most 128 entries are built two (LG = 16), four (LG = 8) or eight (LG = 4) to a
// warp, so that a warp still produces 256 entries per scan and per reciprocal: a whole warp on a 64-entry row
// spent as many instructions per row as on a 256-entry one, and those, not the memory system, set the time
// (2.9 TB/s at 64 entries, 4.3 TB/s at 128).  A lane always holds 8 consecutive entries.
template <int E, bool VEC2, int LG>
__global__ void __launch_bounds__(kGainsWarps *kWarp, 3)
gains_kernel(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
             const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
             int64_t N, int32_t ld, double *__restrict__ gains, int32_t *status_dev) {
    pdl_enter();
    NoTap tap;
    gains_rows_cta<E, VEC2, NoTap, LG>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, tap);
}

template <int E, int LG>
static hora_status_t launch_e(const double *alpha, const double *beta, double alpha0, double beta0, const int32_t *c,
                              int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N, int32_t ld, double *gains,
                              int32_t *status_dev, cudaStream_t stream) {
    const int grid = clamp_grid((N + kCtaRows - 1) / kCtaRows, 3);
    const bool vec2 = (ld % 2 == 0) && ((reinterpret_cast<uintptr_t>(gains) & 15u) == 0);
    if (vec2)
        launch_pdl(gains_kernel<E, true, LG>, grid, kGainsWarps * kWarp, 0, stream, alpha, beta, alpha0, beta0, c, G0, cap,
                   cap_scalar, N, ld, gains, status_dev);
    else
        launch_pdl(gains_kernel<E, false, LG>, grid, kGainsWarps * kWarp, 0, stream, alpha, beta, alpha0, beta0, c, G0, cap,
                   cap_scalar, N, ld, gains, status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}

hora_status_t launch_gains(const double *alpha, const double *beta, double alpha0, double beta0, const int32_t *c,
                           int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N, int32_t ld, double *gains,
                           int32_t *status_dev, cudaStream_t stream) {
    if (ld > 128)
        return launch_e<8, kWarp>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
    if (ld > 64)
        return launch_e<8, 16>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
    if (ld > 32)
        return launch_e<8, 8>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
    return launch_e<8, 4>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
}

}  // namespace hora

extern "C" hora_status_t hora_gains(const double *alpha, const double *beta, double alpha0, double beta0,
                                    const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N,
                                    int32_t ld, double *gains, int32_t *status_dev, void *stream) {
    if (N < 0 || ld < 1 || G0 < 0) return HORA_ERR_INVALID_ARG;
    if ((alpha == nullptr) != (beta == nullptr)) return HORA_ERR_INVALID_ARG;
    if (alpha == nullptr && !(alpha0 > 0.0 && beta0 > 0.0 && alpha0 < 1.0e300 && beta0 < 1.0e300))
        return HORA_ERR_INVALID_ARG;
    if (cap == nullptr && (cap_scalar < 0 || cap_scalar > ld)) return HORA_ERR_INVALID_ARG;
    if (N == 0) return HORA_OK;
    if (c == nullptr || gains == nullptr) return HORA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(gains) & 7u) return HORA_ERR_INVALID_ARG;
    return hora::launch_gains(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev,
                              static_cast<cudaStream_t>(stream));
}
