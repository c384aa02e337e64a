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

constexpr int kGainsWarps = 8;
constexpr int kTile = 8;                      // consecutive rows a warp takes at a time
constexpr int kCtaRows = kGainsWarps * kTile; // rows a CTA stages per step

// A CTA stages the posterior parameters of 64 consecutive rows in shared memory (one coalesced load per
// array, issued one step ahead and parked in registers meanwhile); each warp then takes 8 of those rows.
template <int E, bool VEC2>
__global__ void __launch_bounds__(kGainsWarps *kWarp, 3)
gains_kernel(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
             const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
             int64_t N, int32_t ld, double *__restrict__ gains, int32_t *status_dev) {
    // Staging slab: a lane produces E consecutive entries, but a store instruction should cover one
    // contiguous 512-byte run of the row (full 32-byte sectors; 16-byte pieces at a 64-byte stride cost
    // twice the L1-to-L2 traffic).  Pairs go through shared memory with an XOR swizzle on the 16-byte
    // chunk index (chunk ch of the row sits at ch ^ ((ch >> 3) & (P-1))) that keeps both the lane-major
    // writes and the row-major reads free of bank conflicts.
    constexpr int P = E / 2;
    constexpr bool kStaged = VEC2 && (P > 1);
    __shared__ double2 s_stage[kStaged ? kGainsWarps * kWarp * P : 1];
    __shared__ double s_a[2][kCtaRows], s_b[2][kCtaRows];
    __shared__ int32_t s_cap[2][kCtaRows];
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    double2 *slab = s_stage + (kStaged ? warp * kWarp * P : 0);
    // lane-major write: chunks lane*P + p, p = 0..P-1, swizzled within the lane's group of P chunks;
    // row-major read: chunks q*32 + lane, swizzled by bits 3.. of the chunk index = bits 3.. of the lane
    double2 *wr = slab + lane * P;
    const double2 *rd = slab + (lane ^ ((lane >> 3) & (P - 1)));
    const int64_t n_steps = (N + kCtaRows - 1) / kCtaRows;
    auto fetch = [&](int64_t step) {
        Posterior p;
        p.a = p.b = 1.0;
        p.cap = 0;
        p.ok = true;
        const int64_t row = step * kCtaRows + threadIdx.x;
        if (step < n_steps && threadIdx.x < kCtaRows && row < N)
            p = load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, row);
        return p;
    };
    Posterior nxt = fetch(blockIdx.x);
    int buf = 0;
    for (int64_t step = blockIdx.x; step < n_steps; step += gridDim.x, buf ^= 1) {
        if (threadIdx.x < kCtaRows) {
            if (!nxt.ok) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
            s_a[buf][threadIdx.x] = nxt.ok ? nxt.a : 1.0;
            s_b[buf][threadIdx.x] = nxt.ok ? nxt.b : 1.0;
            s_cap[buf][threadIdx.x] = nxt.cap;
        }
        __syncthreads();                                  // buf was last read two steps ago: safe to have overwritten it
        nxt = fetch(step + gridDim.x);
        const int64_t row0 = step * kCtaRows + warp * kTile;
        for (int i = 0; i < kTile && row0 + i < N; ++i) {
            const double a = s_a[buf][warp * kTile + i], b = s_b[buf][warp * kTile + i];
            const int32_t capi = s_cap[buf][warp * kTile + i];
            const double ab = a + b;
            double *out = gains + (row0 + i) * (int64_t)ld;
            double carry = 1.0;
            for (int32_t k0 = 0; k0 < ld; k0 += kWarp * E) {
                if (k0 + kWarp * E <= capi)               // capi <= ld: the chunk is inside the row as well
                    gains_chunk<E, VEC2, true>(a, b, ab, capi, ld, k0, lane, carry, out, wr, rd);
                else
                    gains_chunk<E, VEC2, false>(a, b, ab, capi, ld, k0, lane, carry, out, wr, rd);
            }
        }
    }
}

template <int E>
static hora_status_t launch_e(const double *alpha, const double *beta, double alpha0, double beta0, const int32_t *c,
                              int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N, int32_t ld, double *gains,
                              int32_t *status_dev, cudaStream_t stream) {
    const int grid = clamp_grid((N + kCtaRows - 1) / kCtaRows, 3);
    const bool vec2 = (ld % 2 == 0) && ((reinterpret_cast<uintptr_t>(gains) & 15u) == 0);
    if (vec2)
        gains_kernel<E, true><<<grid, kGainsWarps * kWarp, 0, stream>>>(alpha, beta, alpha0, beta0, c, G0, cap,
                                                                        cap_scalar, N, ld, gains, status_dev);
    else
        gains_kernel<E, false><<<grid, kGainsWarps * kWarp, 0, stream>>>(alpha, beta, alpha0, beta0, c, G0, cap,
                                                                         cap_scalar, N, ld, gains, status_dev);
    count_launches(1);
    return cuda_ok(cudaGetLastError());
}

hora_status_t launch_gains(const double *alpha, const double *beta, double alpha0, double beta0, const int32_t *c,
                           int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N, int32_t ld, double *gains,
                           int32_t *status_dev, cudaStream_t stream) {
    if (ld > 128)
        return launch_e<8>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
    if (ld > 64)
        return launch_e<4>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
    return launch_e<2>(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev, stream);
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
