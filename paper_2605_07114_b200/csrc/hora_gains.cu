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

namespace hora {

constexpr int kGainsWarps = 8;
constexpr int kTile = 8;                      // consecutive rows a warp takes at a time

// A warp takes kTile consecutive rows at a time.  Lane i (< kTile) loads row i's prior, count and cap
// (one coalesced load per array) ONE TILE AHEAD, so that latency is hidden behind the arithmetic of the
// current tile; the values reach the other lanes by shuffles.
template <int E, bool VEC2>
__global__ void __launch_bounds__(kGainsWarps *kWarp, 3)
gains_kernel(const double *__restrict__ alpha, const double *__restrict__ beta, double alpha0, double beta0,
             const int32_t *__restrict__ c, int32_t G0, const int32_t *__restrict__ cap, int32_t cap_scalar,
             int64_t N, int32_t ld, double *__restrict__ gains, int32_t *status_dev) {
    // Staging slab: a lane produces E consecutive entries, but a store instruction should cover one
    // contiguous 512-byte run of the row (full 32-byte sectors; 16-byte pieces at a 64-byte stride cost
    // twice the L1-to-L2 traffic).  Pairs go through shared memory with an XOR swizzle on the 16-byte
    // chunk index that keeps both the lane-major writes and the row-major reads free of bank conflicts.
    constexpr int P = E / 2;                              // 16-byte chunks per lane
    constexpr bool kStaged = VEC2 && (P > 1);
    __shared__ double2 s_stage[kStaged ? kGainsWarps * kWarp * P : 1];
    double2 *slab = s_stage + (kStaged ? (threadIdx.x >> 5) * kWarp * P : 0);
    const int lane = lane_id();
    const int64_t n_tiles = (N + kTile - 1) / kTile;
    const int64_t tile0 = (int64_t)blockIdx.x * kGainsWarps + (threadIdx.x >> 5);
    const int64_t stride = (int64_t)gridDim.x * kGainsWarps;
    auto fetch = [&](int64_t tile) {
        Posterior p;
        p.a = p.b = 1.0;
        p.cap = 0;
        p.ok = true;
        const int64_t row = tile * kTile + lane;
        if (tile < n_tiles && lane < kTile && row < N)
            p = load_posterior(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, ld, row);
        return p;
    };
    Posterior nxt = fetch(tile0);
    for (int64_t tile = tile0; tile < n_tiles; tile += stride) {
        const Posterior cur = nxt;
        nxt = fetch(tile + stride);
        if (!cur.ok) raise_status(status_dev, HORA_ERR_INVALID_VALUE);
        const int rows = (int)((N - tile * kTile < kTile) ? N - tile * kTile : kTile);
        for (int i = 0; i < rows; ++i) {
            const bool ok = __shfl_sync(kFull, (int)cur.ok, i) != 0;
            const double a = ok ? shfl_idx_f64(cur.a, i) : 1.0, b = ok ? shfl_idx_f64(cur.b, i) : 1.0;
            const int32_t capi = __shfl_sync(kFull, cur.cap, i);
            const double ab = a + b;
            double *out = gains + (tile * kTile + i) * (int64_t)ld;
            double carry = 1.0;
            for (int32_t k0 = 0; k0 < ld; k0 += kWarp * E) {
                const int32_t k = k0 + lane * E;
                // factors of entries k .. k+E-1: num = a (k = 0) or b + k - 1, then +1 each; den = a + b + k, then +1 each
                const double x = b + (double)(k - 1), y = ab + (double)k;
                const double n0 = (k == 0) ? a : x;
                double S[E + 1];
                S[E] = 1.0;
#pragma unroll
                for (int m = E - 1; m >= 0; --m) S[m] = S[m + 1] * (y + (double)m);
                double pt = n0;
#pragma unroll
                for (int m = 1; m < E; ++m) pt *= x + (double)m;
                const double r = 1.0 / S[0];
                double inc = pt * r;                     // this lane's E-factor product
#pragma unroll
                for (int d = 1; d < kWarp; d <<= 1) {
                    const double t = shfl_up_f64(inc, d);
                    if (lane >= d) inc *= t;
                }
                double excl = shfl_up_f64(inc, 1);
                if (lane == 0) excl = 1.0;
                const double total = shfl_idx_f64(inc, kWarp - 1);
                double pm = (carry * excl * r) * n0;     // running numerator product times everything shared
                carry *= total;
#pragma unroll
                for (int m = 0; m < E; m += 2) {         // E is even: entries are produced and stored in pairs
                    const double g0 = (k + m < capi) ? pm * S[m + 1] : 0.0;
                    pm *= x + (double)(m + 1);
                    const double g1 = (k + m + 1 < capi) ? pm * S[m + 2] : 0.0;
                    if (m + 2 < E) pm *= x + (double)(m + 2);
                    if (kStaged) {
                        const int ch = lane * P + (m >> 1);
                        slab[ch ^ ((ch >> 3) & (P - 1))] = make_double2(g0, g1);
                    } else if (VEC2) {
                        if (k + m < ld) *reinterpret_cast<double2 *>(out + k + m) = make_double2(g0, g1);
                    } else {
                        if (k + m < ld) out[k + m] = g0;
                        if (k + m + 1 < ld) out[k + m + 1] = g1;
                    }
                }
                if (kStaged) {
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < P; ++q) {
                        const int ch = q * kWarp + lane;
                        const double2 v = slab[ch ^ ((ch >> 3) & (P - 1))];
                        const int32_t col = k0 + 2 * ch;
                        if (col < ld) *reinterpret_cast<double2 *>(out + col) = v;
                    }
                    __syncwarp();
                }
            }
        }
    }
}

template <int E>
static hora_status_t launch_e(const double *alpha, const double *beta, double alpha0, double beta0, const int32_t *c,
                              int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N, int32_t ld, double *gains,
                              int32_t *status_dev, cudaStream_t stream) {
    const int64_t tiles = (N + kTile - 1) / kTile;
    const int grid = clamp_grid((tiles + kGainsWarps - 1) / kGainsWarps, 3);
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
