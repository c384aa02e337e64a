// The arithmetic of one chunk of a gain row (Eq. marginal and its recurrence as a prefix product), shared by
// hora_gains and by kernels that build rows on the fly, so that equal posteriors give bitwise equal gains
// wherever they are computed.
#pragma once

#include "hora_common.cuh"

namespace hora {

// A "tap" sees every pair of entries a lane produces, while they are still in registers, and is told
// when the lane's part of the chunk is complete.  NoTap does nothing and costs nothing.
struct NoTap {
    __device__ __forceinline__ void pair(int, double, double) {}
    __device__ __forceinline__ void finish(int32_t, int32_t, int32_t, int32_t) {}
};

// One chunk of 32*E entries of one row, starting at column k0.  FULL: the chunk lies entirely below the
// row's cap and inside the row, so no entry needs masking.  `out` may be null when only the tap wants the
// values (then nothing is stored).
template <int E, bool VEC2, bool FULL, typename Tap = NoTap>
__device__ __forceinline__ void gains_chunk(double a, double b, double ab, int32_t capi, int32_t ld, int32_t k0,
                                            int lane, double &carry, double *__restrict__ out, double2 *wr,
                                            const double2 *rd, Tap &&tap = Tap()) {
    constexpr int P = E / 2;                              // 16-byte chunks per lane
    constexpr bool kStaged = VEC2 && (P > 1);
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
    double inc = pt * r;                                  // this lane's E-factor product
#pragma unroll
    for (int d = 1; d < kWarp; d <<= 1) {
        const double t = shfl_up_f64(inc, d);
        if (lane >= d) inc *= t;
    }
    double excl = shfl_up_f64(inc, 1);
    if (lane == 0) excl = 1.0;
    const double total = shfl_idx_f64(inc, kWarp - 1);
    double pm = (carry * excl * r) * n0;                  // running numerator product times everything shared
    carry *= total;
#pragma unroll
    for (int m = 0; m < E; m += 2) {                      // E is even: entries are produced and stored in pairs
        double g0 = pm * S[m + 1];
        pm *= x + (double)(m + 1);
        double g1 = pm * S[m + 2];
        if (m + 2 < E) pm *= x + (double)(m + 2);
        if (!FULL) {
            if (k + m >= capi) g0 = 0.0;
            if (k + m + 1 >= capi) g1 = 0.0;
        }
        tap.pair(m, g0, g1);
        if (kStaged) {
            wr[(m >> 1) ^ ((lane >> (P == 4 ? 1 : 2)) & (P - 1))] = make_double2(g0, g1);   // (lane*P + p) >> 3
        } else if (VEC2) {
            if (FULL || k + m < ld) *reinterpret_cast<double2 *>(out + k + m) = make_double2(g0, g1);
        } else if (out != nullptr) {
            if (FULL || k + m < ld) out[k + m] = g0;
            if (FULL || k + m + 1 < ld) out[k + m + 1] = g1;
        }
    }
    tap.finish(k0, k, capi, ld);
    if (kStaged) {
        __syncwarp();
#pragma unroll
        for (int q = 0; q < P; ++q) {
            const double2 v = rd[q * kWarp];
            const int32_t col = k0 + 2 * (q * kWarp + lane);
            if (FULL || col < ld) *reinterpret_cast<double2 *>(out + col) = v;
        }
        __syncwarp();
    }
}

}  // namespace hora
