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
    __device__ __forceinline__ void begin_row(int64_t, int32_t) {}
};

// One chunk of 32*E entries of one row, starting at column k0.  FULL: the chunk lies entirely below the
// row's cap and inside the row, so no entry needs masking.  `out` may be null when only the tap wants the
// values (then nothing is stored).
//
// LG < 32: packed rows.  The warp holds 32 / LG rows at once, LG lanes each (a, b, capi and `out` then differ
// from group to group, `lane` is the lane's position inside its group, and the scan runs over the group only).
// A lane's entries depend on the lanes before it in its row and on nothing else, so a row computed by a group
// of LG lanes has the same bits as the same row computed by a whole warp whose other lanes lie past its end.
// `tile_ld`: the staged store path treats the warp's 32 * E entries as one run of memory starting at `out` (rows
// of exactly LG * E entries, packed) and writes the first tile_ld of them; for a single row it is ld.
// STAGE: results leave through the swizzled shared-memory slab (the default wherever 16-byte stores are possible and
// a lane has more than one of them); packed rows that are shorter than LG * E entries, hence not back to back in
// memory, store directly instead.
template <int E, bool VEC2, bool FULL, typename Tap = NoTap, int LG = kWarp, bool STAGE = VEC2 && (E > 2)>
__device__ __forceinline__ void gains_chunk(double a, double b, double ab, int32_t capi, int32_t ld, int32_t k0,
                                            int lane, double &carry, double *__restrict__ out, double2 *wr,
                                            const double2 *rd, Tap &&tap = Tap(), int32_t tile_ld = -1) {
    constexpr int P = E / 2;                              // 16-byte chunks per lane
    constexpr bool kStaged = STAGE;
    static_assert(!STAGE || (VEC2 && P > 1), "staging needs 16-byte stores and more than one of them per lane");
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
    for (int d = 1; d < LG; d <<= 1) {
        const double t = __shfl_up_sync(kFull, inc, d, LG);
        if (lane >= d) inc *= t;
    }
    double excl = __shfl_up_sync(kFull, inc, 1, LG);
    if (lane == 0) excl = 1.0;
    const double total = __shfl_sync(kFull, inc, LG - 1, LG);
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
            const int wl = LG == kWarp ? lane : (int)(threadIdx.x & (kWarp - 1));   // position in the warp's tile
            wr[(m >> 1) ^ ((wl >> (P == 4 ? 1 : 2)) & (P - 1))] = make_double2(g0, g1);   // (wl*P + p) >> 3
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
        const int wl = LG == kWarp ? lane : (int)(threadIdx.x & (kWarp - 1));
        const int32_t bound = LG == kWarp ? ld : tile_ld;
#pragma unroll
        for (int q = 0; q < P; ++q) {
            const double2 v = rd[q * kWarp];
            const int32_t col = k0 + 2 * (q * kWarp + wl);
            if ((FULL && LG == kWarp) || col < bound) *reinterpret_cast<double2 *>(out + col) = v;
        }
        __syncwarp();
    }
}

constexpr int kGainsWarps = 8;
constexpr int kTile = 8;                      // consecutive rows a warp takes at a time
constexpr int kCtaRows = kGainsWarps * kTile; // rows a CTA stages per step

// A CTA stages the posterior parameters of 64 consecutive rows in shared memory (one coalesced load per
// array, issued one step ahead and parked in registers meanwhile); each warp then takes 8 of those rows.
// LG < 32 (rows of at most LG * E entries): a warp builds 32 / LG rows at a time, LG lanes a row; a tap is told
// begin_row(-1, 0) for the rows of the last tile that do not exist.
template <int E, bool VEC2, typename Tap, int LG = kWarp>
__device__ __forceinline__ void gains_rows_cta(const double *__restrict__ alpha, const double *__restrict__ beta,
                                               double alpha0, double beta0, const int32_t *__restrict__ c, int32_t G0,
                                               const int32_t *__restrict__ cap, int32_t cap_scalar, int64_t N,
                                               int32_t ld, double *__restrict__ gains, int32_t *status_dev, Tap &tap) {
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
        if constexpr (LG < kWarp) {
            // packed rows: group g of the warp builds row row0 + i + g
            constexpr int R = kWarp / LG;
            const int grp = lane / LG, gl = lane % LG;
            const bool back_to_back = VEC2 && E > 2 && ld == LG * E;   // the rows of a tile are one run of memory
            for (int i = 0; i < kTile && row0 + i < N; i += R) {
                const int64_t row = row0 + i + grp;
                const bool live = row < N;
                const int idx = warp * kTile + i + grp;
                const double a = s_a[buf][idx], b = s_b[buf][idx];
                const int32_t capi = live ? s_cap[buf][idx] : 0;
                double carry = 1.0;
                tap.begin_row(live ? row : -1, capi);
                if (back_to_back) {
                    const int64_t rows_here = N - (row0 + i) < R ? N - (row0 + i) : R;
                    gains_chunk<E, VEC2, false, Tap &, LG, VEC2 && (E > 2)>(a, b, a + b, capi, ld, 0, gl, carry,
                                                                          gains + (row0 + i) * (int64_t)ld, wr, rd, tap,
                                                                          (int32_t)(rows_here * ld));
                } else {
                    gains_chunk<E, VEC2, false, Tap &, LG, false>(a, b, a + b, capi, live ? ld : 0, 0, gl, carry,
                                                                 gains + (live ? row : 0) * (int64_t)ld, nullptr, nullptr, tap);
                }
            }
        } else {
            for (int i = 0; i < kTile && row0 + i < N; ++i) {
                const double a = s_a[buf][warp * kTile + i], b = s_b[buf][warp * kTile + i];
                const int32_t capi = s_cap[buf][warp * kTile + i];
                const double ab = a + b;
                double *out = gains + (row0 + i) * (int64_t)ld;
                tap.begin_row(row0 + i, capi);
                double carry = 1.0;
                for (int32_t k0 = 0; k0 < ld; k0 += kWarp * E) {
                    if (k0 + kWarp * E <= capi)           // capi <= ld: the chunk is inside the row as well
                        gains_chunk<E, VEC2, true>(a, b, ab, capi, ld, k0, lane, carry, out, wr, rd, tap);
                    else
                        gains_chunk<E, VEC2, false>(a, b, ab, capi, ld, k0, lane, carry, out, wr, rd, tap);
                }
            }
        }
    }
}

}  // namespace hora
