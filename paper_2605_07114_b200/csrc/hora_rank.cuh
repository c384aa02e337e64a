// Rank-based exact allocation for a SHARED integer prior (Proposition 1; Eq. marginal).
//
// With one Beta(alpha0, beta0) prior for every prompt there are only G0 + 1 posteriors, hence at most
// T = (G0 + 1) * ld distinct candidate values g_c(Delta).  They are ranked once, exactly; the selection then
// runs on integer ranks and on counts of (c_i, cap_i) pairs, never on a gains matrix: 8 bytes read per prompt.
#pragma once

#include "hora_common.cuh"

namespace hora {

constexpr int kRankMaxTypes = 8192;              // T = (G0 + 1) * ld the route accepts
constexpr int64_t kRankMaxPos = 1 << 20;         // entries of the per-class position table (batched form only)

// Tables of one (alpha0, beta0, G0, ld), in device memory.  The rank of a type is the number of types with a
// strictly larger gain; exactly equal gains share a rank.
struct RankTables {
    int32_t *rank;        // [C][ld]     rank of g_c(Delta), Delta = column + 1
    double *gain;         // [C][ld]     the fp64 value (same bits as hora_gains writes)
    double *util;         // [C][ld+1]   U_c(d), d = 0..ld
    double *lam;          // [T]         fp64 gain by rank (of the member with the smallest c)
    uint16_t *pos;        // [C][T+1]    pos[c][r] = #{Delta : rank_c(Delta) < r}; null when not built
};

// Host: does the route apply to this prior and shape?  (T within bounds; exact ties: integer prior whose exact forms
// fit 512 bits; fp64 ties: any prior)
bool rank_route_applies(double alpha0, double beta0, int32_t G0, int32_t ld, bool exact);
bool rank_pos_applies(int32_t G0, int32_t ld);

// Bytes of the tables (256-byte granularity) and their carving out of `base`.
size_t rank_tables_bytes(int32_t G0, int32_t ld, bool with_pos);
RankTables rank_tables_carve(void *base, int32_t G0, int32_t ld, bool with_pos);

// Enqueue the kernels that fill the tables; `status` (device) receives HORA_ERR_EXACT_RANGE should an exact
// comparison not fit (the host check makes that unreachable).  Returns the number of launches, or -1 on failure.
int launch_rank_tables(double alpha0, double beta0, int32_t G0, int32_t ld, bool exact, const RankTables &t,
                       int32_t *status, cudaStream_t s);

// The single-problem route of hora_allocate.
size_t rank_allocate_workspace_bytes(int64_t N, int32_t G0, int32_t ld);
size_t rank_allocate_workspace_bound(int64_t N);   // over every (G0, ld) the route accepts
hora_status_t launch_rank_allocate(double alpha0, double beta0, const int32_t *c, int32_t G0, const int32_t *cap,
                                   int32_t cap_scalar, int64_t N, int32_t ld, int64_t B, uint32_t flags, int32_t *delta,
                                   int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev, void *workspace,
                                   size_t workspace_bytes, cudaStream_t s, void (*mark)(int, cudaStream_t));

// The per-segment kernel of hora_allocate_batched for the same case (tables already enqueued on `s`).
hora_status_t launch_rank_batched(const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar, int32_t ld,
                                  const int64_t *seg_off_dev, const int64_t *budgets_dev, int64_t S, uint32_t flags,
                                  const RankTables &t, const int32_t *table_status, int32_t *delta, int32_t *G,
                                  hora_alloc_info *info_dev, cudaStream_t s);

}  // namespace hora
