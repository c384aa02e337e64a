/*
 * hora.h — C ABI of the HORA rollout-allocation hot path for NVIDIA B200 (sm_100a).
 *
 * HORA ("Hit-Utility Optimal Rollout Allocation for Group-Based RLVR") splits the rollouts of a
 * training batch in two phases.  Phase A draws G0 rollouts for each of N prompts and counts the
 * correct ones, c_i.  With a Beta(alpha_i, beta_i) prior the posterior of the prompt's success
 * rate is Beta(a_i, b_i), a_i = alpha_i + c_i, b_i = beta_i + G0 - c_i (Eq. posterior).  Phase B
 * hands out B further rollouts so as to maximise sum_i U_i(Delta_i), where U_i(Delta) is the posterior
 * probability that at least one of Delta more rollouts is correct (Eq. hit-utility, Eq.
 * allocation-problem).  The marginal gains g_i(Delta) = U_i(Delta) - U_i(Delta-1) decrease in Delta, so the
 * optimum is the set of the B largest gains over all (prompt, Delta) candidates (Proposition 1).
 * Advantages are then computed over the variable-size groups G_i = G0 + Delta_i and replicated over
 * the tokens of each rollout.
 *
 * This library covers exactly that path, four calls, in execution order:
 *   hora_gains -> hora_allocate -> [rollouts and rewards happen elsewhere] ->
 *   hora_group_advantage -> hora_token_broadcast
 *
 * Conventions for every call
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer on the current CUDA device.
 *   - The caller owns every buffer.  The library allocates nothing; hora_allocate works in a
 *     caller-provided workspace whose size hora_allocate_workspace_bytes returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls enqueue
 *     work and return; they never synchronise the device.
 *   - The return value reports what the host can see at enqueue time (bad sizes, null pointers,
 *     a too-small workspace, a failed launch).  Errors that depend on device DATA (a non-finite
 *     prior, B larger than the total cap, ...) are written to a status word in device memory; the
 *     caller reads it after synchronising.  Nothing traps, spins or aborts.
 *   - Results are deterministic: the same inputs give bitwise identical outputs on every run.
 *   - Calls on different streams may run concurrently as long as they do not share output
 *     buffers or workspaces.
 *   - The kernels of hora_gains, hora_allocate, hora_group_advantage, hora_token_broadcast and
 *     hora_group_advantage_tokens are launched with the programmatic-dependent-launch attribute and wait
 *     (griddepcontrol.wait) for the work before them in the stream before they touch memory, so stream order
 *     holds as usual; a kernel of the caller's that follows them with the same attribute must do its own wait.
 */
#ifndef HORA_H
#define HORA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum hora_status {
    HORA_OK = 0,
    HORA_ERR_INVALID_ARG = 1,    /* host-visible: null pointer, negative size, ld < 1, unknown mode ... */
    HORA_ERR_INVALID_VALUE = 2,  /* device data: prior not finite or <= 0, c outside [0,G0], cap outside [0,ld],
                                    a gain row that is not finite/non-negative/non-increasing, offsets that decrease */
    HORA_ERR_INFEASIBLE = 3,     /* B > sum_i cap_i */
    HORA_ERR_NOT_INTEGER = 4,    /* HORA_FLAG_EXACT_INT given but some alpha_i or beta_i is not a positive integer */
    HORA_ERR_EXACT_RANGE = 5,    /* exact path: a near-threshold gain does not fit the 512-bit exact form (see
                                    hora_allocate), alpha+beta+G0+ld >= 2^20, or more than 1024 distinct tie types */
    HORA_ERR_WORKSPACE = 6,      /* workspace missing, misaligned (needs 256 B) or too small */
    HORA_ERR_CUDA = 7,           /* a CUDA runtime call or kernel launch failed */
    HORA_ERR_INTERNAL = 8        /* device data: a consistency check inside the selection failed (a fault of the
                                    library, never of the inputs); reported like the other data-dependent errors */
} hora_status_t;

enum {
    HORA_FLAG_EXACT_INT = 1u,      /* priors are integer-valued: decide ties by exact rational equality */
    HORA_FLAG_SKIP_OBJECTIVE = 2u, /* do not compute hora_alloc_info.objective (left 0) */
    HORA_FLAG_SHARED_PRIOR = 4u,   /* sizing hint for hora_allocate_workspace_bytes: the call will pass alpha == beta ==
                                      NULL and gains == NULL (see the rank-based route under hora_allocate); ignored
                                      by the calls themselves */
    HORA_FLAG_SHARED_INT_PRIOR = 4u, /* the same flag under the name of its first use (an integer prior, exact ties) */
    HORA_FLAG_HARD_FIRST = 8u      /* hora_allocate_batched only: every segment by the hard-first rule of
                                      hora_allocate_hard_first instead of the hit-utility optimum (priors unused) */
};

enum { HORA_ADV_GRPO = 0, HORA_ADV_RLOO = 1 };

enum { HORA_WEIGHT_PER_TOKEN = 0, HORA_WEIGHT_CONST_LENGTH = 1 };

/* Summary of one allocation; lives in DEVICE memory (64 bytes, 8-byte aligned). */
typedef struct hora_alloc_info {
    int32_t status;        /* hora_status_t of the data-dependent checks */
    int32_t first_pass_bits; /* diagnostic: key bits the full-read pass resolved (23 when its sampled window held the
                                threshold, else 13); 0 when B == 0; -1 when the rank-based route ran (no key pass) */
    double  lambda;        /* gain of the B-th best candidate (the selection threshold); 0 when B == 0 */
    int64_t n_above;       /* candidates strictly better than lambda (all taken) */
    int64_t n_tied;        /* candidates equal to lambda */
    int64_t n_tied_taken;  /* B - n_above: how many of the tied ones were taken, lowest prompt index first */
    double  objective;     /* sum_i U_i(Delta_i) */
    int64_t sum_G;         /* sum_i G_i = N*G0 + B */
    int64_t sum_cap;       /* sum_i cap_i */
} hora_alloc_info;

/*
 * hora_gains — marginal hit-utility rows (Eq. marginal and the recurrence stated after it).
 *
 *   gains[i*ld + (Delta-1)] = g_i(Delta) = M_i(Delta-1)
 *                            = a_i/(a_i+b_i+Delta-1) * prod_{j<Delta-1} (b_i+j)/(a_i+b_i+j)     for 1 <= Delta <= cap_i
 *                            = 0.0                                                              for cap_i < Delta <= ld
 *
 * computed in fp64 as a prefix product (one warp per row, warp scan); every entry is within
 * 4*ld ulp of the exact value.  Rows are strictly decreasing up to cap_i.
 *
 *   alpha, beta   [N] fp64 per-prompt prior, or both NULL to use the shared prior (alpha0, beta0)
 *   c             [N] int32 Phase-A success counts, 0 <= c_i <= G0
 *   cap           [N] int32 per-prompt cap, 0 <= cap_i <= ld, or NULL to use cap_scalar for all
 *   gains         [N*ld] fp64 out, row-major, 8-byte aligned (16-byte aligned enables vector stores)
 *   status_dev    optional int32 in device memory: receives HORA_ERR_INVALID_VALUE if any row's inputs
 *                 are invalid (that row is written as zeros); it is never cleared by this call
 * Returns HORA_ERR_INVALID_ARG for N < 0, ld < 1, G0 < 0, missing pointers.  N == 0 is a no-op.
 */
hora_status_t hora_gains(const double *alpha, const double *beta, double alpha0, double beta0,
                         const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                         int64_t N, int32_t ld, double *gains, int32_t *status_dev, void *stream);

/*
 * hora_allocate — budgeted optimal allocation (Eq. allocation-problem; Algorithm 1 Phase B; Proposition 1).
 *
 * Computes the result of B greedy steps "give one more rollout to the prompt with the largest
 * current marginal gain" without running them one by one: because every row of gains decreases,
 * that result is the set of the B largest candidates g_i(Delta), Delta <= cap_i.  The call finds the
 * B-th largest value lambda by a multi-level radix selection on the 64-bit patterns of the gains
 * (one full read of the matrix, then a short look at each row around a guessed position), counts per row the candidates
 * above lambda, and gives the remaining B - n_above rollouts to the tied candidates in order of
 * increasing prompt index (then increasing Delta).  Outputs:
 *
 *   delta[i]          = Delta_i, 0 <= Delta_i <= cap_i, sum = B                    int32 [N]
 *   G[i]              = G0 + Delta_i                                              int32 [N]
 *   group_offsets[i]  = sum_{j<i} G[j] (CSR offsets of the pooled groups)         int64 [N+1], may be NULL
 *   info_dev          = summary (see hora_alloc_info)                             device, may be NULL
 *
 * Ties.  Without HORA_FLAG_EXACT_INT a tie is equality of the fp64 gains as hora_gains computes
 * them.  With HORA_FLAG_EXACT_INT (every alpha_i, beta_i a positive integer) candidates within a
 * relative band of 2^-30 around the fp64 threshold are re-ranked on exact integers
 * (g = a*(b)_a / (b+Delta-1)_{a+1}, or the equal a*(b)_{Delta-1} / (a+b)_Delta when that has fewer factors,
 * numerator and denominator in 512 bits, compared by cross multiplication), so a tie is an exact rational
 * equality and the result equals exact greedy with lowest-index tie-breaking.  Guaranteed range of the exact
 * form: with m = min(a_i + 1, Delta) factors, each below a_i + b_i + Delta, m * log2(a_i + b_i + Delta) <= 512 —
 * e.g. any posterior with a_i <= 50 up to Delta = 1000 (this covers G0 = 16 and learned priors with
 * alpha_i + beta_i <= 16), or any a_i at all up to Delta = 25.  Only candidates near the threshold are ever
 * formed exactly; one that does not fit raises HORA_ERR_EXACT_RANGE (nothing wraps).
 *
 * Rank-based route.  With ONE prior for all prompts (alpha == beta == NULL) and gains == NULL there are only G0 + 1
 * posteriors and at most (G0 + 1) * ld distinct candidate values.  When (G0 + 1) * ld <= 8192 (and alpha0 + beta0 +
 * G0 + ld < 2^20) the call ranks those values once, counts the prompts per (c_i, cap_i) in one pass and selects on
 * integer ranks: no matrix is built, 8 bytes are read per prompt per pass (three passes).  With HORA_FLAG_EXACT_INT
 * (alpha0, beta0 positive integers whose exact forms fit 512 bits) the ranking is exact and the result is exact
 * greedy by construction; without the flag the values are ranked as the doubles hora_gains would write, equal
 * doubles tie, and the result is what the key-based selection gives on that matrix.  The workspace this route
 * needs is small and independent of ld: pass HORA_FLAG_SHARED_PRIOR to hora_allocate_workspace_bytes to size for
 * it (a workspace sized without that flag is always large enough).  info_dev->lambda is then the fp64 gain of the
 * threshold type.
 *
 *   alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld   as for hora_gains
 *   gains            [N*ld] the matrix hora_gains wrote for the same inputs, or NULL to have it built
 *                    inside the workspace (the workspace must then be sized with gains_is_null = 1)
 *   N                at most 2^31 - 1 prompts per call (HORA_ERR_INVALID_ARG beyond)
 *   B                number of Phase-B rollouts, 0 <= B <= sum_i cap_i
 *   workspace        device scratch, 256-byte aligned, at least hora_allocate_workspace_bytes(...);
 *                    contents are undefined on entry and on exit
 * Data-dependent failures (INVALID_VALUE, INFEASIBLE, NOT_INTEGER, EXACT_RANGE, INTERNAL) set info_dev->status and
 * leave delta, G and group_offsets all zero.
 * One of the call's kernels is launched cooperatively (all its thread blocks resident at once, sized per device
 * on first use); a device or context without cooperative launch makes the call return HORA_ERR_CUDA before
 * anything is enqueued.  Should that launch fail after the earlier passes were enqueued, the call still returns
 * HORA_ERR_CUDA, with zeroed delta / G / group_offsets and the code in info_dev->status.
 */
size_t hora_allocate_workspace_bytes(int64_t N, int32_t ld, int32_t gains_is_null, uint32_t flags);

hora_status_t hora_allocate(const double *alpha, const double *beta, double alpha0, double beta0,
                            const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                            int64_t N, int32_t ld, const double *gains, int64_t B, uint32_t flags,
                            int32_t *delta, int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * hora_allocate_static — hora_allocate for callers that cannot allocate device memory.
 *
 * The paper has no counterpart to this call; it exists for the way the library gets embedded.  Some hosts of
 * this code may not call cudaMalloc (or any allocator that ends up there) at the point where they need an
 * allocation: code that runs inside a region where the allocator is frozen or instrumented, plug-ins that
 * are handed their input and output buffers by a framework and nothing else, or services that pre-size all
 * device memory at start-up and treat a later allocation as a fault.  For them the scratch that hora_allocate
 * needs lives inside the library: a fixed array of hora_allocate_static_capacity() bytes (8 MiB) in device
 * memory, present on every GPU that loads the library for as long as the process lives.
 *
 * Arguments and results are those of hora_allocate without `workspace` / `workspace_bytes`; the caller still
 * passes every input and output buffer.  The call itself allocates nothing and frees nothing.
 *
 *   - Size limit: hora_allocate_workspace_bytes(N, ld, gains == NULL, flags) must not exceed
 *     hora_allocate_static_capacity(); otherwise HORA_ERR_WORKSPACE is returned and nothing is enqueued.
 *     With a materialised gains matrix that admits about 2.5e5 prompts; with gains == NULL the
 *     matrix itself must fit, so only small problems (N*ld*8 bytes well under 8 MiB) qualify — except on the
 *     rank-based route (one prior for all prompts, gains == NULL), which builds no matrix: pass
 *     HORA_FLAG_SHARED_PRIOR as well and the need is about 0.6 MiB + 8 bytes per 256 prompts.
 *   - First use: the first call on each device looks up the array's device address (cudaGetSymbolAddress)
 *     with that device current, and caches it (as hora_allocate caches, per device, how many thread blocks of
 *     its cooperative kernel fit at once).  Make that first call outside any stream capture.  The cached
 *     address belongs to the device's context: after cudaDeviceReset it is stale, and the library must be
 *     reloaded before the call is used again.
 *   - Sharing: every call on a device uses the same array.  It keeps whatever the previous call left there;
 *     each call clears the parts it needs zeroed before using them, so back-to-back calls on one stream
 *     are fine.  Two calls that overlap on the GPU (different streams, or different host threads without
 *     ordering) race on the scratch and give undefined results: serialise them.
 */
size_t hora_allocate_static_capacity(void);   /* host: size of the built-in scratch in bytes */

hora_status_t hora_allocate_static(const double *alpha, const double *beta, double alpha0, double beta0,
                                   const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                                   int64_t N, int32_t ld, const double *gains, int64_t B, uint32_t flags,
                                   int32_t *delta, int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev,
                                   void *stream);

/*
 * hora_allocate_hard_first — the comparison allocator of Sec. 4.2 (paragraph "Comparison with the hard-first heuristic",
 * Table allocator-g0): after the G0 pre-rollouts the whole Phase-B budget goes to the prompts none of whose
 * pre-rollouts was correct (c_i = 0).  The paper prints no split rule; the one taken here is the plainest even
 * split: the budget is dealt one rollout at a time, round-robin in prompt order, to the c_i = 0 prompts that are
 * still below their cap, so they all end within one rollout of each other (or at their caps) and the earlier
 * prompts hold the extra ones.  What the c_i = 0 prompts cannot absorb (all at their caps, or no such prompt in
 * the batch) is dealt the same way to the remaining prompts, which makes the rule the uniform split when no
 * prompt has c_i = 0.  No prior enters: the rule looks at c_i and cap_i only.
 *
 *   c, G0, cap, cap_scalar, N, ld   as for hora_gains (ld <= 8192 here); B as for hora_allocate
 *   delta, G, group_offsets         as for hora_allocate
 *   info_dev                        status, n_above (rollouts dealt in full rounds), n_tied (prompts that could take
 *                                   one more in the last, partial round), n_tied_taken (those that did), sum_G, sum_cap;
 *                                   lambda and objective are 0, first_pass_bits is -1 (0 when B == 0)
 *   workspace                       hora_allocate_hard_first_workspace_bytes(N, ld) bytes, 256-byte aligned
 * Data-dependent failures (INVALID_VALUE for c_i outside [0, G0] or cap_i outside [0, ld]; INFEASIBLE for
 * B > sum_i cap_i) set info_dev->status and leave delta, G and group_offsets zero.
 */
size_t hora_allocate_hard_first_workspace_bytes(int64_t N, int32_t ld);

hora_status_t hora_allocate_hard_first(const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N,
                                       int32_t ld, int64_t B, int32_t *delta, int32_t *G, int64_t *group_offsets,
                                       hora_alloc_info *info_dev, void *workspace, size_t workspace_bytes, void *stream);

/*
 * hora_allocate_batched — many independent allocation problems in one call (the paper's appendix "Training
 * configurations": Phase-B allocation is run on mini-batches of the training batch, e.g. four shards of 15
 * prompts, each with its own budget, and Proposition 1 holds within each shard).
 *
 * Segment s covers prompts seg_offsets_host[s] .. seg_offsets_host[s+1]-1 and hands out budgets_host[s]
 * rollouts among them, exactly as hora_allocate would on that segment alone (same gains bit for bit, same tie
 * rules, same exact mode).  One CTA solves one segment in shared memory (one warp on precomputed ranks when the
 * prior is shared); no gains matrix is materialised.  With HORA_FLAG_HARD_FIRST every segment is allocated by the
 * comparison rule of hora_allocate_hard_first instead (the form the paper's ablation ran it in: per shard); the
 * priors are then unused, lambda and objective are 0, and no segment size limit applies.
 *
 *   alpha .. ld            as for hora_gains (device arrays over all N prompts)
 *   seg_offsets_host       HOST array [S+1], non-decreasing, [0] == 0, [S] == N
 *   budgets_host           HOST array [S], 0 <= budgets[s] <= sum of the segment's caps
 *   delta, G               int32 [N] out;  group_offsets int64 [N+1] out over all prompts, may be NULL
 *   info_dev               device array [S] of per-segment summaries (first_pass_bits is 0), may be NULL;
 *                          data-dependent failures are per segment: that segment's status is set and its
 *                          delta / G are zero, other segments are unaffected
 *   workspace              device scratch, 256-byte aligned, hora_allocate_batched_workspace_bytes(N, S)
 * Rows longer than 256 candidates are first solved on their first 256 (exact unless a prompt takes them all, or
 * the budget exceeds them); only the segments this does not settle are solved at full width, inside the same call.
 * Limits: a segment may hold at most 256 prompts and 176 KiB of keys (prompts * ld * 8 bytes); beyond that the
 * call returns HORA_ERR_WORKSPACE and hora_allocate should be used for that problem.  With ONE prior for all
 * prompts (alpha == beta == NULL) and (G0 + 1) * ld <= 8192 neither limit applies: the candidate values are ranked
 * once for all segments (as under hora_allocate's rank-based route, exactly or as doubles by the tie mode) and
 * every segment is solved on ranks by one warp, whatever its size.  The two host arrays are
 * copied to the device during the call and may be reused as soon as it returns.
 */
size_t hora_allocate_batched_workspace_bytes(int64_t N, int64_t S);

hora_status_t hora_allocate_batched(const double *alpha, const double *beta, double alpha0, double beta0,
                                    const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar,
                                    int64_t N, int32_t ld, const int64_t *seg_offsets_host,
                                    const int64_t *budgets_host, int64_t S, uint32_t flags, int32_t *delta,
                                    int32_t *G, int64_t *group_offsets, hora_alloc_info *info_dev,
                                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * hora_group_advantage — group-relative advantages over ragged groups (Sec. 3.1 for GRPO; the RLOO
 * compatibility paragraph of Sec. 4 for the leave-one-out form).
 *
 * Group g holds rewards[group_offsets[g] .. group_offsets[g+1]).  With S the group's sum and n its size:
 *   HORA_ADV_GRPO:  adv_j = (r_j - S/n) / (sqrt(sum_k (r_k - S/n)^2 / (n - ddof)) + eps); 0 when that
 *                   denominator is 0 (a zero-variance group gives no signal) or n - ddof <= 0
 *   HORA_ADV_RLOO:  adv_j = r_j - (S - r_j)/(n - 1); 0 when n == 1
 * Sums are accumulated in fp64 and rounded to fp32 once.  Empty groups are allowed.
 *
 *   rewards [total] fp32, group_offsets [N+1] int64 non-decreasing with group_offsets[0] == 0,
 *   adv [total] fp32 out, ddof in {0,1}, eps >= 0, status_dev optional (INVALID_VALUE on decreasing offsets).
 */
hora_status_t hora_group_advantage(const float *rewards, const int64_t *group_offsets, int64_t N,
                                   int32_t mode, float eps, int32_t ddof, float *adv,
                                   int32_t *status_dev, void *stream);

/*
 * hora_learned_prior — prior parameters from a predictor's outputs (appendix "Prior-design predictor details",
 * Eq. posterior-learned): alpha_i = s_i p_hat_i, beta_i = s_i (1 - p_hat_i); fed to hora_gains / hora_allocate,
 * which add the Phase-A counts, they give the posterior of Eq. posterior-learned.  s_i = clamp(softplus(s_raw_i),
 * 0.25, 16) when s_raw is given (the dual-head variants), else the fixed s_fixed (2 in the paper's single-head
 * variants; s = 2 with p_hat = 1/2 is the uniform prior).
 *   p_hat [N] fp64 in (0,1); s_raw [N] fp64 raw head output or NULL; alpha, beta [N] fp64 out;
 *   status_dev optional: INVALID_VALUE if some p_hat is outside (0,1) (that prompt gets alpha = beta = 0).
 *
 * hora_beta_binomial_nll — the per-prompt training loss of those predictors (same appendix):
 *   nll_i = -log( B(c_i + s_i p_hat_i, G0 - c_i + s_i (1 - p_hat_i)) / B(s_i p_hat_i, s_i (1 - p_hat_i)) )
 * with s_i as above; log-Beta through lgamma in fp64.  c [N] int32 in [0, G0]; nll [N] fp64 out.
 */
hora_status_t hora_learned_prior(const double *p_hat, const double *s_raw, double s_fixed, int64_t N,
                                 double *alpha, double *beta, int32_t *status_dev, void *stream);

hora_status_t hora_beta_binomial_nll(const double *p_hat, const double *s_raw, double s_fixed, const int32_t *c,
                                     int32_t G0, int64_t N, double *nll, int32_t *status_dev, void *stream);

/*
 * hora_allocation_share — how prompts and Phase-B budget split over the Phase-A success count (the statistic of
 * Fig. 3, Sec. 4.1): for k = 0..G0, prompts[k] = #{i : c_i = k}, budget[k] = sum of delta_i over those prompts.
 *   c, delta [N] int32 device; prompts, budget [G0+1] int64 device out (overwritten); 0 <= G0 <= 2047.
 *   status_dev optional: INVALID_VALUE if some c_i is outside [0, G0] or some delta_i < 0 (that prompt is skipped).
 */
hora_status_t hora_allocation_share(const int32_t *c, const int32_t *delta, int64_t N, int32_t G0,
                                    int64_t *prompts, int64_t *budget, int32_t *status_dev, void *stream);

/*
 * hora_pass_at_k — the unbiased Pass@K estimator (Eq. pass-k) averaged over prompts, for a grid of K values:
 *   pass_at_k[j] = mean over the Q prompts of  1 - C(n - c_q, K_j) / C(n, K_j),
 * c_q = correct samples among the n_samples drawn for prompt q.  Counts outside [0, n_samples] raise
 * INVALID_VALUE in status_dev and are left out of the sums; a K_j outside [0, n_samples] raises
 * INVALID_VALUE too and its output is 0 (C(n, K) is zero there, the estimator undefined).
 *   c [Q] int32 device; K_dev [n_K] int32 device; pass_at_k [n_K] fp64 device out;
 *   workspace: hora_pass_at_k_workspace_bytes(n_samples) bytes of device scratch, 8-byte aligned.
 */
size_t hora_pass_at_k_workspace_bytes(int32_t n_samples);

hora_status_t hora_pass_at_k(const int32_t *c, int64_t Q, int32_t n_samples, const int32_t *K_dev, int32_t n_K,
                             double *pass_at_k, int32_t *status_dev, void *workspace, size_t workspace_bytes,
                             void *stream);

/*
 * hora_rollout_weights — loss weight of every rollout under variable-size groups (Sec. 3.2, paragraph "Training
 * objective with variable-size groups": in Eq. grpo-objective 1/G becomes 1/G_i, so every prompt weighs the
 * same however many rollouts it was given).
 *
 *   HORA_WEIGHT_PER_TOKEN     weights[r] = 1 / (G_g * len_r)          the 1/G_i * 1/|o| of Eq. grpo-objective;
 *                             0 for a zero-length rollout.  The tokens of one prompt then sum to weight 1.
 *   HORA_WEIGHT_CONST_LENGTH  weights[r] = 1 / (G_g * length_const)   a length-free normalisation (the paper says
 *                             its runs use one from Dr. GRPO but prints no formula; the constant is the caller's,
 *                             e.g. the maximum response length)
 * with g the group of rollout r, G_g = group_offsets[g+1] - group_offsets[g], len_r = token_offsets[r+1] -
 * token_offsets[r].  One fp64 division, rounded to fp32.  hora_token_broadcast turns the result into per-token
 * weights in the packed token layout.
 *
 *   group_offsets [N+1] int64, token_offsets [R+1] int64 with R = group_offsets[N] (may be NULL in the
 *   CONST_LENGTH mode), weights [R] fp32 out, status_dev optional (INVALID_VALUE on decreasing offsets).
 */
hora_status_t hora_rollout_weights(const int64_t *group_offsets, int64_t N, const int64_t *token_offsets,
                                   int32_t mode, float length_const, float *weights, int32_t *status_dev,
                                   void *stream);

/*
 * hora_group_advantage_tokens — hora_group_advantage followed by hora_token_broadcast (and, when token_weight is
 * given, hora_rollout_weights broadcast the same way) in one kernel, with no per-rollout array in between
 * (Sec. 3.1, Eq. grpo-objective; Sec. 3.2 for the 1/G_i weight under variable-size groups):
 *   token_adv[t]    = adv of the rollout that owns token t, adv as defined for hora_group_advantage
 *   token_weight[t] = 1/(G_g len_r) (HORA_WEIGHT_PER_TOKEN) or 1/(G_g length_const) (HORA_WEIGHT_CONST_LENGTH)
 * for tokens t < min(T, token_offsets[R]).  Rollout r belongs to the group g with group_offsets[g] <= r <
 * group_offsets[g+1]; rollouts at or beyond group_offsets[N] get advantage and weight 0.
 *   rewards [group_offsets[N]] fp32; group_offsets [N+1] int64 non-decreasing from 0; token_offsets [R+1] int64
 *   non-decreasing from 0; token_adv [T] fp32 out; token_weight [T] fp32 out or NULL (weight_mode and
 *   length_const are then ignored); status_dev optional (INVALID_VALUE on decreasing group offsets).
 * All device pointers, caller-owned; enqueues one kernel on `stream`.
 */
hora_status_t hora_group_advantage_tokens(const float *rewards, const int64_t *group_offsets, int64_t N,
                                          const int64_t *token_offsets, int64_t R, int64_t T, int32_t mode,
                                          float eps, int32_t ddof, int32_t weight_mode, float length_const,
                                          float *token_adv, float *token_weight, int32_t *status_dev,
                                          void *stream);

/*
 * hora_token_broadcast — per-token advantages (Eq. grpo-objective: the advantage of a rollout does not
 * depend on the token position).
 *
 *   token_adv[t] = adv[r]   for token_offsets[r] <= t < token_offsets[r+1],   r = 0..R-1
 *
 *   adv [R] fp32, token_offsets [R+1] int64 non-decreasing with token_offsets[0] == 0,
 *   T = token_offsets[R] (the caller knows it: it sized token_adv), token_adv [T] fp32 out.
 * Zero-length rollouts are allowed.  Tokens at or beyond token_offsets[R] are not written.
 */
hora_status_t hora_token_broadcast(const float *adv, const int64_t *token_offsets, int64_t R, int64_t T,
                                   float *token_adv, void *stream);

/*
 * hora_allocate_profile_events — measurement aid, no counterpart in the paper.  With two non-NULL cudaEvent_t
 * handles (created by the caller with timing enabled), every following hora_allocate / hora_allocate_static
 * call records `start_event` just before and `stop_event` just after the launch of its full-read selection
 * pass (the kernel that reads the whole gains matrix) on the call's stream, so that kernel can be timed on
 * the device without a profiler.  Pass NULLs to switch it off (the default).  The setting belongs to the calling
 * host thread: only hora_allocate calls issued by that thread record the events, so allocations running at the
 * same time from other threads (on other streams) are not touched.
 */
void hora_allocate_profile_events(void *start_event, void *stop_event);

/*
 * hora_allocate_profile_stages — measurement aid, no counterpart in the paper.  `events_host` is a HOST array of
 * n <= 7 cudaEvent_t handles (timing enabled); every following hora_allocate / hora_allocate_static call records
 * them on its stream at these points:  [0] entry (after the workspace is cleared), [1] after the sampled estimate,
 * [2] after the full-read pass, [3] after the per-row pass (level 1), [4] after the tail (threshold complete,
 * prefixes over prompts formed), [5] after the exact tie ranking (right after [4] when that does not run),
 * [6] after the outputs are written.  Differences of consecutive events are the device times of the stages.
 * A NULL handle skips its point; NULL or n = 0 switches everything off (the default).  Per host thread, like
 * hora_allocate_profile_events; the array is read during this call only.  On the rank-based route the points are
 * [0] entry, [1] after the rank tables, [2] = [3] after the counting pass, [4] = [5] after the sums, [6] after the
 * outputs.
 */
void hora_allocate_profile_stages(void *const *events_host, int32_t n);

/*
 * hora_fp64_probe — measurement aid, no counterpart in the paper.  Enqueues one kernel that does nothing but
 * independent fp64 fused multiply-adds (8 chains per thread, 8 CTAs of 256 threads per multiprocessor, `iters`
 * steps per chain) and returns how many FMAs that launch performs (0 on a bad argument or a failed launch).
 * Timed with events by the caller it gives the device's fp64 rate: 2 * FMAs / seconds flop/s, the peak that
 * kernels bound by plain fp64 arithmetic are held against.  sink_dev: one double in device memory (never written
 * in practice; it only keeps the arithmetic alive).
 */
uint64_t hora_fp64_probe(int32_t iters, double *sink_dev, void *stream);

/*
 * hora_checked_violation — verification aid, no counterpart in the paper.  The library can be built a second time
 * with -DHORA_CHECKED (python -m paper_2605_07114_b200.build --checked writes libhora_checked.so): every access of
 * the allocation, batched-allocation and advantage kernels whose index is computed from device data then checks
 * that index against the size of its array; a violation is recorded (never trapped: the access goes to a scratch
 * slot and the kernel runs on).  This call synchronises the device and returns 0 if no check has failed since the
 * last call, else (file id << 20) | source line of the first failure (file ids: 1 hora_allocate.cu,
 * 2 hora_allocate_batched.cu, 3 hora_advantage.cu, 4 hora_rank.cu); the record is cleared.  The normal build has no
 * checks and returns -1; -2 reports a failed synchronisation.
 */
int32_t hora_checked_violation(void);

const char *hora_status_string(hora_status_t status);   /* host: static string */
int         hora_version(void);                         /* host: major*10000 + minor*100 + patch */
uint64_t    hora_launch_count(void);                    /* host: kernels this library has launched so far in this
                                                           process (memsets not counted); for benchmarks' bookkeeping */

#ifdef __cplusplus
}
#endif
#endif /* HORA_H */
