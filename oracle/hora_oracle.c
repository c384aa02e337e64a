/*
 * CPU oracle for the HORA rollout-allocation hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the path computes, written from the paper's
 * definitions.  It shares no code, header, table or helper with the CUDA library and is never
 * on the product path: only the test-suite, the smoke check and the CPU-baseline leg of the
 * benchmark load it.  Everything runs on one host thread.
 *
 *   posterior            a_i = alpha_i + c_i,  b_i = beta_i + G0 - c_i            (Eq. posterior)
 *   marginal gain        M_i(0) = a/(a+b),  M_i(l+1) = M_i(l) (b+l)/(a+b+l+1)      (Sec. 3.2, text after Eq. marginal)
 *                        g_i(Delta) := M_i(Delta-1),  stored at gains[i][Delta-1]
 *   hit utility          U_i(Delta) = 1 - prod_{j<Delta} (b+j)/(a+b+j)             (Eq. appendix-hit-closed-form)
 *   allocation           B greedy steps, each giving one more rollout to the prompt with the
 *                        largest current marginal gain                             (Algorithm 1, Phase B)
 *                        ties: lower prompt index first (the paper is silent; this is the reading
 *                        this repository fixes); caps 0 <= Delta_i <= cap_i restrict the argmax
 *   group sizes          G_i = G0 + Delta_i                                         (Sec. 3.2)
 *   GRPO advantage       (r - mean) / (std + eps) over the group, 0 when that denominator is 0   (Sec. 3.1)
 *   RLOO advantage       r - mean of the other G-1 rewards; 0 for a group of one    (Sec. 4, RLOO paragraph)
 *   token advantage      the rollout's advantage repeated over its tokens           (Eq. grpo-objective)
 *
 * Precision: real-valued priors use x87 long double (64-bit mantissa) for gains, utilities and
 * the objective.  Integer-valued priors use exact rationals (reduced fractions of unsigned
 * 128-bit integers; any overflow is reported, never wrapped), so a tie is an exact equality.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py against closed forms,
 * Beta-function ratios from a library lgamma, Monte-Carlo, brute-force enumeration and a literal
 * O(B*N) transcription of the greedy loop in Python fractions.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_INFEASIBLE = 2, ORACLE_NOT_INTEGER = 3,
       ORACLE_OVERFLOW = 4, ORACLE_NOMEM = 5 };

/* ------------------------------------------------------------------ posterior (Eq. posterior) */
static int posterior(const double *alpha, const double *beta, double alpha0, double beta0,
                     const int32_t *c, int32_t G0, int64_t i, long double *a, long double *b)
{
    long double al = alpha ? (long double)alpha[i] : (long double)alpha0;
    long double be = beta ? (long double)beta[i] : (long double)beta0;
    if (!(al > 0.0L) || !(be > 0.0L) || !isfinite((double)al) || !isfinite((double)be)) return ORACLE_BAD_ARG;
    if (c[i] < 0 || c[i] > G0) return ORACLE_BAD_ARG;
    *a = al + (long double)c[i];
    *b = be + (long double)(G0 - c[i]);
    return ORACLE_OK;
}

/* ------------------------------------------------- gains by the recurrence (long double rows) */
int oracle_gains(const double *alpha, const double *beta, double alpha0, double beta0,
                 const int32_t *c, int32_t G0, const int32_t *cap, int64_t N, int32_t ld,
                 double *gains /* [N][ld]; entries beyond cap_i are 0 */)
{
    for (int64_t i = 0; i < N; ++i) {
        long double a, b;
        int rc = posterior(alpha, beta, alpha0, beta0, c, G0, i, &a, &b);
        if (rc) return rc;
        if (cap[i] < 0 || cap[i] > ld) return ORACLE_BAD_ARG;
        long double m = a / (a + b);                              /* M(0) */
        for (int32_t l = 0; l < ld; ++l) {
            gains[i * (int64_t)ld + l] = (l < cap[i]) ? (double)m : 0.0;
            m = m * (b + l) / (a + b + l + 1);                    /* M(l+1) */
        }
    }
    return ORACLE_OK;
}

/* g(Delta) for one posterior, long double, rounded to double on return */
double oracle_gain_one(double a, double b, int32_t Delta)
{
    long double A = a, Bq = b, m = A / (A + Bq);
    for (int32_t l = 0; l + 1 < Delta; ++l) m = m * (Bq + l) / (A + Bq + l + 1);
    return (double)m;
}

/* U(Delta) = 1 - prod_{j<Delta} (b+j)/(a+b+j) in long double */
static long double utility_ld(long double a, long double b, int32_t Delta)
{
    long double q = 1.0L;
    for (int32_t j = 0; j < Delta; ++j) q = q * (b + j) / (a + b + j);
    return 1.0L - q;
}

double oracle_utility_one(double a, double b, int32_t Delta) { return (double)utility_ld(a, b, Delta); }

/* ---------------------------------------------------------------- heap greedy, real priors */
typedef struct { long double key; int64_t idx; } rnode;

static int r_before(const rnode *x, const rnode *y)      /* x is popped before y */
{
    if (x->key != y->key) return x->key > y->key;
    return x->idx < y->idx;
}

static void r_sift_down(rnode *h, int64_t n, int64_t k)
{
    for (;;) {
        int64_t l = 2 * k + 1, r = l + 1, m = k;
        if (l < n && r_before(&h[l], &h[m])) m = l;
        if (r < n && r_before(&h[r], &h[m])) m = r;
        if (m == k) return;
        rnode t = h[k]; h[k] = h[m]; h[m] = t;
        k = m;
    }
}

int oracle_greedy_real(const double *alpha, const double *beta, double alpha0, double beta0,
                       const int32_t *c, int32_t G0, const int32_t *cap, int64_t N, int64_t B,
                       int32_t *delta /* [N] out */, int32_t *G /* [N] out */,
                       double *lambda_out /* gain of the last rollout given out */,
                       double *objective_out /* sum_i U_i(Delta_i) */)
{
    if (N < 0 || B < 0) return ORACLE_BAD_ARG;
    long double *a = malloc(sizeof(long double) * (size_t)(N ? N : 1));
    long double *b = malloc(sizeof(long double) * (size_t)(N ? N : 1));
    rnode *h = malloc(sizeof(rnode) * (size_t)(N ? N : 1));
    if (!a || !b || !h) { free(a); free(b); free(h); return ORACLE_NOMEM; }
    int rc = ORACLE_OK;
    int64_t n = 0, total_cap = 0;
    for (int64_t i = 0; i < N && !rc; ++i) {
        rc = posterior(alpha, beta, alpha0, beta0, c, G0, i, &a[i], &b[i]);
        if (!rc && cap[i] < 0) rc = ORACLE_BAD_ARG;
        if (rc) break;
        delta[i] = 0;
        total_cap += cap[i];
        if (cap[i] > 0) { h[n].key = a[i] / (a[i] + b[i]); h[n].idx = i; ++n; }   /* M_i(0) */
    }
    if (!rc && B > total_cap) rc = ORACLE_INFEASIBLE;
    if (!rc) {
        for (int64_t k = n / 2 - 1; k >= 0; --k) r_sift_down(h, n, k);
        long double last = 0.0L;
        for (int64_t step = 0; step < B; ++step) {               /* Algorithm 1, Phase B loop */
            int64_t i = h[0].idx;                                 /* argmax_i M_i(Delta_i) */
            last = h[0].key;
            int32_t l = delta[i];
            delta[i] = l + 1;
            if (delta[i] < cap[i]) {
                h[0].key = h[0].key * (b[i] + l) / (a[i] + b[i] + l + 1);   /* M_i(l+1) */
            } else {
                h[0] = h[n - 1]; --n;
            }
            if (n > 0) r_sift_down(h, n, 0);
        }
        long double obj = 0.0L;
        for (int64_t i = 0; i < N; ++i) { obj += utility_ld(a[i], b[i], delta[i]); G[i] = G0 + delta[i]; }
        if (lambda_out) *lambda_out = (double)last;
        if (objective_out) *objective_out = (double)obj;
    }
    free(a); free(b); free(h);
    return rc;
}

/* ------------------------------------------------------------- exact rationals (integer priors) */
typedef struct { u128 n, d; } rat;            /* reduced, d > 0 */

static u128 gcd_u128(u128 x, u128 y) { while (y) { u128 t = x % y; x = y; y = t; } return x; }

/* r * (p/q) with p, q small positive integers; 0 on success, 1 on overflow */
static int rat_mul_small(rat *r, uint64_t p, uint64_t q)
{
    u128 g0 = gcd_u128(p, q); p /= (uint64_t)g0; q /= (uint64_t)g0;
    u128 g1 = gcd_u128(r->n, q);
    u128 g2 = gcd_u128(r->d, p);
    u128 nn, dd;
    if (__builtin_mul_overflow(r->n / g1, (u128)p / g2, &nn)) return 1;
    if (__builtin_mul_overflow(r->d / g2, (u128)q / g1, &dd)) return 1;
    r->n = nn; r->d = dd;
    return 0;
}

/* sign of x - y; *ovf set when the cross products do not fit 128 bits */
static int rat_cmp(const rat *x, const rat *y, int *ovf)
{
    u128 l, r;
    if (__builtin_mul_overflow(x->n, y->d, &l) || __builtin_mul_overflow(y->n, x->d, &r)) { *ovf = 1; return 0; }
    return (l > r) - (l < r);
}

static int as_int(double v, int64_t *out)
{
    if (!(v > 0.0) || v > 1.0e9 || v != floor(v)) return 1;
    *out = (int64_t)v;
    return 0;
}

typedef struct { rat key; int64_t idx; } enode;

static int e_before(const enode *x, const enode *y, int *ovf)
{
    int s = rat_cmp(&x->key, &y->key, ovf);
    if (s) return s > 0;
    return x->idx < y->idx;
}

static void e_sift_down(enode *h, int64_t n, int64_t k, int *ovf)
{
    for (;;) {
        int64_t l = 2 * k + 1, r = l + 1, m = k;
        if (l < n && e_before(&h[l], &h[m], ovf)) m = l;
        if (r < n && e_before(&h[r], &h[m], ovf)) m = r;
        if (m == k) return;
        enode t = h[k]; h[k] = h[m]; h[m] = t;
        k = m;
    }
}

/* exact U(Delta) = 1 - prod_{j<Delta}(b+j)/(a+b+j) as a rational, returned as long double */
static int utility_exact(int64_t a, int64_t b, int32_t Delta, long double *out)
{
    rat q = { 1, 1 };
    for (int32_t j = 0; j < Delta; ++j)
        if (rat_mul_small(&q, (uint64_t)(b + j), (uint64_t)(a + b + j))) return 1;
    u128 num = q.d - q.n;                       /* 1 - n/d */
    *out = (long double)num / (long double)q.d;
    return 0;
}

int oracle_greedy_exact(const double *alpha, const double *beta, double alpha0, double beta0,
                        const int32_t *c, int32_t G0, const int32_t *cap, int64_t N, int64_t B,
                        int32_t *delta, int32_t *G,
                        uint64_t *lambda_num_out /* [2]: lo, hi words */, uint64_t *lambda_den_out /* [2] */,
                        double *objective_out)
{
    if (N < 0 || B < 0) return ORACLE_BAD_ARG;
    int64_t *a = malloc(sizeof(int64_t) * (size_t)(N ? N : 1));
    int64_t *b = malloc(sizeof(int64_t) * (size_t)(N ? N : 1));
    enode *h = malloc(sizeof(enode) * (size_t)(N ? N : 1));
    if (!a || !b || !h) { free(a); free(b); free(h); return ORACLE_NOMEM; }
    int rc = ORACLE_OK, ovf = 0;
    int64_t n = 0, total_cap = 0;
    for (int64_t i = 0; i < N; ++i) {
        int64_t ai, bi;
        if (as_int(alpha ? alpha[i] : alpha0, &ai) || as_int(beta ? beta[i] : beta0, &bi)) { rc = ORACLE_NOT_INTEGER; break; }
        if (c[i] < 0 || c[i] > G0 || cap[i] < 0) { rc = ORACLE_BAD_ARG; break; }
        a[i] = ai + c[i];                                   /* Eq. posterior */
        b[i] = bi + G0 - c[i];
        delta[i] = 0;
        total_cap += cap[i];
        if (cap[i] > 0) {
            rat m = { 1, 1 };
            if (rat_mul_small(&m, (uint64_t)a[i], (uint64_t)(a[i] + b[i]))) { rc = ORACLE_OVERFLOW; break; }  /* M(0) */
            h[n].key = m; h[n].idx = i; ++n;
        }
    }
    if (!rc && B > total_cap) rc = ORACLE_INFEASIBLE;
    if (!rc) {
        for (int64_t k = n / 2 - 1; k >= 0; --k) e_sift_down(h, n, k, &ovf);
        rat last = { 0, 1 };
        for (int64_t step = 0; step < B && !ovf; ++step) {        /* Algorithm 1, Phase B loop */
            int64_t i = h[0].idx;
            last = h[0].key;
            int32_t l = delta[i];
            delta[i] = l + 1;
            if (delta[i] < cap[i]) {
                if (rat_mul_small(&h[0].key, (uint64_t)(b[i] + l), (uint64_t)(a[i] + b[i] + l + 1))) { ovf = 1; break; }
            } else {
                h[0] = h[n - 1]; --n;
            }
            if (n > 0) e_sift_down(h, n, 0, &ovf);
        }
        if (ovf) rc = ORACLE_OVERFLOW;
        if (!rc) {
            long double obj = 0.0L;
            for (int64_t i = 0; i < N; ++i) {
                long double u;
                if (utility_exact(a[i], b[i], delta[i], &u)) { rc = ORACLE_OVERFLOW; break; }
                obj += u;
                G[i] = G0 + delta[i];
            }
            if (lambda_num_out) { lambda_num_out[0] = (uint64_t)last.n; lambda_num_out[1] = (uint64_t)(last.n >> 64); }
            if (lambda_den_out) { lambda_den_out[0] = (uint64_t)last.d; lambda_den_out[1] = (uint64_t)(last.d >> 64); }
            if (objective_out) *objective_out = (double)obj;
        }
    }
    free(a); free(b); free(h);
    return rc;
}

/* ---------------------------------------------------------------- group advantages (Sec. 3.1) */
int oracle_group_advantage(const float *rewards, const int64_t *off, int64_t N, int32_t mode /*0 GRPO, 1 RLOO*/,
                           double eps, int32_t ddof, float *adv)
{
    if (mode != 0 && mode != 1) return ORACLE_BAD_ARG;
    if (ddof != 0 && ddof != 1) return ORACLE_BAD_ARG;
    for (int64_t g = 0; g < N; ++g) {
        int64_t s = off[g], e = off[g + 1];
        if (e < s) return ORACLE_BAD_ARG;
        int64_t Gn = e - s;
        if (Gn == 0) continue;
        double sum = 0.0;
        for (int64_t j = s; j < e; ++j) sum += (double)rewards[j];
        if (mode == 0) {
            double mean = sum / (double)Gn, ss = 0.0;
            for (int64_t j = s; j < e; ++j) { double d = (double)rewards[j] - mean; ss += d * d; }
            double var = (Gn - ddof > 0) ? ss / (double)(Gn - ddof) : 0.0;
            double den = sqrt(var) + eps;
            for (int64_t j = s; j < e; ++j)
                adv[j] = (den > 0.0) ? (float)(((double)rewards[j] - mean) / den) : 0.0f;
        } else {
            for (int64_t j = s; j < e; ++j)
                adv[j] = (Gn > 1) ? (float)((double)rewards[j] - (sum - (double)rewards[j]) / (double)(Gn - 1)) : 0.0f;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------ per-token advantage (Eq. grpo-objective) */
int oracle_token_broadcast(const float *adv, const int64_t *tok_off, int64_t R, float *out)
{
    for (int64_t r = 0; r < R; ++r) {
        if (tok_off[r + 1] < tok_off[r]) return ORACLE_BAD_ARG;
        for (int64_t t = tok_off[r]; t < tok_off[r + 1]; ++t) out[t] = adv[r];
    }
    return ORACLE_OK;
}

/* ----------------------- loss weights under variable-size groups (Sec. 3.2, last paragraph) */
/* mode 0: 1/(G_g * len_r), the 1/G_i and 1/|o| of Eq. grpo-objective; mode 1: 1/(G_g * length_const) */
int oracle_rollout_weights(const int64_t *goff, int64_t N, const int64_t *toff, int32_t mode, double length_const,
                           float *weights)
{
    if (mode != 0 && mode != 1) return ORACLE_BAD_ARG;
    for (int64_t g = 0; g < N; ++g) {
        if (goff[g + 1] < goff[g]) return ORACLE_BAD_ARG;
        double G = (double)(goff[g + 1] - goff[g]);
        for (int64_t r = goff[g]; r < goff[g + 1]; ++r) {
            double denom = G * length_const;
            if (mode == 0) {
                if (toff[r + 1] < toff[r]) return ORACLE_BAD_ARG;
                denom = G * (double)(toff[r + 1] - toff[r]);
            }
            weights[r] = denom > 0.0 ? (float)(1.0 / denom) : 0.0f;
        }
    }
    return ORACLE_OK;
}
