// Exact integer arithmetic for the tie path and the product form of the hit utility; shared by the
// single-problem and the batched allocation kernels.
//
// For an integer posterior (a, b) the gain of Eq. marginal is a ratio of two products of small integers,
//     g(Delta) = a (b)_a / (b + Delta - 1)_{a+1}          (x)_k = x (x+1) ... (x+k-1)
//              = a (b)_{Delta-1} / (a + b)_Delta           (the same value; fewer factors when Delta <= a)
// Numerator and denominator are held unreduced in kLimbs 64-bit words (512 bits); two gains are compared by
// cross multiplication with 1024-bit products formed column by column, so nothing is ever rounded.  Whatever
// does not fit is reported (never wrapped): m = min(a + 1, Delta) factors, each below a + b + Delta, must
// satisfy m log2(a + b + Delta) <= 512 — any a <= 50 with Delta up to 1000, or any a at all with Delta <= 25.
#pragma once

#include "hora_common.cuh"

namespace hora {

constexpr int kLimbs = 8;
template <int L>
struct UBigT { unsigned long long w[L]; };                  // little-endian words
using UBig = UBigT<kLimbs>;

template <int L>
__device__ __forceinline__ void set_small(UBigT<L> &x, unsigned long long v) {
    x.w[0] = v;
#pragma unroll
    for (int i = 1; i < L; ++i) x.w[i] = 0ull;
}

// x *= m; returns false if the product does not fit (x is then meaningless)
template <int L>
__device__ __forceinline__ bool mul_small(UBigT<L> &x, unsigned long long m) {
    unsigned long long carry = 0ull;
#pragma unroll
    for (int i = 0; i < L; ++i) {
        const unsigned long long lo = x.w[i] * m, hi = __umul64hi(x.w[i], m);
        const unsigned long long s = lo + carry;
        x.w[i] = s;
        carry = hi + (s < lo ? 1ull : 0ull);                 // hi <= 2^64 - 2: no wrap
    }
    return carry == 0ull;
}

// (c2, c1, c0) += p * q, a 192-bit accumulator
__device__ __forceinline__ void mac192(unsigned long long &c0, unsigned long long &c1, unsigned long long &c2,
                                       unsigned long long p, unsigned long long q) {
    const unsigned long long lo = p * q, hi = __umul64hi(p, q);
    c0 += lo;
    const unsigned long long k0 = c0 < lo ? 1ull : 0ull;
    const unsigned long long t = hi + k0;                    // hi <= 2^64 - 2: no wrap
    c1 += t;
    c2 += c1 < t ? 1ull : 0ull;
}

// sign of x*y - u*v.  The two double-width products are formed a 64-bit column at a time from the bottom (three
// words of running carry each), and the most significant column in which they differ decides.
template <int L>
__device__ __forceinline__ int cmp_products(const UBigT<L> &x, const UBigT<L> &y, const UBigT<L> &u, const UBigT<L> &v) {
    unsigned long long l0 = 0, l1 = 0, l2 = 0, r0 = 0, r1 = 0, r2 = 0;
    int sign = 0;
#pragma unroll
    for (int k = 0; k < 2 * L; ++k) {
#pragma unroll
        for (int i = 0; i < L; ++i) {
            const int j = k - i;
            if (j >= 0 && j < L) {
                mac192(l0, l1, l2, x.w[i], y.w[j]);
                mac192(r0, r1, r2, u.w[i], v.w[j]);
            }
        }
        if (l0 != r0) sign = l0 > r0 ? 1 : -1;
        l0 = l1; l1 = l2; l2 = 0;
        r0 = r1; r1 = r2; r2 = 0;
    }
    return sign;
}

// Exact gain of type (a, b, Delta) as num/den (not reduced).  Returns false if L words do not suffice.
template <int L>
__device__ __forceinline__ bool exact_gain(unsigned long long a, unsigned long long b, unsigned long long Delta,
                                           UBigT<L> &num, UBigT<L> &den) {
    set_small(num, a);
    set_small(den, 1ull);
    bool ok = true;
    if (a + 1 <= Delta) {               // a (b)_a / (b+Delta-1)_{a+1}
        for (unsigned long long k = 0; k < a && ok; ++k) ok = mul_small(num, b + k);
        for (unsigned long long k = 0; k <= a && ok; ++k) ok = mul_small(den, b + Delta - 1 + k);
    } else {                            // a (b)_{Delta-1} / (a+b)_{Delta}
        for (unsigned long long j = 0; j + 1 < Delta && ok; ++j) ok = mul_small(num, b + j);
        for (unsigned long long j = 0; j < Delta && ok; ++j) ok = mul_small(den, a + b + j);
    }
    return ok;
}

// sign of g_{a1,b1}(D1) - g_{a2,b2}(D2) on exact fractions: in 128-bit words when both fit (the usual case, a
// fraction of the work), else in the full width; *overflow is set when that does not suffice either
static __device__ __noinline__ int exact_compare_types(unsigned long long a1, unsigned long long b1, unsigned long long D1,
                                                unsigned long long a2, unsigned long long b2, unsigned long long D2,
                                                bool *overflow) {
    {
        UBigT<2> n1, d1, n2, d2;
        if (exact_gain(a1, b1, D1, n1, d1) && exact_gain(a2, b2, D2, n2, d2)) return cmp_products(n1, d2, n2, d1);
    }
    UBig n1, d1, n2, d2;
    if (!exact_gain(a1, b1, D1, n1, d1) || !exact_gain(a2, b2, D2, n2, d2)) {
        *overflow = true;
        return 0;
    }
    return cmp_products(n1, d2, n2, d1);
}

// nearest double of a kLimbs-word integer, up to the rounding of the partial sums (used for reporting only)
__device__ __forceinline__ double to_double(const UBig &x) {
    double v = 0.0;
#pragma unroll
    for (int i = kLimbs - 1; i >= 0; --i) v = v * 18446744073709551616.0 + (double)x.w[i];
    return v;
}

// num/den as a double (2^512 is far inside the range of a double; a handful of roundings, reporting only)
__device__ __forceinline__ double ratio_double(const UBig &num, const UBig &den) { return to_double(num) / to_double(den); }

// g_{a,b}(Delta) as the double nearest its exact fraction (reporting only); false if the fraction does not fit.
// Kept out of line: the callers are large kernels that need it once per problem.
static __device__ __noinline__ bool exact_gain_as_double(unsigned long long a, unsigned long long b, unsigned long long Delta,
                                                         double *out) {
    UBig nu, de;
    if (!exact_gain(a, b, Delta, nu, de)) return false;
    *out = ratio_double(nu, de);
    return true;
}

// U(Delta) = 1 - prod_{j<Delta} (b+j)/(a+b+j)  (Eq. appendix-hit-closed-form written as a product)
__device__ __forceinline__ double hit_utility(double a, double b, int32_t Delta) {
    double q = 1.0, num = 1.0, den = 1.0;
    double nb = b, nd = a + b;                              // b + j and a + b + j, advanced by exact additions
    for (int32_t j = 0; j < Delta; ++j) {
        num *= nb;
        den *= nd;
        nb += 1.0;
        nd += 1.0;
        if ((j & 7) == 7) { q *= num / den; num = 1.0; den = 1.0; }
    }
    q *= num / den;
    return 1.0 - q;
}

}  // namespace hora
