// Exact integer arithmetic for the tie path (unsigned 128-bit values as two words, 256-bit products) and
// the product form of the hit utility; shared by the single-problem and the batched allocation kernels.
#pragma once

#include "hora_common.cuh"

namespace hora {

// Exact arithmetic helpers (unsigned 128-bit as two words; overflow is reported, never wrapped).
struct U128 { unsigned long long lo, hi; };

__device__ __forceinline__ bool mul_small(U128 &x, unsigned long long m) {   // returns false on overflow
    const unsigned long long lo = x.lo * m, carry = __umul64hi(x.lo, m);
    const unsigned long long hi = x.hi * m;
    const bool ovf = (__umul64hi(x.hi, m) != 0) || (hi + carry < hi);
    x.lo = lo;
    x.hi = hi + carry;
    return !ovf;
}

// 128 x 128 -> 256 bit product, little-endian words
__device__ __forceinline__ void mul_wide(const U128 &p, const U128 &q, unsigned long long r[4]) {
    const unsigned long long a0 = p.lo, a1 = p.hi, b0 = q.lo, b1 = q.hi;
    r[0] = a0 * b0;
    const unsigned long long t1 = __umul64hi(a0, b0);
    const unsigned long long l01 = a0 * b1, h01 = __umul64hi(a0, b1);
    const unsigned long long l10 = a1 * b0, h10 = __umul64hi(a1, b0);
    const unsigned long long s = t1 + l01;
    unsigned long long c1 = s < t1;
    const unsigned long long s2 = s + l10;
    c1 += s2 < s;
    r[1] = s2;
    const unsigned long long l11 = a1 * b1, h11 = __umul64hi(a1, b1);
    const unsigned long long q2 = h01 + h10;
    unsigned long long c2 = q2 < h01;
    const unsigned long long q3 = q2 + l11;
    c2 += q3 < q2;
    const unsigned long long q4 = q3 + c1;
    c2 += q4 < q3;
    r[2] = q4;
    r[3] = h11 + c2;
}

// sign of x*y - u*v with full 256-bit products
__device__ __forceinline__ int cmp_products(const U128 &x, const U128 &y, const U128 &u, const U128 &v) {
    unsigned long long L[4], Rr[4];
    mul_wide(x, y, L);
    mul_wide(u, v, Rr);
    for (int i = 3; i >= 0; --i) {
        if (L[i] != Rr[i]) return L[i] > Rr[i] ? 1 : -1;
    }
    return 0;
}

// Exact gain of type (a, b, Delta) as num/den (not reduced).  Returns false if 128 bits do not suffice.
__device__ __forceinline__ bool exact_gain(unsigned long long a, unsigned long long b, unsigned long long Delta, U128 &num, U128 &den) {
    num.lo = a; num.hi = 0;
    den.lo = 1; den.hi = 0;
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
