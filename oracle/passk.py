"""Test infrastructure only: the unbiased Pass@K estimator written out from its definition (Eq. pass-k).

For a prompt with c correct samples out of n,  pass@K = 1 - C(n - c, K) / C(n, K); the reported figure is the
mean over prompts.  Exact integer binomials and Fractions, one prompt at a time; converted to float at the end.
"""
from fractions import Fraction
from math import comb


def pass_at_k_one(n: int, c: int, K: int) -> Fraction:
    if not (0 <= c <= n) or not (0 <= K <= n):
        raise ValueError("need 0 <= c <= n and 0 <= K <= n")
    return 1 - Fraction(comb(n - c, K), comb(n, K))


def pass_at_k(counts, n: int, Ks):
    """Mean over prompts, one value per K (floats, rounded once from the exact mean)."""
    counts = [int(v) for v in counts]
    out = []
    for K in Ks:
        tot = Fraction(0)
        for c in counts:
            tot += pass_at_k_one(n, c, int(K))
        out.append(float(tot / len(counts)) if counts else 0.0)
    return out
