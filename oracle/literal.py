"""The method's definitions in Python ``fractions`` — the most literal form, for small cases.

TEST INFRASTRUCTURE ONLY (never imported by the product).  Each function is the paper's
formula or loop written out with exact rationals; no heap, no blocking, no shortcuts.  The
C oracle is checked against these on small inputs, and these are checked against closed forms,
library Beta functions, Monte-Carlo and brute force in ``tests/test_oracle_pins.py``.
"""
from __future__ import annotations

from fractions import Fraction
from typing import List, Sequence, Tuple


def posterior(alpha, beta, c: int, G0: int) -> Tuple[Fraction, Fraction]:
    """Eq. posterior: (a, b) = (alpha + c, beta + G0 - c)."""
    return Fraction(alpha) + c, Fraction(beta) + G0 - c


def marginals(a: Fraction, b: Fraction, count: int) -> List[Fraction]:
    """M(0), ..., M(count-1) by the recurrence stated after Eq. marginal."""
    out = []
    m = a / (a + b)
    for l in range(count):
        out.append(m)
        m = m * (b + l) / (a + b + l + 1)
    return out


def utility(a: Fraction, b: Fraction, Delta: int) -> Fraction:
    """Eq. appendix-hit-closed-form written as a product: 1 - prod_{j<Delta} (b+j)/(a+b+j)."""
    q = Fraction(1)
    for j in range(Delta):
        q = q * (b + j) / (a + b + j)
    return 1 - q


def greedy(ab: Sequence[Tuple[Fraction, Fraction]], cap: Sequence[int], B: int) -> List[int]:
    """The greedy rule of Algorithm 1, Phase B: B times, give one rollout to the prompt with
    the largest current marginal gain.  Ties go to the lowest prompt index (``max`` over an
    ascending scan with a strict comparison); prompts at their cap are not eligible."""
    N = len(ab)
    if B > sum(cap):
        raise ValueError("infeasible")
    delta = [0] * N
    cur = [a / (a + b) for a, b in ab]
    for _ in range(B):
        best = -1
        for i in range(N):
            if delta[i] < cap[i] and (best < 0 or cur[i] > cur[best]):
                best = i
        a, b = ab[best]
        l = delta[best]
        delta[best] = l + 1
        cur[best] = cur[best] * (b + l) / (a + b + l + 1)
    return delta


def greedy_heap(ab: Sequence[Tuple[Fraction, Fraction]], cap: Sequence[int], B: int):
    """The same B greedy steps with the argmax kept in a binary heap (key: gain descending, prompt index
    ascending), in unbounded Python integers: for sizes the O(B*N) scan above is too slow for, and for integer
    posteriors whose exact gains outgrow any fixed word size.  Returns (delta, gain of the last rollout given)."""
    import heapq
    N = len(ab)
    if B > sum(cap):
        raise ValueError("infeasible")
    delta = [0] * N
    heap = [(-(a / (a + b)), i) for i, (a, b) in enumerate(ab) if cap[i] > 0]
    heapq.heapify(heap)
    last = Fraction(0)
    for _ in range(B):
        neg, i = heap[0]
        last = -neg
        a, b = ab[i]
        l = delta[i]
        delta[i] = l + 1
        if delta[i] < cap[i]:
            heapq.heapreplace(heap, (neg * (b + l) / (a + b + l + 1), i))
        else:
            heapq.heappop(heap)
    return delta, last


def objective(ab, delta) -> Fraction:
    return sum((utility(a, b, d) for (a, b), d in zip(ab, delta)), Fraction(0))
