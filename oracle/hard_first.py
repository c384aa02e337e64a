"""The hard-first comparison allocator, in plain Python loops.  TEST INFRASTRUCTURE ONLY.

Sec. 4.2, paragraph "Comparison with the hard-first heuristic" (Table allocator-g0): after the G0 pre-rollouts the
Phase-B budget goes only to the prompts with c_i = 0.  The paper gives no split rule.  Reading taken here: the
budget is dealt one rollout at a time, round-robin in prompt order, to the c_i = 0 prompts still below their cap;
whatever they cannot absorb is dealt the same way to the other prompts (so a batch without any c_i = 0 prompt gets
the uniform split).  Pinned in tests/test_oracle_pins.py by a hand example, by the invariants of an even split and
by the closed form of the water level.
"""
from __future__ import annotations

from typing import List, Sequence


def deal(indices: Sequence[int], cap: Sequence[int], delta: List[int], budget: int) -> int:
    """Round-robin dealing over `indices` (in the given order); returns what is left of the budget."""
    while budget > 0:
        gave = False
        for i in indices:
            if budget == 0:
                break
            if delta[i] < cap[i]:
                delta[i] += 1
                budget -= 1
                gave = True
        if not gave:
            break
    return budget


def hard_first(c: Sequence[int], cap: Sequence[int], B: int) -> List[int]:
    N = len(c)
    if B > sum(cap):
        raise ValueError("infeasible")
    delta = [0] * N
    left = deal([i for i in range(N) if c[i] == 0], cap, delta, B)
    left = deal([i for i in range(N) if c[i] != 0], cap, delta, left)
    assert left == 0
    return delta
