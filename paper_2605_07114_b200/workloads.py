"""Seeded synthetic inputs for the HORA rollout-allocation hot path.

This module only DRAWS inputs (priors, true success rates, caps, Phase-A counts,
Bernoulli rewards, response lengths).  It contains none of the method's arithmetic
(no posterior, no gains, no allocation, no advantages), so both the CUDA path and
the CPU oracle can be fed from it without sharing any of the computation under test.

The five named workloads stand in for the paper's training batches (math prompts
rolled out by a language model), whose data and weights are not needed here: the hot
path only consumes counts, priors, caps, rewards and lengths.  Shapes:

=====  =========  ==  ============================  =================  ===============  =====
name   N          G0  prior                         B                  cap / ld         adv
=====  =========  ==  ============================  =================  ===============  =====
cfg1   512        4   Beta(1,1), exact integers     12*N               60               GRPO
cfg2   8192       8   alpha,beta ~ LogU[0.1,10]     24*N               248              RLOO
cfg3   16384      4   Beta(1,1), exact integers     12*N               124              GRPO + tokens
cfg4   2**20      8   alpha,beta ~ LogU[0.05,20]    24*N               256              GRPO
cfg5   2**22      2   Beta(1,1), exact integers     3*N + 12345        U{0..64}, ld 64  RLOO
=====  =========  ==  ============================  =================  ===============  =====

Draw order per workload (fixed): priors -> p_i -> cap_i from ``numpy.random.Generator(PCG64(seed))``;
rewards and response lengths come from a counter-based 64-bit hash of (seed, prompt, slot), so
the reward of slot j of prompt i is defined for every j independently of any allocation, and the
Phase-A count c_i is the number of successes among slots j < G0 (so the first G0 rewards of a
group always sum to c_i, as Phase-A rollouts are pooled into the final group).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 output function (Steele, Lea, Flood 2014), vectorised on uint64."""
    x = np.asarray(x, dtype=np.uint64)
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        x = x ^ (x >> np.uint64(31))
    return x


def u64hash(seed: int, i: np.ndarray, j: np.ndarray) -> np.ndarray:
    """Well-mixed 64-bit hash of (seed, prompt index i, slot index j)."""
    i = np.asarray(i, dtype=np.uint64)
    j = np.asarray(j, dtype=np.uint64)
    with np.errstate(over="ignore"):
        s = _mix64(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + np.uint64(0x9E3779B97F4A7C15))
        h = _mix64(s ^ (i * np.uint64(0xD1B54A32D192ED03) + np.uint64(0x9E3779B97F4A7C15)))
        h = _mix64(h + j * np.uint64(0x9E3779B97F4A7C15) + np.uint64(1))
    return h


def _u01(h: np.ndarray) -> np.ndarray:
    """Top 53 bits of a hash as a float64 in [0, 1)."""
    return (h >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


GRPO = 0
RLOO = 1


@dataclass
class Workload:
    name: str
    seed: int
    N: int
    G0: int
    ld: int
    B: int
    alpha0: float
    beta0: float
    alpha: Optional[np.ndarray]      # float64[N] or None (shared prior alpha0/beta0)
    beta: Optional[np.ndarray]
    p: np.ndarray                    # float64[N] true success probabilities
    cap: np.ndarray                  # int32[N]
    c: np.ndarray                    # int32[N] Phase-A success counts
    adv_mode: int                    # GRPO or RLOO
    eps: float
    ddof: int
    exact_int: bool                  # integer-valued priors: ties are exact rational ties
    with_tokens: bool = False
    len_lo: int = 32
    len_hi: int = 2048
    notes: str = ""
    extra: dict = field(default_factory=dict)

    # ---- rewards / lengths (depend on a given allocation only through the group sizes) ----
    def group_offsets(self, delta: np.ndarray) -> np.ndarray:
        G = self.G0 + np.asarray(delta, dtype=np.int64)
        off = np.zeros(self.N + 1, dtype=np.int64)
        np.cumsum(G, out=off[1:])
        return off

    def _slots(self, off: np.ndarray):
        total = int(off[-1])
        G = np.diff(off)
        row = np.repeat(np.arange(self.N, dtype=np.int64), G)
        slot = np.arange(total, dtype=np.int64) - off[row]
        return row, slot

    def rewards(self, off: np.ndarray) -> np.ndarray:
        """Packed fp32 binary rewards for groups laid out by ``off`` (pre-rollouts first)."""
        row, slot = self._slots(off)
        u = _u01(u64hash(self.seed, row, slot))
        return (u < self.p[row]).astype(np.float32)

    def lengths(self, n_rollouts: int) -> np.ndarray:
        """Response lengths, Uniform{len_lo..len_hi}, one per packed rollout."""
        r = np.arange(n_rollouts, dtype=np.int64)
        h = u64hash(self.seed ^ 0x5EED1E45, r, np.zeros_like(r))
        span = np.uint64(self.len_hi - self.len_lo + 1)
        return (np.int64(self.len_lo) + (h % span).astype(np.int64)).astype(np.int32)

    def token_offsets(self, n_rollouts: int) -> np.ndarray:
        off = np.zeros(n_rollouts + 1, dtype=np.int64)
        np.cumsum(self.lengths(n_rollouts).astype(np.int64), out=off[1:])
        return off


def _phase_a_counts(seed: int, p: np.ndarray, G0: int) -> np.ndarray:
    N = p.shape[0]
    c = np.zeros(N, dtype=np.int32)
    idx = np.arange(N, dtype=np.int64)
    for j in range(G0):
        u = _u01(u64hash(seed, idx, np.full(N, j, dtype=np.int64)))
        c += (u < p).astype(np.int32)
    return c


def _mixture_p(rng: np.random.Generator, N: int) -> np.ndarray:
    """30 % p=0, 20 % p=1, 50 % Beta(1/2, 1/2): many saturated and many all-wrong prompts."""
    kind = rng.random(N)
    body = rng.beta(0.5, 0.5, N)
    p = np.where(kind < 0.3, 0.0, np.where(kind < 0.5, 1.0, body))
    return p.astype(np.float64)


def _log_uniform(rng: np.random.Generator, lo: float, hi: float, N: int) -> np.ndarray:
    return np.exp(rng.uniform(np.log(lo), np.log(hi), N)).astype(np.float64)


_SPECS = {
    #        N        G0  seed  per-prompt extra budget
    "cfg1": (512,     4,  0),
    "cfg2": (8192,    8,  1),
    "cfg3": (16384,   4,  2),
    "cfg4": (1 << 20, 8,  3),
    "cfg5": (1 << 22, 2,  4),
}


def make(name: str, N: Optional[int] = None, seed: Optional[int] = None) -> Workload:
    """Build workload ``name`` ("cfg1".."cfg5"); ``N`` rescales it (budget scales with N)."""
    if name not in _SPECS:
        raise KeyError(f"unknown workload {name!r}")
    N0, G0, seed0 = _SPECS[name]
    N = N0 if N is None else int(N)
    seed = seed0 if seed is None else int(seed)
    rng = np.random.Generator(np.random.PCG64(seed))
    alpha = beta = None
    alpha0 = beta0 = 1.0
    with_tokens = False
    if name in ("cfg1", "cfg3"):
        p = _mixture_p(rng, N)
        ld = 60 if name == "cfg1" else 124
        cap = np.full(N, ld, dtype=np.int32)
        B = 12 * N
        mode, eps, exact = GRPO, 1e-6, True
        with_tokens = name == "cfg3"
    elif name in ("cfg2", "cfg4"):
        lo, hi = (0.1, 10.0) if name == "cfg2" else (0.05, 20.0)
        alpha = _log_uniform(rng, lo, hi, N)
        beta = _log_uniform(rng, lo, hi, N)
        p = rng.beta(alpha, beta).astype(np.float64)
        ld = 248 if name == "cfg2" else 256
        cap = np.full(N, ld, dtype=np.int32)
        B = 24 * N
        mode, eps, exact = (RLOO, 0.0, False) if name == "cfg2" else (GRPO, 1e-6, False)
    else:  # cfg5
        p = rng.random(N).astype(np.float64)
        ld = 64
        cap = rng.integers(0, 65, N, dtype=np.int32)
        B = 3 * N + (12345 if N >= 4096 else 5)
        mode, eps, exact = RLOO, 0.0, True
    c = _phase_a_counts(seed, p, G0)
    total_cap = int(cap.astype(np.int64).sum())
    if B > total_cap:       # only reachable for tiny rescaled variants
        B = total_cap
    return Workload(name=name, seed=seed, N=N, G0=G0, ld=ld, B=int(B), alpha0=alpha0, beta0=beta0,
                    alpha=alpha, beta=beta, p=p, cap=cap, c=c, adv_mode=mode, eps=eps, ddof=0,
                    exact_int=exact, with_tokens=with_tokens)
