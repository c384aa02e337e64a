"""Learned-prior front end, plain Python/numpy in fp64.  TEST INFRASTRUCTURE ONLY.

Appendix "Prior-design predictor details": Eq. posterior-learned with the confidence s parametrised through a
softplus and clamped to [0.25, 16] (fixed s = 2 for the single-head variants), and the per-prompt Beta-Binomial
negative log-likelihood.  Pinned in tests/test_oracle_pins.py by the s = 2, p_hat = 1/2 collapse to the uniform
prior, by closed forms (G0 = 1), by normalisation over c, and by the large-s limit (the binomial NLL, approached like 1/s)."""
from __future__ import annotations

import math

import numpy as np

S_MIN, S_MAX = 0.25, 16.0


def confidence(s_raw, s_fixed, n):
    if s_raw is None:
        return np.full(n, float(s_fixed))
    sp = np.array([math.log1p(math.exp(x)) if x < 30 else x for x in np.asarray(s_raw, dtype=np.float64)])
    return np.clip(sp, S_MIN, S_MAX)


def learned_prior(p_hat, s_raw=None, s_fixed=2.0):
    """(alpha, beta) of the prior: s * p_hat, s * (1 - p_hat)."""
    p = np.asarray(p_hat, dtype=np.float64)
    s = confidence(s_raw, s_fixed, len(p))
    return s * p, s * (1.0 - p)


def _lbeta(x, y):
    return math.lgamma(x) + math.lgamma(y) - math.lgamma(x + y)


def beta_binomial_nll(p_hat, c, G0, s_raw=None, s_fixed=2.0):
    a, b = learned_prior(p_hat, s_raw, s_fixed)
    return np.array([-(_lbeta(ci + ai, G0 - ci + bi) - _lbeta(ai, bi)) for ai, bi, ci in zip(a, b, c)])
