"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test compares the oracle with something that is NOT the oracle's own formula:
library Beta functions, closed forms, Monte-Carlo, brute-force enumeration, a global
sort of all candidates, numbers printed in the paper.  A last group plants typical mistakes
in a copy of the literal formulas and checks that the pins catch them.
"""
from __future__ import annotations

import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy import special

from oracle import hora_oracle as orc
from oracle import literal

HERE = os.path.dirname(os.path.abspath(__file__))
rng0 = np.random.default_rng(1234)

REAL_AB = [(0.05, 0.05), (0.37, 5.2), (1.0, 1.0), (3.0, 7.0), (19.5, 0.8), (28.0, 20.0), (2.5, 2.5)]


# ------------------------------------------------------------------ gains (Eq. marginal)
def beta_ratio_gain(a, b, Delta):
    """B(a+1, b+Delta-1) / B(a, b) through a library log-Beta (Eq. marginal with l = Delta-1)."""
    return math.exp(special.betaln(a + 1.0, b + Delta - 1.0) - special.betaln(a, b))


def check_gain_pins(gain_fn, ab_list=REAL_AB, deltas=(1, 2, 3, 7, 31, 100, 256)):
    """gain_fn(a, b, Delta) -> float.  Raises AssertionError when a pin fails."""
    for a, b in ab_list:
        assert gain_fn(a, b, 1) == pytest.approx(a / (a + b), rel=1e-15)       # M(0): posterior mean
        prev = None
        for D in deltas:
            g = gain_fn(a, b, D)
            assert g == pytest.approx(beta_ratio_gain(a, b, D), rel=2e-11), (a, b, D)
            g1 = gain_fn(a, b, D + 1)
            assert g1 / g == pytest.approx((b + D - 1) / (a + b + D), rel=1e-14)   # Eq. appendix-ratio
            assert g1 < g                                                             # Eq. appendix-monotone
            if prev is not None:
                assert g < prev
            prev = g


def test_gain_one_pins():
    check_gain_pins(orc.gain_one)


def test_literal_marginals_pins():
    def fn(a, b, D):
        return float(literal.marginals(Fraction(a), Fraction(b), D)[D - 1])
    check_gain_pins(fn)


def test_gain_rows_match_single_gains_and_padding():
    N, ld, G0 = 37, 19, 8
    alpha = np.exp(rng0.uniform(np.log(0.05), np.log(20), N))
    beta = np.exp(rng0.uniform(np.log(0.05), np.log(20), N))
    c = rng0.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng0.integers(0, ld + 1, N).astype(np.int32)
    rows = orc.gains(alpha, beta, 1.0, 1.0, c, G0, cap, ld)
    for i in range(N):
        a, b = alpha[i] + c[i], beta[i] + G0 - c[i]
        for D in range(1, ld + 1):
            if D <= cap[i]:
                assert rows[i, D - 1] == pytest.approx(beta_ratio_gain(a, b, D), rel=2e-11)
            else:
                assert rows[i, D - 1] == 0.0
    # Delta = 1 is the posterior mean (alpha + c) / (alpha + beta + G0)
    m = cap > 0
    np.testing.assert_allclose(rows[m, 0], ((alpha + c) / (alpha + beta + G0))[m], rtol=1e-15)


def test_shared_prior_equals_per_prompt_prior():
    """Eq. posterior-learned collapses to the fixed prior at s = 2, p_hat = 1/2."""
    N, G0, ld = 23, 8, 12
    c = rng0.integers(0, G0 + 1, N).astype(np.int32)
    cap = np.full(N, ld, np.int32)
    s, p_hat = 2.0, 0.5
    alpha = np.full(N, s * p_hat)
    beta = np.full(N, s * (1 - p_hat))
    np.testing.assert_array_equal(orc.gains(alpha, beta, 9.0, 9.0, c, G0, cap, ld),
                                  orc.gains(None, None, 1.0, 1.0, c, G0, cap, ld))
    d1 = orc.greedy_exact(alpha, beta, 9.0, 9.0, c, G0, cap, 5 * N)[0]
    d2 = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, 5 * N)[0]
    np.testing.assert_array_equal(d1, d2)


# ------------------------------------------------------------------ utility (Eq. hit-utility)
@pytest.mark.parametrize("a,b", REAL_AB)
def test_utility_beta_ratio_and_telescoping(a, b):
    for D in (0, 1, 2, 5, 40, 256):
        u = orc.utility_one(a, b, D)
        closed = 1.0 - math.exp(special.betaln(a, b + D) - special.betaln(a, b))   # Eq. appendix-hit-closed-form
        assert u == pytest.approx(closed, rel=1e-9, abs=1e-12)
        tele = math.fsum(orc.gain_one(a, b, k) for k in range(1, D + 1))           # Eq. appendix-objective
        assert u == pytest.approx(tele, rel=1e-13, abs=1e-15)
        uf = float(literal.utility(Fraction(a), Fraction(b), D))
        assert u == pytest.approx(uf, rel=1e-15, abs=1e-18)


@pytest.mark.parametrize("a,b", REAL_AB)
def test_utility_from_the_marginal_itself(a, b):
    """The product inside U(Delta) is M(Delta - 1) (b + Delta - 1) / a (Eq. marginal, Eq. hit-utility), so
    U(Delta) = 1 - g(Delta) (b + Delta - 1) / a: exact in rationals, and to rounding in the oracle's floats."""
    fa, fb = Fraction(a), Fraction(b)
    for D in (1, 2, 3, 17, 100, 256):
        assert literal.utility(fa, fb, D) == 1 - literal.marginals(fa, fb, D)[D - 1] * (fb + D - 1) / fa
        assert orc.utility_one(a, b, D) == pytest.approx(1.0 - orc.gain_one(a, b, D) * (b + D - 1) / a, rel=1e-13, abs=1e-15)


def test_utility_uniform_prior_no_success_closed_form():
    """Beta(1,1), c = 0: a = 1, b = G0 + 1, U(Delta) = Delta / (Delta + G0 + 1)."""
    for G0 in (2, 4, 8):
        a, b = literal.posterior(1, 1, 0, G0)
        for D in range(0, 30):
            assert literal.utility(a, b, D) == Fraction(D, D + G0 + 1)
            assert orc.utility_one(float(a), float(b), D) == pytest.approx(D / (D + G0 + 1), rel=1e-15)


def test_utility_monte_carlo():
    """U(Delta) = E[1 - (1-P)^Delta] is the probability of at least one hit (Eq. hit-utility)."""
    rng = np.random.default_rng(7)
    n = 400_000
    for a, b, D in [(1.0, 9.0, 6), (3.0, 7.0, 3), (0.4, 2.2, 10), (9.0, 1.0, 2)]:
        P = rng.beta(a, b, n)
        hits = rng.random((n, D)) < P[:, None]
        freq = hits.any(axis=1).mean()
        u = orc.utility_one(a, b, D)
        sigma = math.sqrt(u * (1 - u) / n)
        assert abs(freq - u) < 4.5 * sigma + 1e-9
        # and the marginal gain is the probability that the Delta-th draw is the FIRST hit
        first = hits[:, -1] & ~hits[:, :-1].any(axis=1)
        g = orc.gain_one(a, b, D)
        assert abs(first.mean() - g) < 4.5 * math.sqrt(g * (1 - g) / n) + 1e-9


# ------------------------------------------------------------------ allocation (Prop. 1)
def brute_force_best(ab, cap, B):
    best = None
    for d in itertools.product(*[range(cp + 1) for cp in cap]):
        if sum(d) != B:
            continue
        val = literal.objective(ab, d)
        if best is None or val > best:
            best = val
    return best


def sorted_top_B(ab, cap, B):
    """Global top-B of all candidates under (gain desc, prompt index asc, Delta asc)."""
    cands = []
    for i, ((a, b), cp) in enumerate(zip(ab, cap)):
        for D, g in enumerate(literal.marginals(a, b, cp), start=1):
            cands.append((-g, i, D))
    cands.sort()
    d = [0] * len(ab)
    for _, i, D in cands[:B]:
        d[i] += 1
    # prefix closure: a prompt's chosen candidates are Delta = 1..d[i]
    for _, i, D in cands[:B]:
        assert D <= d[i]
    return d


def small_integer_cases():
    rng = np.random.default_rng(99)
    cases = []
    for _ in range(60):
        N = int(rng.integers(1, 5))
        G0 = int(rng.choice([2, 4, 8]))
        al, be = int(rng.integers(1, 3)), int(rng.integers(1, 3))
        c = rng.integers(0, G0 + 1, N)
        cap = rng.integers(0, 5, N)
        B = int(rng.integers(0, min(8, int(cap.sum())) + 1))
        cases.append((G0, al, be, [int(x) for x in c], [int(x) for x in cap], B))
    return cases


@pytest.mark.parametrize("case", small_integer_cases())
def test_greedy_is_optimal_and_tie_broken_small(case):
    G0, al, be, c, cap, B = case
    ab = [literal.posterior(al, be, ci, G0) for ci in c]
    d_lit = literal.greedy(ab, cap, B)
    assert sum(d_lit) == B and all(0 <= x <= cp for x, cp in zip(d_lit, cap))
    assert literal.objective(ab, d_lit) == brute_force_best(ab, cap, B)           # Proposition 1
    assert d_lit == sorted_top_B(ab, cap, B)                                       # tie-break reading
    N = len(c)
    d_c, G_c, (ln, ldn), obj = orc.greedy_exact(None, None, float(al), float(be), np.array(c, np.int32), G0,
                                                np.array(cap, np.int32), B)
    assert list(d_c) == d_lit
    assert list(G_c) == [G0 + x for x in d_lit]
    assert obj == pytest.approx(float(literal.objective(ab, d_lit)), rel=1e-15, abs=1e-18)
    if B > 0:
        lam = min(literal.marginals(a, b, d)[d - 1] for (a, b), d in zip(ab, d_lit) if d > 0)
        assert Fraction(ln, ldn) == lam
    # the long-double heap gives an allocation of the same (optimal) value
    d_r, _, lam_r, obj_r = orc.greedy_real(None, None, float(al), float(be), np.array(c, np.int32), G0,
                                           np.array(cap, np.int32), B)
    assert int(d_r.sum()) == B
    assert float(literal.objective(ab, [int(x) for x in d_r])) == pytest.approx(float(brute_force_best(ab, cap, B)), rel=1e-14)


@pytest.mark.parametrize("case", small_integer_cases()[:30])
def test_heap_greedy_in_python_integers_small(case):
    """literal.greedy_heap against the O(B*N) scan, the global sort (a different algorithm) and brute force."""
    G0, al, be, c, cap, B = case
    ab = [literal.posterior(al, be, ci, G0) for ci in c]
    d, lam = literal.greedy_heap(ab, cap, B)
    assert d == literal.greedy(ab, cap, B) == sorted_top_B(ab, cap, B)
    assert literal.objective(ab, d) == brute_force_best(ab, cap, B)
    if B > 0:
        assert lam == min(literal.marginals(a, b, x)[x - 1] for (a, b), x in zip(ab, d) if x > 0)


def test_heap_greedy_beyond_128_bits():
    """Strong integer priors (alpha, beta up to 64, G0 = 8, up to 300 extra rollouts): for the larger budgets the
    reduced fractions no longer fit the C oracle's 128-bit words (it says so), the Python-integer heap carries on.  Pins: the global sort under
    (gain desc, index asc, Delta asc), the exchange certificate (Eq. appendix-exchange-condition), and agreement
    with the C oracle on the budgets it can still do."""
    rng = np.random.default_rng(20)
    N, G0, ld = 40, 8, 300
    alpha = rng.integers(1, 65, N)
    beta = rng.integers(1, 65, N)
    c = rng.integers(0, G0 + 1, N)
    cap = [int(x) for x in rng.integers(0, ld + 1, N)]
    ab = [literal.posterior(int(al), int(be), int(ci), G0) for al, be, ci in zip(alpha, beta, c)]
    gf = lambda a, b, D: literal.marginals(a, b, D)[D - 1]
    overflowed = 0
    for B in (1, 50, 700, sum(cap) // 2, sum(cap) - 3):
        d, lam = literal.greedy_heap(ab, cap, B)
        assert sum(d) == B and all(0 <= x <= cp for x, cp in zip(d, cap))
        assert d == sorted_top_B(ab, cap, B)
        assert exchange_certificate(gf, ab, cap, d)
        assert lam == min(gf(a, b, x) for (a, b), x in zip(ab, d) if x > 0)
        try:
            d_c = orc.greedy_exact(alpha.astype(np.float64), beta.astype(np.float64), 1.0, 1.0, c.astype(np.int32), G0,
                                   np.array(cap, np.int32), B)[0]
            assert list(d_c) == d
        except orc.OracleError as e:
            assert e.code == orc.OVERFLOW
            overflowed += 1
    assert overflowed > 0                        # this case does leave the 128-bit range


def test_worked_example_fixture():
    G0, c, cap = 2, (0, 1, 2, 0), (3, 3, 3, 3)
    ab = [literal.posterior(1, 1, ci, G0) for ci in c]
    rows = [ln for ln in open(os.path.join(HERE, "golden", "worked_example_g0_2.txt")) if not ln.startswith("#")]
    assert len(rows) == 13
    for ln in rows:
        Bs, ds, os_ = [x.strip() for x in ln.split("|")]
        B, d, obj = int(Bs), [int(x) for x in ds.split()], Fraction(os_)
        assert d == sorted_top_B(ab, cap, B)
        assert obj == brute_force_best(ab, cap, B)
        dc = orc.greedy_exact(None, None, 1.0, 1.0, np.array(c, np.int32), G0, np.array(cap, np.int32), B)[0]
        assert list(dc) == d
    # the cross-class exact ties this example is built around
    m0 = literal.marginals(*ab[0], 3)
    m1 = literal.marginals(*ab[1], 3)
    m2 = literal.marginals(*ab[2], 3)
    assert m0[1] == m2[1] == Fraction(3, 20) and m0[2] == m1[2] == Fraction(1, 10)


def exchange_certificate(gain_fn, ab, cap, delta):
    """Eq. appendix-exchange-condition restricted to feasible moves."""
    taken = [gain_fn(a, b, d) for (a, b), d in zip(ab, delta) if d > 0]
    nxt = [gain_fn(a, b, d + 1) for (a, b), d, cp in zip(ab, delta, cap) if d < cp]
    return (not taken) or (not nxt) or min(taken) >= max(nxt)


def test_medium_integer_case_invariants_and_literal_agreement():
    rng = np.random.default_rng(5)
    N, G0 = 200, 4
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, 20, N).astype(np.int32)
    ab = [literal.posterior(1, 1, int(ci), G0) for ci in c]
    gf = lambda a, b, D: literal.marginals(a, b, D)[D - 1]
    total = int(cap.sum())
    prev = None
    for B in [0, 1, 2, 137, 138, 139, total // 2, total - 1, total]:
        d, G, _, obj = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, B)
        assert int(d.sum()) == B and (d >= 0).all() and (d <= cap).all()
        assert list(d) == literal.greedy(ab, [int(x) for x in cap], B)
        assert exchange_certificate(gf, ab, cap, [int(x) for x in d])
        np.testing.assert_array_equal(G, G0 + d)
        if prev is not None and prev[0] + 1 == B:      # nestedness: one more unit changes one entry by +1
            diff = d.astype(np.int64) - prev[1]
            assert diff.min() == 0 and diff.sum() == 1
        prev = (B, d.astype(np.int64))
    assert list(orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, total)[0]) == list(cap)
    with pytest.raises(orc.OracleError) as e:
        orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, total + 1)
    assert e.value.code == orc.INFEASIBLE
    with pytest.raises(orc.OracleError) as e:
        orc.greedy_exact(None, None, 1.5, 1.0, c, G0, cap, 3)
    assert e.value.code == orc.NOT_INTEGER


def test_real_prior_heap_matches_literal_fractions():
    rng = np.random.default_rng(11)
    N, G0 = 60, 8
    alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, 40, N).astype(np.int32)
    ab = [literal.posterior(Fraction(float(x)), Fraction(float(y)), int(ci), G0) for x, y, ci in zip(alpha, beta, c)]
    for B in (0, 1, 97, 600, int(cap.sum())):
        d, G, lam, obj = orc.greedy_real(alpha, beta, 1.0, 1.0, c, G0, cap, B)
        dl = literal.greedy(ab, [int(x) for x in cap], B)
        assert list(d) == dl          # random real priors: no ties, so the allocation is unique
        assert obj == pytest.approx(float(literal.objective(ab, dl)), rel=1e-15)
        if B:
            lam_l = min(literal.marginals(a, b, x)[x - 1] for (a, b), x in zip(ab, dl) if x > 0)
            assert lam == pytest.approx(float(lam_l), rel=1e-17)


def test_budget_share_matches_paper_statistic():
    """Soft pin: Sec. 4.1 reports 15 % of prompts (c=0) -> 58 % of the Phase-B budget and 51 % (c=8) -> 12 %.

    The split of the remaining 34 % over c = 1..7 is not printed; it is spread evenly here, so
    only agreement within a few points is meaningful."""
    vals = {}
    for ln in open(os.path.join(HERE, "golden", "fig3_budget_share.txt")):
        if ln.startswith("#") or not ln.strip():
            continue
        k, frac, share = ln.split()
        vals[k] = (float(frac), float(share))
    G0, shard, B = 8, 15, 15 * 24
    pmf = np.array([vals["c=0"][0]] + [(1 - vals["c=0"][0] - vals["c=8"][0]) / 7] * 7 + [vals["c=8"][0]])
    rng = np.random.default_rng(2024)
    from oracle import share as share_orc
    got = np.zeros(G0 + 1)
    cnt = np.zeros(G0 + 1)
    cap = np.full(shard, B, np.int32)
    for _ in range(196 * 4):
        c = rng.choice(G0 + 1, size=shard, p=pmf).astype(np.int32)
        d = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, B)[0]
        prompts, budget = share_orc.allocation_share(c, d, G0)
        assert sum(prompts) == shard and sum(budget) == B
        got += budget
        cnt += prompts
    share = got / got.sum()
    assert abs(share[0] - vals["c=0"][1]) < 0.04
    assert abs(share[8] - vals["c=8"][1]) < 0.04
    # a saturated prompt still gets a little budget, a hopeless one gets the most per prompt
    assert share[8] > 0.05 and got[0] / cnt[0] > 5 * got[8] / cnt[8]


def test_posterior_avoids_plugin_degeneracy():
    """App. 'Degeneracy of plug-in hit utility': with c = 0 the plug-in gain is 0 for every Delta,
    the posterior gain is not; under the posterior a c = 0 prompt receives rollouts."""
    G0 = 8
    c = np.array([0, 4, 8, 2], np.int32)
    cap = np.full(4, 50, np.int32)
    d = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, 40)[0]
    assert d[0] > 0 and d[0] == d.max()
    plug = [(ci / G0) * (1 - ci / G0) ** l for ci in c for l in range(3)]
    assert plug[0] == plug[1] == plug[2] == 0.0
    assert orc.gain_one(1.0, 9.0, 1) == pytest.approx(0.1)


# ------------------------------------------------------------------ advantages
def ragged_groups(rng, n_groups, max_size, values):
    sizes = rng.integers(1, max_size + 1, n_groups)
    off = np.zeros(n_groups + 1, np.int64)
    np.cumsum(sizes, out=off[1:])
    r = rng.choice(values, int(off[-1])).astype(np.float32)
    return r, off


@pytest.mark.parametrize("ddof", [0, 1])
def test_grpo_closed_form_binary_groups(ddof):
    eps = 1e-6
    for G in (2, 3, 8, 33, 264):
        for k in range(0, G + 1):
            r = np.array([1.0] * k + [0.0] * (G - k), np.float32)
            off = np.array([0, G], np.int64)
            adv = orc.group_advantage(r, off, orc.GRPO, eps, ddof)
            mean = k / G
            var = k * (G - k) / (G * G) if ddof == 0 else k * (G - k) / (G * (G - 1))
            exp = (r.astype(np.float64) - mean) / (math.sqrt(var) + eps)
            np.testing.assert_allclose(adv, exp.astype(np.float32), rtol=1e-6, atol=1e-7)
            if k in (0, G):
                assert not adv.any()                 # zero-variance group: no signal (Sec. 3.1)


def test_grpo_against_numpy_std_and_invariants():
    rng = np.random.default_rng(3)
    r, off = ragged_groups(rng, 300, 40, [0.0, 0.5, 1.0])
    for ddof in (0, 1):
        adv = orc.group_advantage(r, off, orc.GRPO, 0.0, ddof)
        for g in range(300):
            seg = r[off[g]:off[g + 1]].astype(np.float64)
            n = len(seg)
            sd = seg.std(ddof=ddof) if n - ddof > 0 else 0.0
            exp = (seg - seg.mean()) / sd if sd > 0 else np.zeros(n)
            np.testing.assert_allclose(adv[off[g]:off[g + 1]], exp, rtol=1e-6, atol=1e-6)
            a = adv[off[g]:off[g + 1]].astype(np.float64)
            assert abs(a.sum()) < 1e-4
            if sd > 0:
                assert (a * a).sum() == pytest.approx(n - ddof, rel=1e-5)


def test_rloo_identities():
    rng = np.random.default_rng(4)
    r, off = ragged_groups(rng, 300, 40, [0.0, 1.0])
    adv = orc.group_advantage(r, off, orc.RLOO, 0.0, 0)
    for g in range(300):
        seg = r[off[g]:off[g + 1]].astype(np.float64)
        n = len(seg)
        if n == 1:
            assert adv[off[g]] == 0.0
            continue
        exp = np.array([seg[j] - np.delete(seg, j).mean() for j in range(n)])
        np.testing.assert_allclose(adv[off[g]:off[g + 1]], exp, atol=1e-6)
        np.testing.assert_allclose(adv[off[g]:off[g + 1]], n / (n - 1) * (seg - seg.mean()), atol=1e-6)
        assert abs(adv[off[g]:off[g + 1]].astype(np.float64).sum()) < 1e-4
        if seg.min() == seg.max():
            assert not adv[off[g]:off[g + 1]].any()


def test_empty_groups_are_skipped():
    r = np.array([1, 0, 1], np.float32)
    off = np.array([0, 0, 2, 2, 3], np.int64)
    adv = orc.group_advantage(r, off, orc.RLOO, 0.0, 0)
    np.testing.assert_array_equal(adv, np.array([1.0, -1.0, 0.0], np.float32))


def test_token_broadcast_is_repeat():
    rng = np.random.default_rng(6)
    R = 500
    adv = rng.standard_normal(R).astype(np.float32)
    lens = rng.integers(0, 30, R)
    off = np.zeros(R + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    out = orc.token_broadcast(adv, off)
    np.testing.assert_array_equal(out.view(np.uint32), np.repeat(adv, lens).view(np.uint32))


def test_rollout_weights_give_every_prompt_the_same_weight():
    """Sec. 3.2: with 1/G_i in place of 1/G each prompt has equal weight however many rollouts it got.  Summed
    over the tokens of a prompt, 1/(G_i |o|) gives exactly 1; the length-free form gives G_i/(G_i L) = 1/L per
    prompt when summed over rollouts."""
    rng = np.random.default_rng(12)
    sizes = rng.integers(1, 40, 200)
    goff = np.zeros(201, np.int64)
    np.cumsum(sizes, out=goff[1:])
    R = int(goff[-1])
    lens = rng.integers(1, 500, R)
    toff = np.zeros(R + 1, np.int64)
    np.cumsum(lens, out=toff[1:])
    w = orc.rollout_weights(goff, toff, 0).astype(np.float64)
    per_prompt = np.add.reduceat(w * lens, goff[:-1])
    np.testing.assert_allclose(per_prompt, 1.0, rtol=1e-6)
    w1 = orc.rollout_weights(goff, None, 1, 2048.0).astype(np.float64)
    np.testing.assert_allclose(np.add.reduceat(w1, goff[:-1]), 1.0 / 2048.0, rtol=1e-6)
    # direct form on one group
    np.testing.assert_allclose(w[:sizes[0]], 1.0 / (sizes[0] * lens[:sizes[0]]), rtol=1e-7)
    lens0 = lens.copy()
    lens0[3] = 0
    toff0 = np.zeros(R + 1, np.int64)
    np.cumsum(lens0, out=toff0[1:])
    assert orc.rollout_weights(goff, toff0, 0)[3] == 0.0


def test_learned_prior_front_end_pins():
    from oracle import prior
    # s = 2, p_hat = 1/2 is the uniform Beta(1,1) prior (stated below Eq. posterior-learned)
    a, b = prior.learned_prior([0.5], None, 2.0)
    assert a[0] == 1.0 and b[0] == 1.0
    # softplus and the clamp to [0.25, 16]
    a, b = prior.learned_prior([0.25, 0.25, 0.25], [-50.0, 0.0, 50.0])
    np.testing.assert_allclose(a + b, [0.25, math.log(2.0), 16.0], rtol=1e-15)
    np.testing.assert_allclose(a / (a + b), 0.25, rtol=1e-15)
    # one Phase-A draw: the Beta-Binomial probability of a success is the prior mean
    for p_hat in (0.1, 0.5, 0.83):
        for s in (0.3, 2.0, 11.0):
            assert prior.beta_binomial_nll([p_hat], [1], 1, None, s)[0] == pytest.approx(-math.log(p_hat), rel=1e-12)
            assert prior.beta_binomial_nll([p_hat], [0], 1, None, s)[0] == pytest.approx(-math.log(1 - p_hat), rel=1e-12)
    # the Beta-Binomial pmf sums to one over c
    G0 = 8
    for p_hat, s in ((0.3, 2.0), (0.9, 0.25), (0.5, 16.0)):
        nll = prior.beta_binomial_nll([p_hat] * (G0 + 1), list(range(G0 + 1)), G0, None, s)
        total = sum(math.comb(G0, c) * math.exp(-nll[c]) for c in range(G0 + 1))
        assert total == pytest.approx(1.0, rel=1e-12)
    # uniform prior: every count is equally likely, pmf = 1/(G0+1)
    nll = prior.beta_binomial_nll([0.5] * (G0 + 1), list(range(G0 + 1)), G0, None, 2.0)
    for c in range(G0 + 1):
        assert math.comb(G0, c) * math.exp(-nll[c]) == pytest.approx(1.0 / (G0 + 1), rel=1e-12)
    # large confidence: the posterior over the success rate collapses on p_hat and the loss tends to the binomial
    # negative log-likelihood -[c log p_hat + (G0 - c) log(1 - p_hat)], with an error that shrinks like 1/s
    for p_hat, c in ((0.3, 2), (0.71, 8), (0.5, 0)):
        binom = -(c * math.log(p_hat) + (G0 - c) * math.log(1 - p_hat))
        err = [abs(prior.beta_binomial_nll([p_hat], [c], G0, None, s)[0] - binom) for s in (1e3, 1e4, 1e5)]
        assert err[2] < 1e-3 * binom and err[0] > 5 * err[1] > 25 * err[2]
    # agreement with a library log-Beta
    a, b = prior.learned_prior([0.37], None, 5.0)
    assert prior.beta_binomial_nll([0.37], [3], 8, None, 5.0)[0] == pytest.approx(
        -(special.betaln(3 + a[0], 5 + b[0]) - special.betaln(a[0], b[0])), rel=1e-12)


# ------------------------------------------------------------------ planted mistakes are caught
def _mutant(kind):
    def marg(a, b, D):
        m = a / (a + b)
        for l in range(D - 1):
            if kind == "den_off_by_one":
                m = m * (b + l) / (a + b + l)
            elif kind == "num_uses_a":
                m = m * (a + l) / (a + b + l + 1)
            elif kind == "index_shift":
                m = m * (b + l + 1) / (a + b + l + 2)
            elif kind == "start_b":
                m = m * (b + l) / (a + b + l + 1) if l else b / (a + b)
        return m
    return marg


@pytest.mark.parametrize("kind", ["den_off_by_one", "num_uses_a", "index_shift", "start_b"])
def test_pins_catch_planted_gain_mistakes(kind):
    with pytest.raises(AssertionError):
        check_gain_pins(_mutant(kind))


def test_pins_catch_wrong_tie_break_and_wrong_argmax():
    G0, c, cap = 2, (0, 1, 2, 0), [3, 3, 3, 3]
    ab = [literal.posterior(1, 1, ci, G0) for ci in c]

    def greedy_highest_index(ab, cap, B):             # planted: ties to the HIGHEST index
        d = [0] * len(ab)
        cur = [a / (a + b) for a, b in ab]
        for _ in range(B):
            best = max((i for i in range(len(ab)) if d[i] < cap[i]), key=lambda i: (cur[i], i))
            a, b = ab[best]
            cur[best] = cur[best] * (b + d[best]) / (a + b + d[best] + 1)
            d[best] += 1
        return d

    assert any(greedy_highest_index(ab, cap, B) != sorted_top_B(ab, cap, B) for B in range(13))

    def greedy_by_mean(ab, cap, B):                   # planted: rank by posterior mean only
        d = [0] * len(ab)
        for _ in range(B):
            best = max((i for i in range(len(ab)) if d[i] < cap[i]), key=lambda i: (ab[i][0] / sum(ab[i]), -i))
            d[best] += 1
        return d

    assert any(literal.objective(ab, greedy_by_mean(ab, cap, B)) < brute_force_best(ab, cap, B) for B in range(13))


def test_pass_at_k_estimator_pins():
    """Eq. pass-k: pinned by special cases, by brute force over K-subsets, and by unbiasedness."""
    import itertools
    from oracle import passk
    n = 7
    for c in range(n + 1):
        assert passk.pass_at_k_one(n, c, 1) == Fraction(c, n)            # K = 1: the plain success rate
        assert passk.pass_at_k_one(n, c, n) == (1 if c > 0 else 0)        # K = n: any correct sample at all
        assert passk.pass_at_k_one(n, c, 0) == 0
        for K in range(1, n + 1):
            # brute force: fraction of K-subsets of the n samples that contain a correct one
            marks = [1] * c + [0] * (n - c)
            subsets = list(itertools.combinations(range(n), K))
            hit = sum(1 for sub in subsets if any(marks[i] for i in sub))
            assert passk.pass_at_k_one(n, c, K) == Fraction(hit, len(subsets))
    for K in range(1, n + 1):
        assert passk.pass_at_k_one(n, 0, K) == 0 and passk.pass_at_k_one(n, n, K) == 1
    # unbiased: averaged over c ~ Binomial(n, p) it equals 1 - (1-p)^K exactly
    p = Fraction(3, 10)
    for K in (1, 2, 5, 7):
        mean = sum(Fraction(math.comb(n, c)) * p**c * (1 - p)**(n - c) * passk.pass_at_k_one(n, c, K) for c in range(n + 1))
        assert mean == 1 - (1 - p)**K
    assert passk.pass_at_k([0, 7, 3], 7, [1, 7]) == [float(Fraction(10, 21)), float(Fraction(2, 3))]


def test_allocation_share_statistic_pins():
    """Fig. 3 statistic: hand example, and agreement with numpy's bincount (an independent routine)."""
    from oracle import share as share_orc
    prompts, budget = share_orc.allocation_share([0, 2, 2, 1, 0], [5, 1, 0, 3, 7], 2)
    assert prompts == [2, 1, 2] and budget == [12, 3, 1]
    rng = np.random.default_rng(8)
    c = rng.integers(0, 9, 5000)
    d = rng.integers(0, 100, 5000)
    prompts, budget = share_orc.allocation_share(c, d, 8)
    assert prompts == np.bincount(c, minlength=9).tolist()
    assert budget == np.bincount(c, weights=d, minlength=9).astype(np.int64).tolist()
    with pytest.raises(ValueError):
        share_orc.allocation_share([3], [1], 2)


# ------------------------------------------------------------------ hard-first heuristic (Sec. 4.2)
def test_hard_first_pins():
    """The comparison allocator of Sec. 4.2 under the even-split reading: a hand example, the invariants of an even
    split, the closed form of the water level, and the fall-through cases."""
    from oracle import hard_first as hf
    # hand example: prompts 0, 2, 5 have c = 0; caps 3, 9, 1, 9, 9, 9; 6 rollouts: rounds (0,2,5), (0,5), (0) -> 3, 1, 2
    c = [0, 1, 0, 4, 2, 0]
    cap = [3, 9, 1, 9, 9, 9]
    assert hf.hard_first(c, cap, 6) == [3, 0, 1, 0, 0, 2]
    assert hf.hard_first(c, cap, 7) == [3, 0, 1, 0, 0, 3]
    # the c = 0 prompts hold 3 + 1 + 9 = 13; the 14th and 15th rollout fall through to prompts 1 and 3
    assert hf.hard_first(c, cap, 13) == [3, 0, 1, 0, 0, 9]
    assert hf.hard_first(c, cap, 15) == [3, 1, 1, 1, 0, 9]
    # no c = 0 prompt at all: the uniform split, remainder to the lowest indices
    assert hf.hard_first([1, 2, 3, 1], [9, 9, 9, 9], 10) == [3, 3, 2, 2]
    with pytest.raises(ValueError):
        hf.hard_first(c, cap, sum(cap) + 1)
    rng = np.random.default_rng(42)
    for _ in range(200):
        N = int(rng.integers(1, 30))
        G0 = int(rng.integers(1, 6))
        cc = [int(x) for x in rng.integers(0, G0 + 1, N)]
        cp = [int(x) for x in rng.integers(0, 12, N)]
        B = int(rng.integers(0, sum(cp) + 1))
        d = hf.hard_first(cc, cp, B)
        assert sum(d) == B and all(0 <= x <= y for x, y in zip(d, cp))
        hard = [i for i in range(N) if cc[i] == 0]
        rest = [i for i in range(N) if cc[i] != 0]
        hard_room = sum(cp[i] for i in hard)
        if B <= hard_room:
            assert all(d[i] == 0 for i in rest)                       # only c = 0 prompts receive budget
            tier, Bt = hard, B
        else:
            assert all(d[i] == cp[i] for i in hard)                   # they are full before anyone else gets any
            tier, Bt = rest, B - hard_room
        # water level: the largest L with sum_i min(cap_i, L) <= Bt; everyone sits at min(cap, L) or one above,
        # and the ones above are the lowest-index prompts with room
        L = max(l for l in range(0, 13) if sum(min(cp[i], l) for i in tier) <= Bt)
        R = Bt - sum(min(cp[i], L) for i in tier)
        extra = [i for i in tier if cp[i] > L][:R]
        assert len(extra) == R
        for i in tier:
            assert d[i] == min(cp[i], L) + (1 if i in extra else 0)

