"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element, on the
same seeded inputs.  Integer, index and byte results must be bit-exact; fp64 gains within 4*ld ulp of the
long-double oracle; real-prior allocations may differ only inside the 1e-12 band around the threshold;
fp32 advantages within 1e-5 absolute; broadcast output bitwise."""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import hora_oracle as orc  # noqa: E402
from paper_2605_07114_b200 import workloads as wl  # noqa: E402

U = 2.0 ** -53


def _util():
    import gpu_util
    return gpu_util


# ------------------------------------------------------------------------------------------ gains
def gains_tol(ld):
    return 4 * max(ld, 16) * U


@pytest.mark.parametrize("ld", [1, 2, 3, 31, 60, 64, 65, 124, 129, 248, 256, 300, 700])
@pytest.mark.parametrize("integer_prior", [False, True])
def test_gains_match_oracle(ld, integer_prior):
    gu = _util()
    rng = np.random.default_rng(ld * 2 + integer_prior)
    N, G0 = 333, 8
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    cap[:3] = [ld, 0, min(1, ld)]
    if integer_prior:
        alpha = beta = None
        a0, b0 = 1.0, 1.0
    else:
        alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
        beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
        alpha[0], beta[0] = 0.05, 0.05
        alpha[1], beta[1] = 20.0, 20.0
        a0 = b0 = 1.0
    got, status = gu.gpu_gains(alpha, beta, a0, b0, c, G0, cap, ld)
    exp = orc.gains(alpha, beta, a0, b0, c, G0, cap, ld)
    assert status == 0
    mask = np.arange(ld)[None, :] < cap[:, None]
    assert (got[~mask] == 0.0).all()                                # padding is exactly zero
    rel = np.abs(got[mask] - exp[mask]) / exp[mask]
    assert rel.max(initial=0.0) <= gains_tol(ld), rel.max()
    # rows strictly decrease (Eq. appendix-monotone) in the computed values too
    d = np.diff(got, axis=1)
    assert (d[mask[:, 1:]] < 0).all()


def test_gains_scalar_cap_and_equal_posteriors_give_equal_bits():
    gu = _util()
    N, G0, ld = 1000, 4, 124
    c = (np.arange(N) % (G0 + 1)).astype(np.int32)
    got, status = gu.gpu_gains(None, None, 1.0, 1.0, c, G0, None, ld, cap_scalar=100)
    assert status == 0
    assert (got[:, 100:] == 0).all() and (got[:, :100] > 0).all()
    for k in range(G0 + 1):
        rows = got[c == k]
        assert (rows.view(np.uint64) == rows[0].view(np.uint64)).all()


def test_gains_flags_invalid_rows():
    gu = _util()
    N, G0, ld = 64, 4, 32
    c = np.full(N, 2, np.int32)
    cap = np.full(N, ld, np.int32)
    alpha = np.ones(N)
    beta = np.ones(N)
    alpha[5] = -1.0
    beta[6] = np.nan
    c[7] = G0 + 1
    cap[8] = ld + 1
    alpha[9] = np.inf
    got, status = gu.gpu_gains(alpha, beta, 1.0, 1.0, c, G0, cap, ld)
    assert status == 2
    for i in (5, 6, 7, 8, 9):
        assert (got[i] == 0).all()
    assert (got[10] > 0).all()


# ------------------------------------------------------------------------------------- allocation
def run_and_compare(w, materialise=True):
    gu = _util()
    d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
    d, G, off, info = gu.gpu_allocate(w.alpha, w.beta, w.alpha0, w.beta0, w.c, w.G0, w.cap, w.ld, w.B,
                                      exact=w.exact_int, materialise=materialise)
    gu.assert_allocation_matches(w, d, G, off, info, d_o, lam_o, obj_o)
    if w.exact_int and w.alpha is None and not materialise and (w.G0 + 1) * w.ld <= 8192:
        assert info.first_pass_bits == -1           # one integer prior, no matrix: the rank-based route ran
    else:
        assert info.first_pass_bits == 23           # on these workloads the sampled window holds the threshold
    return d, G, off, info


@pytest.mark.parametrize("name,N", [("cfg1", None), ("cfg2", None), ("cfg3", None), ("cfg4", 1 << 15), ("cfg5", 1 << 16),
                                    ("cfg1", 37), ("cfg5", 1000), ("cfg4", 777), ("cfg2", 1)])
def test_allocation_matches_oracle(name, N):
    run_and_compare(wl.make(name, N))


@pytest.mark.parametrize("name,N", [("cfg1", None), ("cfg2", 2048), ("cfg5", 5000), ("cfg3", None), ("cfg4", 30000),
                                    ("cfg5", 1 << 17)])
def test_allocation_without_materialised_gains(name, N):
    run_and_compare(wl.make(name, N), materialise=False)


def test_every_budget_on_the_worked_example():
    """G0 = 2, c = (0,1,2,0), cap 3: B = 6, 7 hit the cross-class tie 3/20, B = 9, 10 the tie 1/10."""
    gu = _util()
    c = np.array([0, 1, 2, 0], np.int32)
    cap = np.full(4, 3, np.int32)
    for B in range(0, 13):
        d_o = orc.greedy_exact(None, None, 1.0, 1.0, c, 2, cap, B)[0]
        d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, 2, cap, 3, B, exact=True)
        assert info.status == 0
        np.testing.assert_array_equal(d, d_o)
        np.testing.assert_array_equal(G, 2 + d_o)


@pytest.mark.parametrize("G0", [2, 4, 8])
def test_budget_sweep_through_cross_class_ties(G0):
    """Many budgets on a small tie-heavy problem: every threshold, including exact cross-class ties,
    must reproduce exact greedy with lowest-index tie-breaking."""
    gu = _util()
    rng = np.random.default_rng(G0)
    N, ld = 97, 40
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    total = int(cap.sum())
    budgets = sorted(set([0, 1, 2, total - 1, total] + list(rng.integers(0, total + 1, 40))))
    for B in budgets:
        d_o = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, int(B))[0]
        d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, int(B), exact=True)
        assert info.status == 0, (B, info)
        np.testing.assert_array_equal(d, d_o, err_msg=f"B={B}")


def test_per_prompt_integer_priors_exact():
    gu = _util()
    rng = np.random.default_rng(77)
    N, G0, ld = 500, 4, 30
    alpha = rng.integers(1, 4, N).astype(np.float64)
    beta = rng.integers(1, 4, N).astype(np.float64)
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    for B in (1, 100, 2500, int(cap.sum()) // 2):
        d_o = orc.greedy_exact(alpha, beta, 1.0, 1.0, c, G0, cap, B)[0]
        d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, B, exact=True)
        assert info.status == 0
        np.testing.assert_array_equal(d, d_o)


def _exact_oracle_any_width(alpha, beta, a0, b0, c, G0, cap, B):
    """Exact greedy: the C oracle while its 128-bit reduced fractions suffice, else the Python-integer heap."""
    from fractions import Fraction
    from oracle import literal
    try:
        return orc.greedy_exact(alpha, beta, a0, b0, c, G0, cap, B)[0]
    except orc.OracleError as e:
        assert e.code == orc.OVERFLOW
    al = np.full(len(c), a0) if alpha is None else alpha
    be = np.full(len(c), b0) if beta is None else beta
    ab = [literal.posterior(int(x), int(y), int(ci), G0) for x, y, ci in zip(al, be, c)]
    return np.array(literal.greedy_heap(ab, [int(x) for x in cap], int(B))[0], np.int32)


@pytest.mark.parametrize("prior_max,G0,ld", [(20, 8, 256), (40, 8, 256), (16, 16, 256), (3, 4, 1000)])
def test_strong_integer_priors_exact(prior_max, G0, ld):
    """Integer priors well beyond the uniform one: the exact numerators and denominators of the near-threshold
    candidates outgrow 128 bits (a = 28 at Delta = 250 needs about 240), and the result must still be exact greedy."""
    gu = _util()
    rng = np.random.default_rng(prior_max * 100 + G0)
    N = 400
    alpha = rng.integers(1, prior_max + 1, N).astype(np.float64)
    beta = rng.integers(1, prior_max + 1, N).astype(np.float64)
    alpha[::3], beta[::3] = alpha[0], beta[0]            # repeated priors: exact ties between prompts
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    c[::3] = c[0]
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    total = int(cap.sum())
    for B in (1, N, total // 4, total // 2, total - 5):
        d_o = _exact_oracle_any_width(alpha, beta, 1.0, 1.0, c, G0, cap, B)
        d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, B, exact=True)
        assert info.status == 0, (B, info)
        np.testing.assert_array_equal(d, d_o, err_msg=f"B={B}")


def test_threshold_on_candidates_wider_than_128_bits():
    """G0 = 16 with the uniform prior (the paper's G0 ablation, Table allocator-g0): a prompt with every Phase-A
    rollout correct has a = 17, b = 1, and g(Delta) = 17 * 17! / (Delta)_18, whose denominator passes 2^128 near
    Delta = 140.  Budgets that put the threshold on such candidates, alone and tied across classes, must
    reproduce exact greedy with the lowest-index tie-break."""
    gu = _util()
    from fractions import Fraction
    from oracle import literal
    G0, ld, N = 16, 256, 300
    rng = np.random.default_rng(16)
    c = np.where(rng.random(N) < 0.5, G0, rng.integers(0, G0 + 1, N)).astype(np.int32)
    cap = np.full(N, ld, np.int32)
    # budgets whose threshold lies on a c = 16 candidate with Delta >= 150: take every candidate at least as good as
    # g_{c=16}(Delta*), minus a few so that the last ones are handed out by index
    ab = [literal.posterior(1, 1, int(ci), G0) for ci in c]
    rows = {int(k): literal.marginals(*literal.posterior(1, 1, int(k), G0), ld) for k in set(c.tolist())}
    for D_star in (150, 201, 256):
        lam = rows[G0][D_star - 1]
        B = sum(sum(1 for g in rows[int(ci)] if g >= lam) for ci in c) - 7
        d_o, lam_o = literal.greedy_heap(ab, [ld] * N, B)
        unreduced = 1
        for k in range(18):
            unreduced *= D_star + k                   # (Delta)_18, the denominator as the GPU path forms it
        assert lam_o == lam and unreduced.bit_length() > 128
        d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, B, exact=True)
        assert info.status == 0
        np.testing.assert_array_equal(d, np.array(d_o, np.int32))
        assert info.lambda_ == pytest.approx(float(lam), rel=1e-12)
        d2, _, _, info2 = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, B, exact=True, materialise=False)
        assert info2.status == 0
        np.testing.assert_array_equal(d2, d)


def test_exact_range_is_reported_not_wrapped():
    """A posterior too strong for the 512-bit exact form (a about 5000 at Delta about 500) must give EXACT_RANGE and
    zeroed outputs, never a wrong allocation."""
    gu = _util()
    N, G0, ld = 64, 4, 600
    alpha = np.full(N, 5000.0)
    beta = np.full(N, 3.0)
    c = np.full(N, 2, np.int32)
    cap = np.full(N, ld, np.int32)
    d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, 500 * N + 3, exact=True)
    assert info.status == 5 and not d.any() and not G.any()


def test_single_class_is_pure_index_tie_break():
    gu = _util()
    N, G0, ld = 1000, 4, 8
    c = np.zeros(N, np.int32)
    cap = np.full(N, ld, np.int32)
    B = 3 * N + 123
    d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, B, exact=True)
    assert info.status == 0
    exp = np.full(N, 3, np.int32)
    exp[:123] = 4
    np.testing.assert_array_equal(d, exp)
    assert info.n_tied == N and info.n_tied_taken == 123 and info.n_above == 3 * N
    # the fp64 path ties on equal bit patterns and must give the same answer here
    d2, _, _, info2 = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, B, exact=False)
    np.testing.assert_array_equal(d2, exp)


def test_edge_budgets_and_caps():
    gu = _util()
    rng = np.random.default_rng(8)
    N, G0, ld = 301, 8, 17
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = np.zeros(N, np.int32)
    cap[::3] = rng.integers(0, ld + 1, len(cap[::3]))
    total = int(cap.sum())
    for exact in (True, False):
        d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, 0, exact=exact)
        assert info.status == 0 and not d.any() and (G == G0).all() and off[-1] == N * G0 and info.lambda_ == 0.0
        d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, total, exact=exact)
        assert info.status == 0
        np.testing.assert_array_equal(d, cap)
        d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, total + 1, exact=exact)
        assert info.status == 3 and not d.any() and not G.any() and not off.any()
    one = np.zeros(N, np.int32)
    one[200] = 5
    d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, one, ld, 4, exact=True)
    assert info.status == 0 and d[200] == 4 and d.sum() == 4


@pytest.mark.parametrize("materialise", [True, False])
@pytest.mark.parametrize("exact", [True, False])
def test_allocation_when_the_sampled_window_misses(exact, materialise):
    """The full-read pass refines 23 bits inside a window placed from a sample of every k-th row.  Here the
    sampled rows (index multiple of 5) are all hopeless prompts and the others all saturated ones, so the
    sample says nothing about the threshold and the window lands in the wrong place: the selection must
    fall back to plain 13-bit digits and still reproduce the oracle."""
    gu = _util()
    N, G0, ld = 20000, 8, 96                      # N > 4096 rows: every ceil(N / 4096) = 5th row is sampled
    idx = np.arange(N)
    c = np.where(idx % 5 == 0, 0, G0).astype(np.int32)
    cap = np.full(N, ld, np.int32)
    rng = np.random.default_rng(5)
    if exact:
        alpha = beta = np.ones(N)                    # per-prompt arrays: the key-based selection, not the rank route
    else:
        alpha = np.exp(rng.uniform(np.log(0.5), np.log(2.0), N))
        beta = np.exp(rng.uniform(np.log(0.5), np.log(2.0), N))
    for B in (1000, 7 * N, 40 * N):
        if exact:
            d_o, _, lam, obj = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, B)
        else:
            d_o, _, lam, obj = orc.greedy_real(alpha, beta, 1.0, 1.0, c, G0, cap, B)
        d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, B, exact=exact,
                                          materialise=materialise)
        assert info.status == 0
        assert info.first_pass_bits == 13            # the window did miss: this is the fallback being tested
        np.testing.assert_array_equal(d, d_o)
        assert abs(info.objective - obj) <= 1e-12 * obj


@pytest.mark.parametrize("materialise", [True, False])
@pytest.mark.parametrize("exact", [True, False])
def test_heavy_ties_take_the_digit_route_at_moderate_size(exact, materialise):
    """One posterior class, 2^17 prompts: the threshold is a value that 131072 candidates share, more than the
    candidate list holds, so the tail narrows the rows digit by digit — with the matrix given and with the
    matrix built inside the call.  The result is a pure index tie-break."""
    gu = _util()
    N, G0, ld = 1 << 17, 4, 24
    c = np.zeros(N, np.int32)
    cap = np.full(N, ld, np.int32)
    cap[::7] = 5                                     # some rows end before the threshold's column
    B = 9 * N + 4321
    d_o, _, lam, obj = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, B)
    ones = np.ones(N)                                # per-prompt arrays: the key-based selection, not the rank route
    d, G, off, info = gu.gpu_allocate(ones, ones, 1.0, 1.0, c, G0, cap, ld, B, exact=exact, materialise=materialise)
    assert info.status == 0 and info.first_pass_bits in (13, 23)
    assert info.n_tied > 65536                       # what forces the digit route
    np.testing.assert_array_equal(d, d_o)
    np.testing.assert_array_equal(off, np.concatenate(([0], np.cumsum(G0 + d_o.astype(np.int64)))))
    assert abs(info.objective - obj) <= 1e-12 * obj


@pytest.mark.parametrize("case", ["two_values", "zeros"])
def test_mass_ties_in_a_given_matrix_that_are_not_one_value(case):
    """The digit route has a shortcut for the case that every key carrying the resolved prefix is one value.  Here
    it must not fire: (two_values) 2^17 keys share 23 bits but are two values 2^-40 apart, the threshold being the
    larger; (zeros) the budget reaches into 2^18 zero gains, two a row.  Expected: the B largest candidates under
    (gain descending, prompt ascending, column ascending), by a global sort of the matrix."""
    from paper_2605_07114_b200 import hora
    N, G0, ld = 1 << 17, 2, 4
    rng = np.random.default_rng(17)
    k1 = 0.5
    k2 = float(np.float64(0.5) * (1.0 + 2.0 ** -40))
    second = np.where(rng.random(N) < 0.5, k1, k2)
    g = np.stack([np.full(N, 0.9), second, np.zeros(N), np.zeros(N)], axis=1)
    B = N + N // 4 if case == "two_values" else 2 * N + N // 2
    order = np.lexsort((np.tile(np.arange(ld), N), np.repeat(np.arange(N), ld), -g.ravel()))
    d_o = np.bincount(order[:B] // ld, minlength=N).astype(np.int32)
    al = hora.Allocator(N, ld, G0, exact_int=False)
    al.gains.copy_(torch.from_numpy(g).cuda())
    ones = gu_dev(np.ones(N))
    hora.hora_allocate(ones, ones, 1.0, 1.0, gu_dev(np.zeros(N, np.int32)), G0, None, ld, N, ld, al.gains, B, al.flags,
                       al.delta, al.G, al.group_offsets, al.info, al.workspace)
    torch.cuda.synchronize()
    info = al.read_info()
    assert info.status == 0
    assert info.n_tied == (int((second == k2).sum()) if case == "two_values" else 2 * N)
    assert info.lambda_ == (k2 if case == "two_values" else 0.0)
    np.testing.assert_array_equal(al.delta.cpu().numpy(), d_o)


def test_allocation_with_long_rows():
    """ld > 256: several items per row in the full-read pass, whose counts above the guess add up per row."""
    gu = _util()
    rng = np.random.default_rng(9)
    N, G0, ld = 3000, 4, 700
    alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    for B in (5000, 300000):
        d_o, _, lam, obj = orc.greedy_real(alpha, beta, 1.0, 1.0, c, G0, cap, B)
        d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, B, exact=False)
        assert info.status == 0
        np.testing.assert_array_equal(d, d_o)
        assert abs(info.lambda_ - lam) <= 1e-12 * lam


@pytest.mark.parametrize("seed", range(12))
def test_allocation_on_random_shapes(seed):
    """Random sizes, row lengths (odd ones too: no 16-byte loads), caps and budgets, real and integer priors,
    with the matrix given and built inside: Delta, G, offsets and the objective against the oracle."""
    gu = _util()
    rng = np.random.default_rng(1000 + seed)
    N = int(rng.integers(1, 6000))
    ld = int(rng.choice([1, 2, 7, 31, 64, 65, 100, 128, 129, 255, 256, 257, 300, 513]))
    G0 = int(rng.integers(1, 9))
    exact = bool(seed % 2)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    if seed % 3 == 0:
        cap[:] = ld
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    if exact:
        alpha = rng.integers(1, 4, N).astype(np.float64)
        beta = rng.integers(1, 4, N).astype(np.float64)
    else:
        alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
        beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    total = int(cap.sum())
    for B in sorted({0, 1, total // 3, total - 1 if total > 0 else 0, total}):
        if exact:
            d_o, _, lam, obj = orc.greedy_exact(alpha, beta, 1.0, 1.0, c, G0, cap, B)
        else:
            d_o, _, lam, obj = orc.greedy_real(alpha, beta, 1.0, 1.0, c, G0, cap, B)
        for materialise in (True, False):
            d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, B, exact=exact,
                                              materialise=materialise)
            assert info.status == 0, (N, ld, G0, B, materialise)
            np.testing.assert_array_equal(d, d_o)
            np.testing.assert_array_equal(G, G0 + d_o)
            np.testing.assert_array_equal(off, np.concatenate(([0], np.cumsum(G0 + d_o.astype(np.int64)))))
            assert abs(info.objective - obj) <= 1e-12 * max(abs(obj), 1e-300)


def test_allocation_status_codes():
    gu = _util()
    N, G0, ld = 100, 4, 16
    c = np.full(N, 1, np.int32)
    cap = np.full(N, ld, np.int32)
    alpha = np.ones(N)
    beta = np.ones(N)
    alpha[3] = 1.5
    d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, 50, exact=True)
    assert info.status == 4 and not d.any()
    alpha[3] = 2.0e6
    d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, 50, exact=True)
    assert info.status == 5 and not d.any()
    alpha[3] = -1.0
    d, G, off, info = gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, 50, exact=False)
    assert info.status == 2 and not d.any()


@pytest.mark.parametrize("ld,cap_value", [(256, 256), (256, 200), (96, 96), (40, 33), (64, 64), (64, 50)])
def test_allocation_validates_a_given_gains_matrix(ld, cap_value):
    """hora_allocate checks the matrix it is given: every row finite, non-negative and non-increasing up to its
    cap.  Equal neighbours are allowed; a disorder that shows only in the low 32 bits of two keys with equal
    high words, a NaN, an infinity, a negative value and a negative zero are not."""
    from paper_2605_07114_b200 import hora
    N, G0, B = 300, 4, 700
    rng = np.random.default_rng(ld + cap_value)
    alpha, beta = rng.uniform(0.5, 3.0, N), rng.uniform(0.5, 3.0, N)
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    al = hora.Allocator(N, ld, G0, exact_int=False)
    a_d, b_d, c_d = gu_dev(alpha), gu_dev(beta), gu_dev(c)
    hora.hora_gains(a_d, b_d, 1.0, 1.0, c_d, G0, None, cap_value, N, ld, al.gains)
    torch.cuda.synchronize()
    clean = al.gains.clone()

    def status_with(edit):
        al.gains.copy_(clean)
        edit(al.gains)
        hora.hora_allocate(a_d, b_d, 1.0, 1.0, c_d, G0, None, cap_value, N, ld, al.gains, B, al.flags, al.delta, al.G,
                           al.group_offsets, al.info, al.workspace)
        torch.cuda.synchronize()
        return al.read_info().status, al.delta.cpu().numpy()

    def bits(g):
        return g.view(torch.int64)

    st, d = status_with(lambda g: None)
    assert st == 0 and d.sum() == B
    j = cap_value // 2                                    # a column well inside every row
    # equal neighbours: still non-increasing
    def tie(g): g[7, j + 1] = g[7, j]
    st, d = status_with(tie)
    assert st == 0 and d.sum() == B
    # same high word, low word one step UP: increasing by one unit in the last place
    def lo_up(g): bits(g)[11, j + 1] = bits(g)[11, j] + 1
    assert status_with(lo_up)[0] == 2
    # plainly increasing, at a slice boundary of the full-read pass too
    def swap(g): g[13, j], g[13, j + 1] = g[13, j + 1].clone(), g[13, j].clone()
    assert status_with(swap)[0] == 2
    if cap_value > 66:
        def at_64(g): g[17, 64] = g[17, 62]
        assert status_with(at_64)[0] == 2
    for bad in (float("nan"), float("inf"), -1.0e-3, -0.0):
        def put(g, bad=bad): g[19, cap_value - 1] = bad
        st, d = status_with(put)
        assert st == 2 and not d.any(), bad
    def first_inf(g): g[23, 0] = float("inf")
    assert status_with(first_inf)[0] == 2


def test_allocate_stage_events_are_recorded_in_order():
    """hora_allocate_profile_stages: the seven events land on the call's stream in stage order, and switching
    the aid off stops the recording."""
    from paper_2605_07114_b200 import hora
    w = wl.make("cfg2", 2048)
    al = hora.Allocator(w.N, w.ld, w.G0, exact_int=False)
    args = (gu_dev(w.alpha), gu_dev(w.beta), 1.0, 1.0, gu_dev(w.c), gu_dev(w.cap), 0, w.B)
    al.run(*args)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(7)]
    for e in evs:
        e.record()
    torch.cuda.synchronize()
    hora.hora_allocate_profile_stages([e.cuda_event for e in evs])
    try:
        al.run(*args)
    finally:
        hora.hora_allocate_profile_stages(None)
    torch.cuda.synchronize()
    gaps = [evs[i].elapsed_time(evs[i + 1]) for i in range(6)]
    assert all(g >= 0.0 for g in gaps) and sum(gaps) > 0.0
    assert al.read_info().status == 0
    tail = torch.cuda.Event(enable_timing=True)
    tail.record()
    al.run(*args)                                         # recording is off: the old events keep their times
    torch.cuda.synchronize()
    assert evs[6].elapsed_time(tail) >= 0.0


def test_allocation_host_errors():
    from paper_2605_07114_b200 import hora
    N, ld = 10, 8
    c = torch.zeros(N, dtype=torch.int32, device="cuda")
    delta = torch.zeros(N, dtype=torch.int32, device="cuda")
    G = torch.zeros(N, dtype=torch.int32, device="cuda")
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(hora.HoraError) as e:
        hora.hora_allocate(None, None, 1.0, 1.0, c, 4, None, ld, N, ld, None, 5, 0, delta, G, None, None, ws)
    assert e.value.code == hora.ERR_WORKSPACE
    with pytest.raises(hora.HoraError) as e:
        hora.hora_allocate(None, None, 1.0, 1.0, c, 4, None, ld, N, ld, None, -5, 0, delta, G, None, None, ws)
    assert e.value.code == hora.ERR_INVALID_ARG


def test_allocation_is_reproducible():
    gu = _util()
    w = wl.make("cfg4", 4096)
    a = gu.gpu_allocate(w.alpha, w.beta, 1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B, exact=False)
    b = gu.gpu_allocate(w.alpha, w.beta, 1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B, exact=False)
    np.testing.assert_array_equal(a[0], b[0])
    assert np.float64(a[3].objective).view(np.uint64) == np.float64(b[3].objective).view(np.uint64)


def gu_dev(a):
    return _util().dev(a)


# ------------------------------------------------------------------------------------- advantages
def ragged(rng, n_groups, sizes, values):
    sizes = rng.choice(sizes, n_groups)
    off = np.zeros(n_groups + 1, np.int64)
    np.cumsum(sizes, out=off[1:])
    return rng.choice(values, int(off[-1])).astype(np.float32), off


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("ddof", [0, 1])
@pytest.mark.parametrize("eps", [0.0, 1e-6])
def test_group_advantage_matches_oracle(mode, ddof, eps):
    gu = _util()
    rng = np.random.default_rng(mode * 4 + ddof * 2 + (eps > 0))
    sizes = [0, 1, 2, 3, 8, 9, 31, 32, 33, 64, 100, 264, 288, 289, 500, 3000]
    for values in ([0.0, 1.0], [0.0, 0.5, 1.0], [1.0], [-3.25, 0.1, 7.0, 1e3]):
        r, off = ragged(rng, 700, sizes, values)
        got, status = gu.gpu_advantage(r, off, mode, np.float32(eps), ddof)
        exp = orc.group_advantage(r, off, mode, float(np.float32(eps)), ddof)
        assert status == 0
        tol = 1e-5 * max(1.0, float(np.abs(values).max()))
        np.testing.assert_allclose(got, exp, rtol=0, atol=tol)
        if len(values) == 1:
            assert not got.any()                                  # zero-variance groups give zero advantage


def test_group_advantage_on_workload_groups():
    gu = _util()
    for name, N in (("cfg1", None), ("cfg2", None), ("cfg5", 20000)):
        w = wl.make(name, N)
        d_o = gu.oracle_allocate(w)[0]
        off = w.group_offsets(d_o)
        r = w.rewards(off)
        got, status = gu.gpu_advantage(r, off, w.adv_mode, np.float32(w.eps), w.ddof)
        exp = orc.group_advantage(r, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
        assert status == 0
        np.testing.assert_allclose(got, exp, rtol=0, atol=1e-5)
        sums = np.add.reduceat(got.astype(np.float64), off[:-1])
        assert np.abs(sums).max() < 1e-3                          # advantages of a group sum to zero


@pytest.mark.parametrize("mis_in,mis_out", [(0, 0), (1, 0), (0, 3), (2, 2)])
def test_group_advantage_with_unaligned_buffers_stays_in_bounds(mis_in, mis_out):
    """Rewards and advantages that do not start on a 16-byte boundary (no vector path), and a guard band around
    the output: nothing before the first or after the last element is written."""
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(10 * mis_in + mis_out)
    r, off = ragged(rng, 3000, [0, 1, 5, 8, 31, 32, 33, 100, 264, 2000], [0.0, 1.0])
    total = int(off[-1])
    rbuf = torch.zeros(total + 8, dtype=torch.float32, device="cuda")
    obuf = torch.full((total + 16,), float("nan"), dtype=torch.float32, device="cuda")
    rin = rbuf[mis_in:mis_in + total]
    rin.copy_(torch.from_numpy(r))
    out = obuf[4 + mis_out:4 + mis_out + total]
    for mode in (0, 1):
        obuf.fill_(float("nan"))
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        hora.hora_group_advantage(rin, torch.from_numpy(off).cuda(), len(off) - 1, mode, 1e-6, 0, out, status)
        torch.cuda.synchronize()
        exp = orc.group_advantage(r, off, mode, float(np.float32(1e-6)), 0)
        assert int(status.item()) == 0
        np.testing.assert_allclose(out.cpu().numpy(), exp, rtol=0, atol=1e-5)
        assert torch.isnan(obuf[:4 + mis_out]).all() and torch.isnan(obuf[4 + mis_out + total:]).all()


def test_group_advantage_flags_decreasing_offsets():
    gu = _util()
    r = np.ones(10, np.float32)
    off = np.array([0, 5, 3, 10], np.int64)
    got, status = gu.gpu_advantage(r, off, 0, np.float32(0), 0)
    assert status == 2


# -------------------------------------------------------------------------------------- broadcast
@pytest.mark.parametrize("misalign", [0, 1, 3])
@pytest.mark.parametrize("kind", ["paper", "short", "zeros", "tiny_many", "one_long", "single_token"])
def test_token_broadcast_bitwise(kind, misalign):
    gu = _util()
    rng = np.random.default_rng(len(kind) + misalign)
    if kind == "paper":
        lens = rng.integers(32, 2049, 5000)
    elif kind == "short":
        lens = rng.integers(0, 9, 40000)
    elif kind == "zeros":
        lens = np.where(rng.random(30000) < 0.7, 0, rng.integers(1, 300, 30000))
    elif kind == "tiny_many":
        lens = np.concatenate([np.ones(5000, np.int64), np.zeros(4000, np.int64), rng.integers(0, 3, 200000),
                               rng.integers(1000, 5000, 50)])
    elif kind == "one_long":
        lens = np.array([0, 0, 1234567, 0])
    else:
        lens = np.array([1])
    R = len(lens)
    adv = rng.standard_normal(R).astype(np.float32)
    off = np.zeros(R + 1, np.int64)
    np.cumsum(lens, out=off[1:])
    got = gu.gpu_broadcast(adv, off, misalign=misalign)
    exp = orc.token_broadcast(adv, off)
    np.testing.assert_array_equal(got.view(np.uint32), exp.view(np.uint32))


def test_token_broadcast_on_cfg3_layout_scaled():
    gu = _util()
    w = wl.make("cfg3", 1024)
    d_o = gu.oracle_allocate(w)[0]
    off = w.group_offsets(d_o)
    r = w.rewards(off)
    adv = orc.group_advantage(r, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
    tok = w.token_offsets(len(r))
    got = gu.gpu_broadcast(adv, tok)
    np.testing.assert_array_equal(got.view(np.uint32), orc.token_broadcast(adv, tok).view(np.uint32))


# ---------------------------------------------------------------------------------------- weights
@pytest.mark.parametrize("mode", [0, 1])
def test_rollout_weights_bitwise(mode):
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(21 + mode)
    sizes = rng.choice([0, 1, 2, 8, 9, 31, 32, 33, 100, 264, 1000], 3000)
    goff = np.zeros(len(sizes) + 1, np.int64)
    np.cumsum(sizes, out=goff[1:])
    R = int(goff[-1])
    lens = rng.integers(0, 2049, R)
    toff = np.zeros(R + 1, np.int64)
    np.cumsum(lens, out=toff[1:])
    w = torch.full((R,), -1.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hora.hora_rollout_weights(torch.from_numpy(goff).cuda(), len(sizes), torch.from_numpy(toff).cuda(), mode, 2048.0, w,
                              status)
    torch.cuda.synchronize()
    exp = orc.rollout_weights(goff, toff, mode, 2048.0)
    assert int(status.item()) == 0
    assert np.array_equal(w.cpu().numpy().view(np.uint32), exp.view(np.uint32))
    # through the token broadcast: per-token weights of one prompt sum to 1 in the per-token mode
    if mode == 0:
        T = int(toff[-1])
        tw = torch.empty(T, dtype=torch.float32, device="cuda")
        hora.hora_token_broadcast(w, torch.from_numpy(toff).cuda(), R, T, tw)
        per_rollout = np.add.reduceat(tw.cpu().numpy().astype(np.float64), toff[:-1][lens > 0])
        g_of_r = np.repeat(np.arange(len(sizes)), sizes)[lens > 0]
        per_prompt = np.bincount(g_of_r, weights=per_rollout, minlength=len(sizes))
        full = np.array([sizes[g] > 0 and (lens[goff[g]:goff[g + 1]] > 0).all() for g in range(len(sizes))])
        np.testing.assert_allclose(per_prompt[full], 1.0, rtol=1e-5)


# ------------------------------------------------------------------------------------ learned prior
def test_learned_prior_and_nll_match_oracle():
    from oracle import prior
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(33)
    N, G0 = 5000, 8
    p_hat = rng.uniform(0.001, 0.999, N)
    s_raw = rng.uniform(-6, 20, N)
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    for raw in (s_raw, None):
        alpha = torch.empty(N, dtype=torch.float64, device="cuda")
        beta = torch.empty(N, dtype=torch.float64, device="cuda")
        nll = torch.empty(N, dtype=torch.float64, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        hora.hora_learned_prior(t(p_hat), None if raw is None else t(raw), 2.0, N, alpha, beta, status)
        hora.hora_beta_binomial_nll(t(p_hat), None if raw is None else t(raw), 2.0, t(c), G0, N, nll, status)
        torch.cuda.synchronize()
        a_o, b_o = prior.learned_prior(p_hat, raw, 2.0)
        assert int(status.item()) == 0
        np.testing.assert_allclose(alpha.cpu().numpy(), a_o, rtol=1e-14)
        np.testing.assert_allclose(beta.cpu().numpy(), b_o, rtol=1e-14)
        np.testing.assert_allclose(nll.cpu().numpy(), prior.beta_binomial_nll(p_hat, c, G0, raw, 2.0), rtol=1e-11, atol=1e-12)
    # the priors plug into the allocation: learned prior with s = 2, p_hat = 1/2 equals the uniform prior
    import gpu_util as gu
    alpha = torch.empty(64, dtype=torch.float64, device="cuda")
    beta = torch.empty(64, dtype=torch.float64, device="cuda")
    hora.hora_learned_prior(torch.full((64,), 0.5, dtype=torch.float64, device="cuda"), None, 2.0, 64, alpha, beta)
    cc = rng.integers(0, 5, 64).astype(np.int32)
    cap = np.full(64, 20, np.int32)
    d1 = gu.gpu_allocate(alpha.cpu().numpy(), beta.cpu().numpy(), 1.0, 1.0, cc, 4, cap, 20, 300, exact=True)[0]
    d2 = gu.gpu_allocate(None, None, 1.0, 1.0, cc, 4, cap, 20, 300, exact=True)[0]
    np.testing.assert_array_equal(d1, d2)
    bad = torch.tensor([0.5, 1.0, 0.2], dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hora.hora_learned_prior(bad, None, 2.0, 3, alpha[:3], beta[:3], status)
    assert int(status.item()) == 2


# ------------------------------------------------------------------------------------ Pass@K estimator
@pytest.mark.parametrize("Q,n", [(1, 1), (257, 16), (40000, 128), (3000, 1024)])
def test_pass_at_k_matches_oracle(Q, n):
    from oracle import passk
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(Q + n)
    p = rng.beta(0.5, 1.5, Q)                                   # many hard prompts, a tail of easy ones
    c = rng.binomial(n, p).astype(np.int32)
    Ks = sorted({min(k, n) for k in (1, 2, 4, 8, max(n // 2, 1), n)})
    c_d = torch.from_numpy(c).cuda()
    K_d = torch.tensor(Ks, dtype=torch.int32, device="cuda")
    out = torch.full((len(Ks),), -1.0, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(hora.hora_pass_at_k_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    hora.hora_pass_at_k(c_d, Q, n, K_d, len(Ks), out, status, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # 1 - prod of up to n ratios, each rounded once: absolute error below n * 2^-52, far inside 1e-12
    np.testing.assert_allclose(out.cpu().numpy(), passk.pass_at_k(c, n, Ks), rtol=0, atol=1e-12)
    again = torch.empty_like(out)
    hora.hora_pass_at_k(c_d, Q, n, K_d, len(Ks), again, status, ws)
    assert torch.equal(out, again)                              # fixed summation order


def test_pass_at_k_rejects_bad_counts_and_k():
    from paper_2605_07114_b200 import hora
    n = 8
    ws = torch.empty(hora.hora_pass_at_k_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    out = torch.empty(2, dtype=torch.float64, device="cuda")
    for c, Ks in (([1, 9, 2], [1, 2]), ([1, 2, 3], [1, 9])):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        hora.hora_pass_at_k(torch.tensor(c, dtype=torch.int32, device="cuda"), 3, n,
                            torch.tensor(Ks, dtype=torch.int32, device="cuda"), 2, out, status, ws)
        assert int(status.item()) == 2
    with pytest.raises(hora.HoraError):
        hora.hora_pass_at_k(torch.zeros(3, dtype=torch.int32, device="cuda"), 3, n,
                            torch.ones(2, dtype=torch.int32, device="cuda"), 2, out, None, ws[:8])


# ------------------------------------------------------------------------ fused advantage -> tokens
def _fused_case(rng, sizes, len_lo, len_hi, binary):
    goff = np.zeros(len(sizes) + 1, np.int64)
    np.cumsum(sizes, out=goff[1:])
    R = int(goff[-1])
    rewards = (rng.random(R) < 0.35).astype(np.float32) if binary else rng.choice([0.0, 0.5, 1.0], R).astype(np.float32)
    lens = rng.integers(len_lo, len_hi + 1, R)
    toff = np.zeros(R + 1, np.int64)
    np.cumsum(lens, out=toff[1:])
    return goff, rewards, toff


@pytest.mark.parametrize("mode,ddof,wmode", [(0, 0, None), (0, 1, 0), (1, 0, 1), (1, 0, None)])
@pytest.mark.parametrize("shape", ["mixed", "long_groups", "short_rollouts", "tiny"])
def test_group_advantage_tokens_matches_oracle(mode, ddof, wmode, shape):
    """Fused call == oracle advantage, then oracle broadcast (and oracle weights, broadcast), element by element."""
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng([mode, ddof, len(shape)])
    if shape == "mixed":
        sizes, lo, hi = rng.choice([0, 1, 2, 8, 9, 31, 32, 33, 100, 264], 1500), 0, 700
    elif shape == "long_groups":
        sizes, lo, hi = rng.choice([1024, 1500, 3000, 8], 40), 1, 300       # groups that span several chunks and stages
    elif shape == "short_rollouts":
        sizes, lo, hi = rng.choice([8, 32, 40], 6000), 0, 3                 # thousands of rollouts per chunk: many stage rounds
    else:
        sizes, lo, hi = np.array([3, 0, 2]), 1, 5
    goff, rewards, toff = _fused_case(rng, sizes, lo, hi, binary=(mode == 0))
    N, R, T = len(sizes), int(goff[-1]), int(toff[-1])
    eps = 1e-6
    for misalign in (0, 1):
        buf = torch.full((T + 8,), -7.0, dtype=torch.float32, device="cuda")
        wbuf = torch.full((T + 8,), -7.0, dtype=torch.float32, device="cuda")
        out, wout = buf[misalign:misalign + T], wbuf[misalign:misalign + T]
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        hora.hora_group_advantage_tokens(torch.from_numpy(rewards).cuda(), torch.from_numpy(goff).cuda(), N,
                                         torch.from_numpy(toff).cuda(), R, T, mode, eps, ddof, out,
                                         None if wmode is None else wout, 0 if wmode is None else wmode, 512.0, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        adv = orc.group_advantage(rewards, goff, mode, eps, ddof)
        np.testing.assert_allclose(out.cpu().numpy(), orc.token_broadcast(adv, toff), rtol=0, atol=1e-5)
        assert float(buf[misalign + T:].min()) == -7.0 and (misalign == 0 or float(buf[0]) == -7.0)
        if wmode is not None:
            w = orc.rollout_weights(goff, toff, wmode, 512.0)
            assert np.array_equal(wout.cpu().numpy().view(np.uint32), orc.token_broadcast(w, toff).view(np.uint32))


def test_group_advantage_tokens_partial_cover():
    """T below the token count stops early; rollouts beyond the last group get 0."""
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(5)
    goff, rewards, toff = _fused_case(rng, rng.choice([8, 32], 300), 1, 400, True)
    N, R = 300, int(goff[-1])
    T = int(toff[-1]) - 12345
    out = torch.full((int(toff[-1]),), -7.0, dtype=torch.float32, device="cuda")
    hora.hora_group_advantage_tokens(torch.from_numpy(rewards).cuda(), torch.from_numpy(goff).cuda(), N,
                                     torch.from_numpy(toff).cuda(), R, T, 0, 1e-6, 0, out)
    exp = orc.token_broadcast(orc.group_advantage(rewards, goff, 0, 1e-6, 0), toff)
    got = out.cpu().numpy()
    np.testing.assert_allclose(got[:T], exp[:T], rtol=0, atol=1e-5)
    assert (got[T:] == -7.0).all()
    # only the first 200 groups are described: later rollouts carry no advantage
    out.fill_(-7.0)
    hora.hora_group_advantage_tokens(torch.from_numpy(rewards).cuda(), torch.from_numpy(goff[:201].copy()).cuda(), 200,
                                     torch.from_numpy(toff).cuda(), R, int(toff[-1]), 0, 1e-6, 0, out)
    got = out.cpu().numpy()
    cut = int(toff[goff[200]])
    np.testing.assert_allclose(got[:cut], exp[:cut], rtol=0, atol=1e-5)
    assert (got[cut:] == 0.0).all()


# ----------------------------------------------------------------------- allocation share (Fig. 3)
@pytest.mark.parametrize("N,G0", [(0, 8), (1, 0), (77, 8), (100003, 8), (250000, 16), (50000, 2047)])
def test_allocation_share_bit_exact(N, G0):
    from oracle import share as share_orc
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(N + G0)
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    d = rng.integers(0, 1025, N).astype(np.int32)
    if N > 10:
        d[:4] = 2**31 - 1                                   # sums beyond 32 bits
        c[:4] = c[0]
    prompts = torch.full((G0 + 1,), -1, dtype=torch.int64, device="cuda")
    budget = torch.full((G0 + 1,), -1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hora.hora_allocation_share(torch.from_numpy(c).cuda(), torch.from_numpy(d).cuda(), N, G0, prompts, budget, status)
    torch.cuda.synchronize()
    exp_p, exp_b = share_orc.allocation_share(c, d, G0)
    assert int(status.item()) == 0
    assert prompts.cpu().tolist() == exp_p and budget.cpu().tolist() == exp_b


def test_allocation_share_of_an_allocation_and_bad_input():
    from oracle import share as share_orc
    from paper_2605_07114_b200 import hora
    import gpu_util as gu
    from paper_2605_07114_b200 import workloads as wl
    w = wl.make("cfg2", 4096)
    d = gu.gpu_allocate(w.alpha, w.beta, w.alpha0, w.beta0, w.c, w.G0, w.cap, w.ld, w.B, exact=w.exact_int)[0]
    prompts = torch.empty(w.G0 + 1, dtype=torch.int64, device="cuda")
    budget = torch.empty(w.G0 + 1, dtype=torch.int64, device="cuda")
    hora.hora_allocation_share(torch.from_numpy(w.c).cuda(), torch.from_numpy(d).cuda(), w.N, w.G0, prompts, budget)
    assert int(budget.sum()) == w.B and int(prompts.sum()) == w.N
    assert (prompts.cpu().tolist(), budget.cpu().tolist()) == share_orc.allocation_share(w.c, d, w.G0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    hora.hora_allocation_share(torch.tensor([0, 9, 1], dtype=torch.int32, device="cuda"),
                               torch.tensor([1, 1, 1], dtype=torch.int32, device="cuda"), 3, 8, prompts, budget, status)
    assert int(status.item()) == 2 and int(prompts.sum()) == 2
    with pytest.raises(hora.HoraError):
        hora.hora_allocation_share(None, None, 0, 4096, prompts, budget)


# ------------------------------------------------------------------------------- concurrency
def test_two_allocations_on_two_streams_with_their_own_workspaces():
    """Calls on different streams may overlap as long as they share neither outputs nor workspaces: two different
    problems are enqueued alternately on two streams, several rounds, from two host threads, and each result is held
    against the oracle (and against the same problem run alone)."""
    import threading
    from paper_2605_07114_b200 import hora
    gu = _util()
    probs = []
    for name, N in (("cfg4", 40000), ("cfg5", 60000)):
        w = wl.make(name, N)
        d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
        al = hora.Allocator(w.N, w.ld, w.G0, exact_int=w.exact_int)
        dev = lambda x: None if x is None else gu.dev(x)
        probs.append(dict(w=w, al=al, args=(dev(w.alpha), dev(w.beta), 1.0, 1.0, dev(w.c), dev(w.cap), 0, w.B),
                          oracle=(d_o, lam_o, obj_o), stream=torch.cuda.Stream()))
    torch.cuda.synchronize()
    errors = []

    def worker(p):
        try:
            with torch.cuda.stream(p["stream"]):
                for _ in range(6):
                    p["al"].delta.fill_(-1)
                    p["al"].run(*p["args"])
        except Exception as exc:                                 # pragma: no cover - reported below
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(p,)) for p in probs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for p in probs:
        al, w = p["al"], p["w"]
        d_o, lam_o, obj_o = p["oracle"]
        gu.assert_allocation_matches(w, al.delta.cpu().numpy(), al.G.cpu().numpy(), al.group_offsets.cpu().numpy(),
                                     al.read_info(), d_o, lam_o, obj_o)


def test_back_to_back_steps_on_one_stream_keep_stream_order():
    """The kernels of the four calls start their launch while the kernel before them still runs and then wait for
    it.  Here two different batches go through the SAME buffers (gains matrix, workspace, rewards, advantages) in
    alternation, twelve steps enqueued without a synchronisation between them, each step's results copied aside by
    the stream; every copy must be that batch's oracle result — a kernel that started on its inputs too early, or
    overwrote a buffer the step before was still reading, would show."""
    gu = _util()
    from paper_2605_07114_b200 import hora, workloads as wl
    ws = [wl.make("cfg4", 50000, seed=101), wl.make("cfg4", 50000, seed=202)]
    w0 = ws[0]
    al = hora.Allocator(w0.N, w0.ld, w0.G0, exact_int=False)
    exp, dev_in = [], []
    for w in ws:
        d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
        off = np.zeros(w.N + 1, np.int64)
        np.cumsum(G_o.astype(np.int64), out=off[1:])
        rewards = w.rewards(off)
        adv_o = orc.group_advantage(rewards, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
        exp.append((d_o, adv_o, lam_o))
        dev_in.append((gu.dev(w.alpha), gu.dev(w.beta), gu.dev(w.c), gu.dev(rewards)))
    n_roll = [len(e[1]) for e in exp]
    r_buf = torch.empty(max(n_roll), dtype=torch.float32, device="cuda")
    a_buf = torch.empty(max(n_roll), dtype=torch.float32, device="cuda")
    tok = np.arange(0, 3 * max(n_roll) + 1, 3, dtype=np.int64)          # three tokens a rollout
    tok_d = gu.dev(tok)
    t_buf = torch.empty(3 * max(n_roll), dtype=torch.float32, device="cuda")
    kept = []
    for step in range(12):
        k = step % 2
        w = ws[k]
        alpha, beta, c, rewards = dev_in[k]
        r_buf[:n_roll[k]].copy_(rewards, non_blocking=True)
        al.run(alpha, beta, 1.0, 1.0, c, None, w.ld, w.B)
        hora.hora_group_advantage(r_buf, al.group_offsets, w.N, w.adv_mode, float(w.eps), w.ddof, a_buf)
        hora.hora_token_broadcast(a_buf, tok_d, n_roll[k], 3 * n_roll[k], t_buf)
        kept.append((k, al.delta.clone(), a_buf[:n_roll[k]].clone(), t_buf[:3 * n_roll[k]].clone(), al.info.clone()))
    torch.cuda.synchronize()
    for k, d, a, t, info in kept:
        d_o, adv_o, lam_o = exp[k]
        d = d.cpu().numpy()
        assert hora.read_infos(info, 1)[0].status == 0
        assert int(d.sum()) == ws[k].B
        assert (d != d_o).sum() <= 2                                    # (real priors: a tie at the threshold may swap)
        a = a.cpu().numpy()
        if (d == d_o).all():
            assert np.abs(a - adv_o).max() <= 1e-5
        np.testing.assert_array_equal(t.cpu().numpy(), np.repeat(a, 3))
