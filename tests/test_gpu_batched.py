"""hora_allocate_batched against the oracle run segment by segment (GPU, through the C ABI)."""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import hora_oracle as orc  # noqa: E402


def run_batched(alpha, beta, a0, b0, c, G0, cap, ld, seg, budgets, exact):
    from paper_2605_07114_b200 import hora
    dev = "cuda"
    t = lambda x: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).to(dev)
    N, S = len(c), len(budgets)
    delta = torch.full((N,), -1, dtype=torch.int32, device=dev)
    G = torch.full((N,), -1, dtype=torch.int32, device=dev)
    off = torch.full((N + 1,), -1, dtype=torch.int64, device=dev)
    info = torch.zeros(max(S, 1) * hora.INFO_BYTES, dtype=torch.uint8, device=dev)
    ws = torch.empty(max(hora.hora_allocate_batched_workspace_bytes(N, S), 256), dtype=torch.uint8, device=dev)
    hora.hora_allocate_batched(t(alpha), t(beta), a0, b0, t(c), G0, t(cap), 0, N, ld, seg, budgets,
                               hora.FLAG_EXACT_INT if exact else 0, delta, G, off, info, ws)
    torch.cuda.synchronize()
    return delta.cpu().numpy(), G.cpu().numpy(), off.cpu().numpy(), hora.read_infos(info, S)


def oracle_segments(alpha, beta, a0, b0, c, G0, cap, seg, budgets, exact):
    d = np.zeros(len(c), np.int32)
    lam, obj = [], []
    for s, B in enumerate(budgets):
        sl = slice(int(seg[s]), int(seg[s + 1]))
        al = None if alpha is None else alpha[sl]
        be = None if beta is None else beta[sl]
        if exact:
            ds, _, (ln, ldn), o = orc.greedy_exact(al, be, a0, b0, c[sl], G0, cap[sl], int(B))
            lam.append(ln / ldn if ldn else 0.0)
        else:
            ds, _, l, o = orc.greedy_real(al, be, a0, b0, c[sl], G0, cap[sl], int(B))
            lam.append(l)
        d[sl] = ds
        obj.append(o)
    return d, lam, obj


def random_problem(rng, S, G0, ld, real, max_rows=40, int_priors=False):
    sizes = rng.integers(1, max_rows + 1, S)
    sizes[rng.integers(0, S)] = 1
    seg = np.zeros(S + 1, np.int64)
    np.cumsum(sizes, out=seg[1:])
    N = int(seg[-1])
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    alpha = beta = None
    if real:
        alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
        beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    elif int_priors:
        alpha = rng.integers(1, 4, N).astype(np.float64)
        beta = rng.integers(1, 4, N).astype(np.float64)
    budgets = np.zeros(S, np.int64)
    for s in range(S):
        tot = int(cap[seg[s]:seg[s + 1]].sum())
        budgets[s] = rng.choice([0, tot, int(rng.integers(0, tot + 1))], p=[0.05, 0.05, 0.9])
    return alpha, beta, c, cap, seg, budgets


@pytest.mark.parametrize("G0,ld", [(2, 24), (4, 60), (8, 130), (8, 256), (8, 300)])
@pytest.mark.parametrize("prior", ["shared", "integer", "real"])
@pytest.mark.parametrize("max_rows", [40, 15])
def test_batched_matches_oracle_per_segment(G0, ld, prior, max_rows):
    """shared: one Beta(1,1) prior, exact ties (solved on exact ranks, a warp per segment); integer: per-prompt
    integer priors, exact ties (a CTA per segment, keys in shared memory); real: per-prompt real priors.
    max_rows: segments of up to 40 prompts run 256 threads a CTA (a lane owns several rows in the selection where a
    segment has more than 32), calls whose segments all have at most 32 prompts run 128 threads a CTA.
    ld = 300: rows longer than 256 candidates are solved on their first 256 first; with random caps and budgets many
    segments are not settled by that and go through the full-width pass."""
    real = prior == "real"
    rng = np.random.default_rng(G0 * 1000 + ld + real + 7 * (max_rows != 40))
    alpha, beta, c, cap, seg, budgets = random_problem(rng, 300, G0, ld, real, max_rows=max_rows,
                                                       int_priors=prior == "integer")
    d, G, off, infos = run_batched(alpha, beta, 1.0, 1.0, c, G0, cap, ld, seg, budgets, exact=not real)
    d_o, lam_o, obj_o = oracle_segments(alpha, beta, 1.0, 1.0, c, G0, cap, seg, budgets, exact=not real)
    np.testing.assert_array_equal(d, d_o)
    np.testing.assert_array_equal(G, G0 + d_o)
    exp_off = np.zeros(len(c) + 1, np.int64)
    np.cumsum(G.astype(np.int64), out=exp_off[1:])
    np.testing.assert_array_equal(off, exp_off)
    for s, inf in enumerate(infos):
        assert inf.status == 0
        B = int(budgets[s])
        assert inf.sum_G == (seg[s + 1] - seg[s]) * G0 + B
        assert inf.sum_cap == int(cap[seg[s]:seg[s + 1]].sum())
        if B > 0:
            assert abs(inf.objective - obj_o[s]) <= 1e-12 * abs(obj_o[s])
            assert abs(inf.lambda_ - lam_o[s]) <= 1e-12 * lam_o[s]
            assert inf.n_above + inf.n_tied_taken == B and 1 <= inf.n_tied_taken <= inf.n_tied


def test_paper_shard_shape_and_agreement_with_single_problem_call():
    """Four shards of 15 prompts, 360 rollouts each (G = 32, G0 = 8), uniform prior, exact ties; and each
    shard solved alone by hora_allocate gives the same allocation."""
    import gpu_util as gu
    rng = np.random.default_rng(60)
    G0, shard, B, ld = 8, 15, 360, 360
    N = 4 * shard
    c = rng.choice(G0 + 1, size=N, p=[0.15] + [0.34 / 7] * 7 + [0.51]).astype(np.int32)
    cap = np.full(N, ld, np.int32)
    seg = np.arange(0, N + 1, shard, dtype=np.int64)
    budgets = np.full(4, B, np.int64)
    d, G, off, infos = run_batched(None, None, 1.0, 1.0, c, G0, cap, ld, seg, budgets, exact=True)
    d_o, _, _ = oracle_segments(None, None, 1.0, 1.0, c, G0, cap, seg, budgets, exact=True)
    np.testing.assert_array_equal(d, d_o)
    for s in range(4):
        sl = slice(s * shard, (s + 1) * shard)
        d1, _, _, info1 = gu.gpu_allocate(None, None, 1.0, 1.0, c[sl], G0, cap[sl], ld, B, exact=True)
        np.testing.assert_array_equal(d[sl], d1)
        assert infos[s].n_above == info1.n_above and infos[s].n_tied == info1.n_tied
        assert abs(infos[s].objective - info1.objective) <= 1e-13 * info1.objective
    assert d[c == 0].mean() > d[c == G0].mean()          # hopeless prompts get more than saturated ones


@pytest.mark.parametrize("exact", [False, True])
def test_paper_shard_shape_with_per_prompt_priors(exact):
    """The shape the benchmark times through the CTA-per-segment kernel: shards of 15 prompts, ld = 360, budget 360,
    G0 = 8, per-prompt priors (real with fp64 ties, integer with exact ties)."""
    rng = np.random.default_rng(61 + exact)
    G0, shard, B, ld, S = 8, 15, 360, 360, 96
    N = S * shard
    c = rng.choice(G0 + 1, size=N, p=[0.15] + [0.34 / 7] * 7 + [0.51]).astype(np.int32)
    cap = np.full(N, ld, np.int32)
    if exact:
        alpha = rng.integers(1, 4, N).astype(np.float64)
        beta = rng.integers(1, 4, N).astype(np.float64)
    else:
        alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
        beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    seg = np.arange(0, N + 1, shard, dtype=np.int64)
    budgets = np.full(S, B, np.int64)
    budgets[:8] = [0, 1, 2, 15, 359, 361, 15 * 360, 15 * 360 - 1]      # the ends of the range too
    # Rows of 360 candidates are first solved on their first 256; segments 8..15 hold one hopeless prompt among
    # saturated ones, which takes (nearly) the whole budget — more than 256 — so these must be solved again in full;
    # so must the two budgets above that exceed 15 * 256.
    for s in range(8, 16):
        sl = slice(s * shard, (s + 1) * shard)
        c[sl] = G0
        c[s * shard + s % shard] = 0
        alpha[sl], beta[sl] = (3.0, 1.0) if exact else (20.0, 0.05)
        alpha[s * shard + s % shard], beta[s * shard + s % shard] = (1.0, 3.0) if exact else (0.05, 20.0)
        budgets[s] = 250 + 12 * (s - 8)                            # 250 .. 334: on both sides of 256
    d, G, off, infos = run_batched(alpha, beta, 1.0, 1.0, c, G0, cap, ld, seg, budgets, exact=exact)
    assert d[8 * shard:16 * shard].max() > 256                  # (some row did take more than the narrow pass holds)
    d_o, lam_o, obj_o = oracle_segments(alpha, beta, 1.0, 1.0, c, G0, cap, seg, budgets, exact=exact)
    np.testing.assert_array_equal(d, d_o)
    np.testing.assert_array_equal(G, G0 + d_o)
    for s, inf in enumerate(infos):
        assert inf.status == 0
        if budgets[s] > 0:
            assert abs(inf.objective - obj_o[s]) <= 1e-12 * abs(obj_o[s])
            assert abs(inf.lambda_ - lam_o[s]) <= 1e-12 * lam_o[s]
            assert inf.n_above + inf.n_tied_taken == budgets[s] and 1 <= inf.n_tied_taken <= inf.n_tied


def test_a_failing_segment_leaves_the_others_alone():
    rng = np.random.default_rng(3)
    alpha, beta, c, cap, seg, budgets = random_problem(rng, 20, 4, 32, real=True, max_rows=10)
    budgets[5] = int(cap[seg[5]:seg[6]].sum()) + 1       # infeasible
    alpha[seg[9]] = -2.0                                 # invalid prior in segment 9
    d, G, off, infos = run_batched(alpha, beta, 1.0, 1.0, c, 4, cap, 32, seg, budgets, exact=False)
    assert infos[5].status == 3 and not d[seg[5]:seg[6]].any() and not G[seg[5]:seg[6]].any()
    assert infos[9].status == 2 and not d[seg[9]:seg[10]].any()
    ok = [s for s in range(20) if s not in (5, 9)]
    b2, a2 = budgets.copy(), alpha.copy()
    a2[seg[9]] = 1.0
    d_o, _, _ = oracle_segments(a2, beta, 1.0, 1.0, c, 4, cap, seg, b2 * 0 + np.where(np.arange(20) == 5, 0, b2), False)
    for s in ok:
        assert infos[s].status == 0
        np.testing.assert_array_equal(d[seg[s]:seg[s + 1]], d_o[seg[s]:seg[s + 1]])


def test_segments_beyond_the_per_cta_limits_are_refused():
    from paper_2605_07114_b200 import hora
    N, ld = 600, 64
    c = np.zeros(N, np.int32)
    cap = np.full(N, ld, np.int32)
    ones = np.ones(N)
    with pytest.raises(hora.HoraError) as e:            # per-prompt priors: a CTA per segment, 256 prompts at most
        run_batched(ones, ones, 1.0, 1.0, c, 4, cap, ld, np.array([0, 300, 600]), np.array([10, 10]), exact=False)
    assert e.value.code == hora.ERR_WORKSPACE
    with pytest.raises(hora.HoraError) as e:
        run_batched(None, None, 1.0, 1.0, c, 4, cap, ld, np.array([0, 300, 500]), np.array([10, 10]), exact=True)
    assert e.value.code == hora.ERR_INVALID_ARG


@pytest.mark.parametrize("a0,b0", [(1.0, 1.0), (2.0, 3.0)])
def test_shared_integer_prior_has_no_segment_size_limit(a0, b0):
    """One integer prior and exact ties: segments are solved on ranks by one warp each, whatever their size
    (1, 31, 32, 33, 300 and 2000 prompts here), empty segments included."""
    rng = np.random.default_rng(int(a0 * 10 + b0))
    G0, ld = 8, 96
    sizes = np.array([1, 31, 0, 32, 33, 300, 2000, 15, 0, 64])
    seg = np.zeros(len(sizes) + 1, np.int64)
    np.cumsum(sizes, out=seg[1:])
    N = int(seg[-1])
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    budgets = np.array([int(rng.integers(0, int(cap[seg[s]:seg[s + 1]].sum()) + 1)) for s in range(len(sizes))], np.int64)
    d, G, off, infos = run_batched(None, None, a0, b0, c, G0, cap, ld, seg, budgets, exact=True)
    d_o, lam_o, obj_o = oracle_segments(None, None, a0, b0, c, G0, cap, seg, budgets, exact=True)
    np.testing.assert_array_equal(d, d_o)
    np.testing.assert_array_equal(off, np.concatenate(([0], np.cumsum(G0 + d_o.astype(np.int64)))))
    for s, inf in enumerate(infos):
        assert inf.status == 0 and inf.sum_cap == int(cap[seg[s]:seg[s + 1]].sum())
        if budgets[s] > 0:
            assert abs(inf.objective - obj_o[s]) <= 1e-12 * abs(obj_o[s])
            assert abs(inf.lambda_ - lam_o[s]) <= 1e-12 * lam_o[s]
            assert inf.n_above + inf.n_tied_taken == budgets[s] and 1 <= inf.n_tied_taken <= inf.n_tied


@pytest.mark.parametrize("a0,b0", [(1.0, 1.0), (0.37, 2.9)])
def test_shared_prior_with_fp64_ties_matches_the_per_prompt_form(a0, b0):
    """Without the exact flag a shared prior is ranked as doubles: the result must be what the per-prompt form of the
    same call (the same prior in arrays: a CTA per segment on its own rows) gives, bit for bit, and the oracle's
    within its band."""
    rng = np.random.default_rng(5)
    G0, ld = 8, 60
    sizes = rng.integers(1, 40, 200)
    seg = np.zeros(len(sizes) + 1, np.int64)
    np.cumsum(sizes, out=seg[1:])
    N = int(seg[-1])
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    budgets = np.array([int(rng.integers(0, int(cap[seg[s]:seg[s + 1]].sum()) + 1)) for s in range(len(sizes))], np.int64)
    d, G, off, infos = run_batched(None, None, a0, b0, c, G0, cap, ld, seg, budgets, exact=False)
    d2, G2, off2, infos2 = run_batched(np.full(N, a0), np.full(N, b0), 1.0, 1.0, c, G0, cap, ld, seg, budgets, exact=False)
    np.testing.assert_array_equal(d, d2)
    np.testing.assert_array_equal(off, off2)
    for x, y in zip(infos, infos2):
        assert (x.status, x.n_above, x.n_tied, x.n_tied_taken) == (y.status, y.n_above, y.n_tied, y.n_tied_taken)
        assert x.lambda_ == y.lambda_ and abs(x.objective - y.objective) <= 1e-12 * max(abs(y.objective), 1e-300)
    if a0 != 1.0:                                        # a real prior: no ties, the oracle's allocation is the only one
        d_o, _, _ = oracle_segments(np.full(N, a0), np.full(N, b0), 1.0, 1.0, c, G0, cap, seg, budgets, exact=False)
        np.testing.assert_array_equal(d, d_o)


def test_shared_prior_segments_fail_one_by_one():
    rng = np.random.default_rng(12)
    G0, ld, S = 4, 20, 12
    seg = np.arange(0, 15 * S + 1, 15, dtype=np.int64)
    N = int(seg[-1])
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    budgets = np.full(S, 40, np.int64)
    budgets[3] = int(cap[seg[3]:seg[4]].sum()) + 1       # infeasible
    c[seg[7] + 2] = G0 + 1                               # a count outside [0, G0]
    d, G, off, infos = run_batched(None, None, 1.0, 1.0, c, G0, cap, ld, seg, budgets, exact=True)
    assert infos[3].status == 3 and infos[7].status == 2
    assert not d[seg[3]:seg[4]].any() and not G[seg[7]:seg[8]].any()
    for s in range(S):
        if s in (3, 7):
            continue
        sl = slice(int(seg[s]), int(seg[s + 1]))
        assert infos[s].status == 0
        np.testing.assert_array_equal(d[sl], orc.greedy_exact(None, None, 1.0, 1.0, c[sl], G0, cap[sl], 40)[0])
