"""The rank-based route of hora_allocate (one integer prior for all prompts, exact ties, no gains matrix) against
exact greedy: bit-exact Delta, G and offsets; the threshold, the tie counts and the objective against the oracle."""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import hora_oracle as orc  # noqa: E402
from paper_2605_07114_b200 import workloads as wl  # noqa: E402


def _gu():
    import gpu_util
    return gpu_util


def rank_allocate(a0, b0, c, G0, cap, ld, B, **kw):
    gu = _gu()
    d, G, off, info = gu.gpu_allocate(None, None, a0, b0, c, G0, cap, ld, B, exact=True, materialise=False,
                                      shared_int_prior=True, **kw)
    if info.status == 0 and B > 0:
        assert info.first_pass_bits == -1                # the route under test did run
    return d, G, off, info


def check(a0, b0, c, G0, cap, ld, B):
    d_o, G_o, (ln, ldn), obj = orc.greedy_exact(None, None, a0, b0, c, G0, cap, B)
    d, G, off, info = rank_allocate(a0, b0, c, G0, cap, ld, B)
    assert info.status == 0, info
    np.testing.assert_array_equal(d, d_o, err_msg=f"B={B}")
    np.testing.assert_array_equal(G, G0 + d_o)
    np.testing.assert_array_equal(off, np.concatenate(([0], np.cumsum(G0 + d_o.astype(np.int64)))))
    assert info.sum_G == len(c) * G0 + B and info.sum_cap == int(cap.astype(np.int64).sum())
    assert info.n_above + info.n_tied_taken == B
    if B > 0:
        lam = ln / ldn
        assert abs(info.lambda_ - lam) <= 1e-12 * lam
        assert abs(info.objective - obj) <= 1e-12 * obj
        assert 1 <= info.n_tied_taken <= info.n_tied
        # n_tied is the number of candidates exactly equal to the threshold: count them with the oracle's rationals
        from fractions import Fraction
        from oracle import literal
        tied = 0
        for k in range(G0 + 1):
            row = literal.marginals(*literal.posterior(int(a0), int(b0), k, G0), ld)
            for D, g in enumerate(row, start=1):
                if g == Fraction(ln, ldn):
                    tied += int(((c == k) & (cap >= D)).sum())
        assert info.n_tied == tied
    return info


def test_every_budget_on_the_worked_example():
    c = np.array([0, 1, 2, 0], np.int32)
    cap = np.full(4, 3, np.int32)
    for B in range(0, 13):
        check(1.0, 1.0, c, 2, cap, 3, B)


@pytest.mark.parametrize("G0", [2, 4, 8, 16])
def test_budget_sweep_through_cross_class_ties(G0):
    rng = np.random.default_rng(G0)
    N, ld = 97, 40
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    total = int(cap.sum())
    for B in sorted(set([0, 1, 2, total - 1, total] + [int(x) for x in rng.integers(0, total + 1, 40)])):
        check(1.0, 1.0, c, G0, cap, ld, B)


@pytest.mark.parametrize("seed", range(10))
def test_random_shapes_and_shared_integer_priors(seed):
    rng = np.random.default_rng(500 + seed)
    N = int(rng.integers(1, 9000))
    G0 = int(rng.integers(0, 10))
    ld = int(rng.choice([1, 2, 7, 31, 64, 65, 100, 256, 300, 700]))
    if (G0 + 1) * ld > 8192:
        ld = 8192 // (G0 + 1)
    a0, b0 = float(rng.integers(1, 5)), float(rng.integers(1, 5))
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    if seed % 3 == 0:
        cap[:] = ld
    total = int(cap.sum())
    for B in sorted({0, 1, total // 3, total // 2, max(total - 1, 0), total}):
        check(a0, b0, c, G0, cap, ld, B)


def test_scalar_cap_and_unaligned_outputs():
    gu = _gu()
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(3)
    N, G0, ld, B = 3001, 4, 50, 40000
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    d_o = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, np.full(N, 37, np.int32), B)[0]
    d, G, off, info = rank_allocate(1.0, 1.0, c, G0, None, ld, B, cap_scalar=37)
    assert info.status == 0
    np.testing.assert_array_equal(d, d_o)
    # outputs that start one element into their buffers (no 16-byte stores), guard values around them
    buf_d = torch.full((N + 2,), -7, dtype=torch.int32, device="cuda")
    buf_G = torch.full((N + 2,), -7, dtype=torch.int32, device="cuda")
    buf_o = torch.full((N + 3,), -7, dtype=torch.int64, device="cuda")
    ws = torch.empty(hora.hora_allocate_workspace_bytes(N, ld, True, 5), dtype=torch.uint8, device="cuda")
    inf = torch.zeros(hora.INFO_BYTES, dtype=torch.uint8, device="cuda")
    hora.hora_allocate(None, None, 1.0, 1.0, gu.dev(c), G0, None, 37, N, ld, None, B, hora.FLAG_EXACT_INT, buf_d[1:N + 1],
                       buf_G[1:N + 1], buf_o[1:N + 2], inf, ws)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(buf_d[1:N + 1].cpu().numpy(), d_o)
    np.testing.assert_array_equal(buf_o[1:N + 2].cpu().numpy(), np.concatenate(([0], np.cumsum(G0 + d_o.astype(np.int64)))))
    assert buf_d[0] == -7 and buf_d[-1] == -7 and buf_G[0] == -7 and buf_G[-1] == -7 and buf_o[0] == -7 and buf_o[-1] == -7


def test_status_codes_and_zeroed_outputs():
    N, G0, ld = 500, 4, 16
    c = np.full(N, 1, np.int32)
    cap = np.full(N, ld, np.int32)
    d, G, off, info = rank_allocate(1.0, 1.0, c, G0, cap, ld, N * ld + 1)
    assert info.status == 3 and not d.any() and not G.any() and not off.any()
    for bad_c in (G0 + 1, -1, -5):
        c2 = c.copy()
        c2[77] = bad_c
        d, G, off, info = rank_allocate(1.0, 1.0, c2, G0, cap, ld, 50)
        assert info.status == 2 and not d.any() and not G.any()
    cap2 = cap.copy()
    cap2[400] = ld + 1
    d, G, off, info = rank_allocate(1.0, 1.0, c, G0, cap2, ld, 50)
    assert info.status == 2 and not d.any()
    d, G, off, info = rank_allocate(1.0, 1.0, c, G0, cap, ld, 0)
    assert info.status == 0 and not d.any() and (G == G0).all() and off[-1] == N * G0 and info.lambda_ == 0.0


def test_route_agrees_with_the_general_exact_path():
    """The same problem through the general exact path (matrix given): identical Delta, tie counts and threshold."""
    gu = _gu()
    w = wl.make("cfg5", 1 << 16)
    d1, G1, off1, i1 = gu.gpu_allocate(None, None, 1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B, exact=True, materialise=True)
    d2, G2, off2, i2 = rank_allocate(1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B)
    np.testing.assert_array_equal(d1, d2)
    np.testing.assert_array_equal(off1, off2)
    assert (i1.n_above, i1.n_tied, i1.n_tied_taken) == (i2.n_above, i2.n_tied, i2.n_tied_taken)
    assert abs(i1.lambda_ - i2.lambda_) <= 1e-13 * i1.lambda_ and abs(i1.objective - i2.objective) <= 1e-12 * i1.objective


@pytest.mark.parametrize("a0,b0", [(1.0, 1.0), (2.0, 5.0), (0.5, 0.5), (3.7, 0.21)])
def test_fp64_ties_on_ranks_equal_the_key_based_selection(a0, b0):
    """Without the exact flag the shared prior's candidate values are ranked as the doubles hora_gains writes, equal
    doubles tie: Delta, the tie counts and the threshold must be those of the key-based selection on the
    materialised matrix, bit for bit; for a real prior (no ties) also the oracle's."""
    gu = _gu()
    rng = np.random.default_rng(int(a0 * 100 + b0 * 10))
    N, G0, ld = 20011, 6, 90
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    total = int(cap.sum())
    for B in (0, 1, total // 5, total // 2, total - 1, total):
        d1, G1, off1, i1 = gu.gpu_allocate(None, None, a0, b0, c, G0, cap, ld, B, exact=False, materialise=True)
        d2, G2, off2, i2 = gu.gpu_allocate(None, None, a0, b0, c, G0, cap, ld, B, exact=False, materialise=False,
                                           shared_int_prior=True)
        assert i1.status == 0 and i2.status == 0
        assert i2.first_pass_bits == (-1 if B > 0 else 0) and i1.first_pass_bits in (0, 13, 23)
        np.testing.assert_array_equal(d1, d2, err_msg=f"B={B}")
        np.testing.assert_array_equal(off1, off2)
        assert (i1.n_above, i1.n_tied, i1.n_tied_taken) == (i2.n_above, i2.n_tied, i2.n_tied_taken)
        assert i1.lambda_ == i2.lambda_
        assert abs(i1.objective - i2.objective) <= 1e-12 * max(abs(i1.objective), 1e-300)
        if a0 != np.floor(a0) and B > 0:
            d_o, _, lam_o, obj_o = orc.greedy_real(None, None, a0, b0, c, G0, cap, B)
            np.testing.assert_array_equal(d2, d_o)
            assert abs(i2.lambda_ - lam_o) <= 1e-12 * lam_o and abs(i2.objective - obj_o) <= 1e-12 * obj_o


def test_shapes_outside_the_route_fall_back_to_the_general_path():
    """(G0 + 1) * ld above 8192 types: the call builds the matrix as before (needs the full-size workspace)."""
    gu = _gu()
    rng = np.random.default_rng(4)
    N, G0, ld = 400, 8, 1000
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    B = int(cap.sum()) // 3
    d_o = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, B)[0]
    d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, G0, cap, ld, B, exact=True, materialise=False)
    assert info.status == 0 and info.first_pass_bits in (13, 23)
    np.testing.assert_array_equal(d, d_o)


def test_cfg5_full_size_on_ranks():
    gu = _gu()
    w = wl.make("cfg5")
    d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
    d, G, off, info = rank_allocate(1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B)
    gu.assert_allocation_matches(w, d, G, off, info, d_o, lam_o, obj_o)
    assert info.n_tied > 1_000_000 and 0 < info.n_tied_taken < info.n_tied
