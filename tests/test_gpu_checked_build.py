"""The checked build (-DHORA_CHECKED): the allocation, batched-allocation, rank-route and advantage kernels with an
index check on every access whose index comes from device data.  Odd sizes (N and ld off the multiples of 32 and 4,
ragged caps, unaligned buffers, missed windows, heavy ties) run through it; results must equal the oracle's and the
violation word must stay 0.  Nothing here provokes a violation: the check records, it never traps."""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import hora_oracle as orc  # noqa: E402
from paper_2605_07114_b200 import workloads as wl  # noqa: E402


@pytest.fixture()
def checked():
    from paper_2605_07114_b200 import build, hora
    path = build.build(checked=True)
    assert hora.hora_checked_violation() == -1              # the default build has no checks and says so
    hora.use_library(path)
    assert hora.hora_checked_violation() == 0
    yield hora
    left = hora.hora_checked_violation()
    hora.use_library(None)
    assert left == 0, f"index check failed: file {left >> 20}, line {left & 0xFFFFF}"


def _alloc(hora, alpha, beta, c, G0, cap, ld, B, exact, materialise):
    import gpu_util as gu
    return gu.gpu_allocate(alpha, beta, 1.0, 1.0, c, G0, cap, ld, B, exact=exact, materialise=materialise)


@pytest.mark.parametrize("seed", range(6))
def test_allocation_on_odd_shapes(checked, seed):
    rng = np.random.default_rng(4000 + seed)
    N = int(rng.integers(1, 5000)) | 1
    ld = int(rng.choice([1, 3, 7, 31, 63, 65, 129, 255, 257, 301]))
    G0 = int(rng.integers(1, 9))
    exact = bool(seed % 2)
    c = rng.integers(0, G0 + 1, N).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    if exact:
        alpha = rng.integers(1, 4, N).astype(np.float64)
        beta = rng.integers(1, 4, N).astype(np.float64)
    else:
        alpha = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
        beta = np.exp(rng.uniform(np.log(0.05), np.log(20), N))
    total = int(cap.sum())
    for B in sorted({0, 1, total // 3, total}):
        d_o = (orc.greedy_exact if exact else orc.greedy_real)(alpha, beta, 1.0, 1.0, c, G0, cap, B)[0]
        for materialise in (True, False):
            d, G, off, info = _alloc(checked, alpha, beta, c, G0, cap, ld, B, exact, materialise)
            assert info.status == 0
            np.testing.assert_array_equal(d, d_o)
    assert checked.hora_checked_violation() == 0


def test_missed_window_heavy_ties_and_rank_route(checked):
    import gpu_util as gu
    # a sample that misleads (the 13-bit fallback), then a single class with more ties than the list holds
    N, G0, ld = 20001, 8, 95
    idx = np.arange(N)
    c = np.where(idx % 5 == 0, 0, G0).astype(np.int32)
    cap = np.full(N, ld, np.int32)
    ones = np.ones(N)
    for B in (1000, 7 * N):
        d_o = orc.greedy_exact(None, None, 1.0, 1.0, c, G0, cap, B)[0]
        for materialise in (True, False):
            d, _, _, info = gu.gpu_allocate(ones, ones, 1.0, 1.0, c, G0, cap, ld, B, exact=True, materialise=materialise)
            assert info.status == 0
            np.testing.assert_array_equal(d, d_o)
    N = (1 << 17) + 3
    c = np.zeros(N, np.int32)
    cap = np.full(N, 23, np.int32)
    cap[::7] = 5
    B = 9 * N + 4321
    d_o = orc.greedy_exact(None, None, 1.0, 1.0, c, 4, cap, B)[0]
    ones = np.ones(N)
    d, _, _, info = gu.gpu_allocate(ones, ones, 1.0, 1.0, c, 4, cap, 23, B, exact=True)
    assert info.status == 0 and info.n_tied > 65536
    np.testing.assert_array_equal(d, d_o)
    # the rank-based route on the same data, and on a cfg5-like ragged problem
    d, _, _, info = gu.gpu_allocate(None, None, 1.0, 1.0, c, 4, cap, 23, B, exact=True, materialise=False, shared_int_prior=True)
    assert info.status == 0 and info.first_pass_bits == -1
    np.testing.assert_array_equal(d, d_o)
    w = wl.make("cfg5", 30001)
    d_o = orc.greedy_exact(None, None, 1.0, 1.0, w.c, w.G0, w.cap, w.B)[0]
    d, _, _, info = gu.gpu_allocate(None, None, 1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B, exact=True, materialise=False)
    np.testing.assert_array_equal(d, d_o)
    assert checked.hora_checked_violation() == 0


def test_batched_and_advantages(checked):
    import gpu_util as gu
    import test_gpu_batched as tb
    rng = np.random.default_rng(77)
    for prior, max_rows in (("shared", 37), ("integer", 37), ("real", 37), ("integer", 15), ("real", 15)):
        alpha, beta, c, cap, seg, budgets = tb.random_problem(rng, 120, 8, 131, prior == "real", max_rows=max_rows,
                                                              int_priors=prior == "integer")
        d, G, off, infos = tb.run_batched(alpha, beta, 1.0, 1.0, c, 8, cap, 131, seg, budgets, exact=prior != "real")
        d_o, _, _ = tb.oracle_segments(alpha, beta, 1.0, 1.0, c, 8, cap, seg, budgets, exact=prior != "real")
        np.testing.assert_array_equal(d, d_o)
    # ragged groups (empty, single, long), 0/1 and general rewards, unaligned buffers
    sizes = np.concatenate([rng.integers(0, 70, 3000), [0, 1, 1537, 3000, 2, 0]])
    off = np.zeros(len(sizes) + 1, np.int64)
    np.cumsum(sizes, out=off[1:])
    total = int(off[-1])
    for rewards in ((rng.random(total) < 0.3).astype(np.float32), rng.choice([0.0, 0.5, 1.0], total).astype(np.float32)):
        for mode in (0, 1):
            exp = orc.group_advantage(rewards, off, mode, 1e-6, 0)
            for mis in (0, 1):
                buf_r = torch.zeros(total + 8, dtype=torch.float32, device="cuda")
                buf_a = torch.full((total + 8,), 7.0, dtype=torch.float32, device="cuda")
                buf_r[mis:mis + total] = torch.from_numpy(rewards).cuda()
                checked.hora_group_advantage(buf_r[mis:mis + total], gu.dev(off), len(sizes), mode, 1e-6, 0, buf_a[mis:mis + total])
                torch.cuda.synchronize()
                assert np.abs(buf_a[mis:mis + total].cpu().numpy() - exp).max() <= 1e-5
                assert (buf_a[mis + total:] == 7.0).all() and (buf_a[:mis] == 7.0).all()
    assert checked.hora_checked_violation() == 0
