"""hora_allocate_hard_first (the comparison allocator of Sec. 4.2) against its plain-loop oracle: bit-exact."""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import hard_first as hf  # noqa: E402


def run(c, G0, cap, ld, B, cap_scalar=None):
    from paper_2605_07114_b200 import hora
    dev = "cuda"
    N = len(c)
    t = lambda x: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).to(dev)
    delta = torch.full((N,), -1, dtype=torch.int32, device=dev)
    G = torch.full((N,), -1, dtype=torch.int32, device=dev)
    off = torch.full((N + 1,), -1, dtype=torch.int64, device=dev)
    info = torch.zeros(hora.INFO_BYTES, dtype=torch.uint8, device=dev)
    ws = torch.empty(max(hora.hora_allocate_hard_first_workspace_bytes(N, ld), 256), dtype=torch.uint8, device=dev)
    hora.hora_allocate_hard_first(t(c), G0, t(cap), 0 if cap_scalar is None else cap_scalar, N, ld, B, delta, G, off, info, ws)
    torch.cuda.synchronize()
    return delta.cpu().numpy(), G.cpu().numpy(), off.cpu().numpy(), hora.read_info(info)


def check(c, G0, cap, ld, B):
    d_o = np.array(hf.hard_first([int(x) for x in c], [int(x) for x in cap], int(B)), np.int32)
    d, G, off, info = run(c, G0, cap, ld, B)
    assert info.status == 0
    np.testing.assert_array_equal(d, d_o, err_msg=f"B={B}")
    np.testing.assert_array_equal(G, G0 + d_o)
    np.testing.assert_array_equal(off, np.concatenate(([0], np.cumsum(G0 + d_o.astype(np.int64)))))
    assert info.sum_G == len(c) * G0 + B and info.sum_cap == int(cap.astype(np.int64).sum())
    assert info.n_above + info.n_tied_taken == B and 0 <= info.n_tied_taken <= info.n_tied
    assert info.lambda_ == 0.0 and info.objective == 0.0


def test_hand_example_every_budget():
    c = np.array([0, 1, 0, 4, 2, 0], np.int32)
    cap = np.array([3, 9, 1, 9, 9, 9], np.int32)
    for B in range(0, int(cap.sum()) + 1):
        check(c, 4, cap, 9, B)


@pytest.mark.parametrize("seed", range(8))
def test_random_shapes(seed):
    rng = np.random.default_rng(900 + seed)
    N = int(rng.integers(1, 7000))
    G0 = int(rng.integers(1, 9))
    ld = int(rng.choice([1, 3, 24, 64, 360, 1000]))
    p0 = [0.0, 0.15, 0.5, 1.0][seed % 4]                     # share of c = 0 prompts: none, few, half, all
    c = np.where(rng.random(N) < p0, 0, rng.integers(1, G0 + 1, N)).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    if seed % 3 == 0:
        cap[:] = ld
    total = int(cap.sum())
    hard_room = int(cap[c == 0].sum())
    for B in sorted({0, 1, hard_room // 2, max(hard_room - 1, 0), hard_room, min(hard_room + 1, total), (hard_room + total) // 2, total}):
        check(c, G0, cap, ld, B)


def test_paper_shape_shard():
    """A shard of 15 prompts with 360 extra rollouts (G = 32, G0 = 8): all of them go to the c = 0 prompts."""
    rng = np.random.default_rng(1)
    G0, N, B, ld = 8, 15, 360, 360
    c = rng.choice(G0 + 1, size=N, p=[0.15] + [0.34 / 7] * 7 + [0.51]).astype(np.int32)
    c[3] = 0
    cap = np.full(N, ld, np.int32)
    d, G, off, info = run(c, G0, cap, ld, B)
    assert info.status == 0 and d.sum() == B and not d[c != 0].any()
    assert d[c == 0].max() - d[c == 0].min() <= 1
    check(c, G0, cap, ld, B)


def test_scalar_cap_and_status_codes():
    N, G0, ld = 1000, 4, 32
    c = (np.arange(N) % 5).astype(np.int32)
    d, G, off, info = run(c, G0, None, ld, 3000, cap_scalar=20)
    assert info.status == 0
    np.testing.assert_array_equal(d, np.array(hf.hard_first(list(c), [20] * N, 3000), np.int32))
    d, G, off, info = run(c, G0, None, ld, 20 * N + 1, cap_scalar=20)
    assert info.status == 3 and not d.any() and not G.any() and not off.any()
    bad = c.copy()
    bad[17] = -1
    d, G, off, info = run(bad, G0, None, ld, 100, cap_scalar=20)
    assert info.status == 2 and not d.any()
    cap = np.full(N, 20, np.int32)
    cap[5] = ld + 1
    d, G, off, info = run(c, G0, cap, ld, 100)
    assert info.status == 2 and not d.any()


def test_hard_first_per_segment():
    """hora_allocate_batched with HORA_FLAG_HARD_FIRST: every segment by the comparison rule, against the plain loops
    run segment by segment (segments of 0, 1, 15, 32, 33 and 700 prompts; budgets below, at and above what the c = 0
    prompts can take; an infeasible and an invalid segment that leave the others alone)."""
    from paper_2605_07114_b200 import hora
    rng = np.random.default_rng(321)
    G0, ld = 8, 40
    sizes = np.array([15] * 40 + [0, 1, 32, 33, 700, 15, 15])
    seg = np.zeros(len(sizes) + 1, np.int64)
    np.cumsum(sizes, out=seg[1:])
    N, S = int(seg[-1]), len(sizes)
    c = np.where(rng.random(N) < 0.2, 0, rng.integers(1, G0 + 1, N)).astype(np.int32)
    cap = rng.integers(0, ld + 1, N).astype(np.int32)
    budgets = np.zeros(S, np.int64)
    for s in range(S):
        sl = slice(int(seg[s]), int(seg[s + 1]))
        hard, total = int(cap[sl][c[sl] == 0].sum()), int(cap[sl].sum())
        budgets[s] = [0, hard // 2, hard, min(hard + 3, total), total, int(rng.integers(0, total + 1))][s % 6]
    budgets[S - 2] = int(cap[seg[S - 2]:seg[S - 1]].sum()) + 1          # infeasible
    c[seg[S - 1] + 4] = G0 + 3                                           # invalid count in the last segment
    dev = "cuda"
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(dev)
    delta = torch.full((N,), -1, dtype=torch.int32, device=dev)
    G = torch.full((N,), -1, dtype=torch.int32, device=dev)
    off = torch.full((N + 1,), -1, dtype=torch.int64, device=dev)
    info = torch.zeros(S * hora.INFO_BYTES, dtype=torch.uint8, device=dev)
    ws = torch.empty(hora.hora_allocate_batched_workspace_bytes(N, S), dtype=torch.uint8, device=dev)
    hora.hora_allocate_batched(None, None, 1.0, 1.0, t(c), G0, t(cap), 0, N, ld, seg, budgets, hora.FLAG_HARD_FIRST, delta, G,
                               off, info, ws)
    torch.cuda.synchronize()
    d, infos = delta.cpu().numpy(), hora.read_infos(info, S)
    exp = np.zeros(N, np.int32)
    for s in range(S):
        sl = slice(int(seg[s]), int(seg[s + 1]))
        if s == S - 2:
            assert infos[s].status == 3
        elif s == S - 1:
            assert infos[s].status == 2
        else:
            assert infos[s].status == 0
            exp[sl] = hf.hard_first([int(x) for x in c[sl]], [int(x) for x in cap[sl]], int(budgets[s]))
            assert infos[s].n_above + infos[s].n_tied_taken == budgets[s] and infos[s].sum_cap == int(cap[sl].sum())
    np.testing.assert_array_equal(d, exp)
    Gx = np.where(np.repeat([i.status == 0 for i in infos], sizes), G0 + exp, 0)
    np.testing.assert_array_equal(G.cpu().numpy(), Gx)
    np.testing.assert_array_equal(off.cpu().numpy(), np.concatenate(([0], np.cumsum(Gx.astype(np.int64)))))
