"""Parity at the full sizes of the named workloads, in the launch configuration the benchmark times
(materialised gains, the Allocator's buffers): cfg4 (N = 2^20, real priors), cfg5 (N = 2^22, tie-heavy,
exact), cfg3's token layout (2.7e8 tokens).  The oracle runs in full on the host (tens of seconds)."""
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


def test_cfg4_full_size():
    gu = _gu()
    from paper_2605_07114_b200 import hora
    w = wl.make("cfg4")
    d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
    al = hora.Allocator(w.N, w.ld, w.G0, exact_int=False)
    dev = gu.dev
    al.run(dev(w.alpha), dev(w.beta), 1.0, 1.0, dev(w.c), None, w.ld, w.B)
    torch.cuda.synchronize()
    info = al.read_info()
    d, G, off = al.delta.cpu().numpy(), al.G.cpu().numpy(), al.group_offsets.cpu().numpy()
    gu.assert_allocation_matches(w, d, G, off, info, d_o, lam_o, obj_o)
    # gain rows: sampled rows against the long-double oracle
    rows = np.random.default_rng(0).choice(w.N, 512, replace=False)
    got = al.gains[torch.from_numpy(rows).to("cuda")].cpu().numpy()
    exp = orc.gains(w.alpha[rows], w.beta[rows], 1.0, 1.0, w.c[rows], w.G0, w.cap[rows], w.ld)
    assert (np.abs(got - exp) / exp).max() <= 4 * w.ld * 2.0 ** -53
    # exchange certificate at full size (Eq. appendix-exchange-condition) from the GPU's own gain matrix
    g = al.gains
    idx = torch.arange(w.N, device="cuda")
    dd = al.delta.long()
    taken_min = g[idx[dd > 0], dd[dd > 0] - 1].min().item()
    nxt_max = g[idx[dd < w.ld], dd[dd < w.ld]].max().item()
    assert taken_min >= nxt_max
    # advantages over the resulting groups
    rewards = w.rewards(off)
    got_adv, status = gu.gpu_advantage(rewards, off, w.adv_mode, np.float32(w.eps), w.ddof)
    exp_adv = orc.group_advantage(rewards, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
    assert status == 0
    assert np.abs(got_adv - exp_adv).max() <= 1e-5


def test_cfg5_full_size_tie_heavy_exact():
    gu = _gu()
    w = wl.make("cfg5")
    d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
    d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B, exact=True)
    gu.assert_allocation_matches(w, d, G, off, info, d_o, lam_o, obj_o)
    assert info.n_tied > 1_000_000 and 0 < info.n_tied_taken < info.n_tied      # the threshold sits in a mass tie
    rewards = w.rewards(off)
    got_adv, status = gu.gpu_advantage(rewards, off, w.adv_mode, np.float32(w.eps), w.ddof)
    exp_adv = orc.group_advantage(rewards, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
    assert status == 0
    assert np.abs(got_adv - exp_adv).max() <= 1e-5


def test_cfg3_full_size_token_broadcast():
    gu = _gu()
    w = wl.make("cfg3")
    d_o, G_o, lam_o, obj_o = gu.oracle_allocate(w)
    d, G, off, info = gu.gpu_allocate(None, None, 1.0, 1.0, w.c, w.G0, w.cap, w.ld, w.B, exact=True)
    gu.assert_allocation_matches(w, d, G, off, info, d_o, lam_o, obj_o)
    rewards = w.rewards(off)
    adv = orc.group_advantage(rewards, off, w.adv_mode, float(np.float32(w.eps)), w.ddof)
    got_adv, _ = gu.gpu_advantage(rewards, off, w.adv_mode, np.float32(w.eps), w.ddof)
    assert np.abs(got_adv - adv).max() <= 1e-5
    tok = w.token_offsets(len(rewards))
    assert tok[-1] > 2.6e8
    got = gu.gpu_broadcast(adv, tok)
    exp = orc.token_broadcast(adv, tok)
    assert np.array_equal(got.view(np.uint32), exp.view(np.uint32))
