"""Helpers shared by the GPU parity tests: run a workload through the C-ABI path and through the oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import hora_oracle as orc
from paper_2605_07114_b200 import hora

DEV = "cuda"


def dev(a, dtype=None):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(DEV)


def gpu_gains(alpha, beta, alpha0, beta0, c, G0, cap, ld, cap_scalar=None):
    N = len(c)
    out = torch.full((N, ld), -7.0, dtype=torch.float64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    hora.hora_gains(dev(alpha), dev(beta), alpha0, beta0, dev(c), G0, None if cap is None else dev(cap),
                    0 if cap_scalar is None else cap_scalar, N, ld, out, status)
    torch.cuda.synchronize()
    return out.cpu().numpy(), int(status.item())


def gpu_allocate(alpha, beta, alpha0, beta0, c, G0, cap, ld, B, *, exact, materialise=True, cap_scalar=None,
                 skip_objective=False, shared_int_prior=False):
    """Returns (delta, G, offsets, info).  shared_int_prior sizes the workspace for the rank-based route only."""
    N = len(c)
    al = hora.Allocator(N, ld, G0, exact_int=exact, materialise=materialise, skip_objective=skip_objective,
                        shared_int_prior=shared_int_prior)
    al.delta.fill_(-1)
    al.G.fill_(-1)
    al.group_offsets.fill_(-1)
    al.run(dev(alpha), dev(beta), alpha0, beta0, dev(c), None if cap is None else dev(cap),
           0 if cap_scalar is None else cap_scalar, B)
    torch.cuda.synchronize()
    return al.delta.cpu().numpy(), al.G.cpu().numpy(), al.group_offsets.cpu().numpy(), al.read_info()


def gpu_advantage(rewards, off, mode, eps, ddof):
    N = len(off) - 1
    r = dev(rewards)
    out = torch.full_like(r, 123.0)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    hora.hora_group_advantage(r, dev(off), N, mode, eps, ddof, out, status)
    torch.cuda.synchronize()
    return out.cpu().numpy(), int(status.item())


def gpu_broadcast(adv, tok_off, misalign=0):
    R = len(adv)
    T = int(tok_off[-1])
    buf = torch.full((T + 8 + misalign,), float("nan"), dtype=torch.float32, device=DEV)
    out = buf[misalign:misalign + T]
    hora.hora_token_broadcast(dev(adv), dev(tok_off), R, T, out)
    torch.cuda.synchronize()
    guard = buf[misalign + T:].cpu().numpy()
    assert np.isnan(guard).all(), "wrote past the end"
    if misalign:
        assert np.isnan(buf[:misalign].cpu().numpy()).all(), "wrote before the start"
    return out.cpu().numpy()


def oracle_allocate(w):
    if w.exact_int:
        d, G, lam, obj = orc.greedy_exact(w.alpha, w.beta, w.alpha0, w.beta0, w.c, w.G0, w.cap, w.B)
        lam = lam[0] / lam[1] if lam[1] else 0.0
    else:
        d, G, lam, obj = orc.greedy_real(w.alpha, w.beta, w.alpha0, w.beta0, w.c, w.G0, w.cap, w.B)
    return d, G, lam, obj


def posterior_ab(w):
    al = np.full(w.N, w.alpha0) if w.alpha is None else w.alpha
    be = np.full(w.N, w.beta0) if w.beta is None else w.beta
    return al + w.c, be + (w.G0 - w.c)


def assert_allocation_matches(w, d_gpu, G_gpu, off_gpu, info, d_orc, lam_orc, obj_orc, band=1e-12):
    """Bit-exact for integer priors; for real priors Delta may differ only on candidates whose oracle
    gain is within ``band`` (relative) of the oracle threshold.  Objective within 1e-12 relative."""
    assert info.status == 0, hora.status_string(info.status)
    assert int(d_gpu.astype(np.int64).sum()) == w.B
    assert (d_gpu >= 0).all() and (d_gpu <= w.cap).all()
    np.testing.assert_array_equal(G_gpu, w.G0 + d_gpu)
    exp_off = np.zeros(w.N + 1, np.int64)
    np.cumsum(G_gpu.astype(np.int64), out=exp_off[1:])
    np.testing.assert_array_equal(off_gpu, exp_off)
    if w.exact_int:
        np.testing.assert_array_equal(d_gpu, d_orc)
    else:
        diff = np.nonzero(d_gpu != d_orc)[0]
        a, b = posterior_ab(w)
        for i in diff:
            lo, hi = sorted((int(d_gpu[i]), int(d_orc[i])))
            for D in range(lo + 1, hi + 1):
                g = orc.gain_one(float(a[i]), float(b[i]), D)
                assert abs(g - lam_orc) <= band * lam_orc, (i, D, g, lam_orc)
    if w.B > 0:
        assert abs(info.objective - obj_orc) <= 1e-12 * abs(obj_orc)
        assert abs(info.lambda_ - lam_orc) <= 1e-12 * lam_orc
    assert info.sum_G == w.N * w.G0 + w.B
    assert info.sum_cap == int(w.cap.astype(np.int64).sum())
    assert info.n_above + info.n_tied_taken == w.B
    assert 0 <= info.n_tied_taken <= info.n_tied
