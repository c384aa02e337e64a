"""hora_allocate_static: the allocation entry point that brings its own scratch.

Some callers of this library are not allowed to allocate device memory when they need the allocation
(plug-ins that only receive input and output buffers, code running where the allocator is frozen, services
that size all device memory up front).  hora_allocate_static serves them from a fixed array inside the
library.  This test drives it through the C ABI, twice in a row on different problems, and requires the same
Delta, G, offsets and summary as hora_allocate with a caller-provided workspace: bit-exact for the integer
outputs, and the same 1e-12 relative bound on objective and threshold that the parity tests use.  The second
call checks that nothing left in the shared scratch by the first one leaks into its result.

The file name sorts last on purpose: a run that stops at the first failure has then already run every other
test.
"""
from __future__ import annotations

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2605_07114_b200 import workloads as wl  # noqa: E402


def _run_both(w, B=None):
    from paper_2605_07114_b200 import hora
    dev = "cuda"
    B = w.B if B is None else B
    t = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    alpha, beta, c, cap = t(w.alpha), t(w.beta), t(w.c), t(w.cap)
    flags = hora.FLAG_EXACT_INT if w.exact_int else 0
    gains = torch.empty((w.N, w.ld), dtype=torch.float64, device=dev)
    hora.hora_gains(alpha, beta, w.alpha0, w.beta0, c, w.G0, cap, 0, w.N, w.ld, gains)

    def outputs():
        return (torch.full((w.N,), -1, dtype=torch.int32, device=dev), torch.full((w.N,), -1, dtype=torch.int32, device=dev),
                torch.full((w.N + 1,), -1, dtype=torch.int64, device=dev), torch.zeros(hora.INFO_BYTES, dtype=torch.uint8, device=dev))

    d0, G0_, off0, info0 = outputs()
    ws = torch.empty(hora.hora_allocate_workspace_bytes(w.N, w.ld, False, flags), dtype=torch.uint8, device=dev)
    hora.hora_allocate(alpha, beta, w.alpha0, w.beta0, c, w.G0, cap, 0, w.N, w.ld, gains, B, flags, d0, G0_, off0, info0, ws)
    d1, G1, off1, info1 = outputs()
    hora.hora_allocate_static(alpha, beta, w.alpha0, w.beta0, c, w.G0, cap, 0, w.N, w.ld, gains, B, flags, d1, G1, off1, info1)
    torch.cuda.synchronize()
    a, b = hora.read_info(info0), hora.read_info(info1)
    assert a.status == 0 and b.status == 0
    assert torch.equal(d0, d1) and torch.equal(G0_, G1) and torch.equal(off0, off1)
    assert int(d1.sum().item()) == B
    assert (a.n_above, a.n_tied, a.n_tied_taken, a.sum_G, a.sum_cap) == (b.n_above, b.n_tied, b.n_tied_taken, b.sum_G, b.sum_cap)
    assert abs(a.objective - b.objective) <= 1e-12 * abs(a.objective)
    assert abs(a.lambda_ - b.lambda_) <= 1e-12 * abs(a.lambda_)


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    _run_both(wl.make("cfg1"))                 # integer priors, exact tie path, N = 512
    _run_both(wl.make("cfg2", 4096))           # real priors, a larger problem that overwrites the same scratch
    _run_both(wl.make("cfg1"), B=777)          # and back to the first shape with another budget


def test_static_scratch_serves_the_rank_route_at_sizes_no_matrix_would_fit():
    """One integer prior, exact ties, no matrix: the route that builds none needs well under the built-in 8 MiB even
    for 2^18 prompts (a matrix of that problem would take 128 MiB).  Twice in a row, against the workspace call."""
    from paper_2605_07114_b200 import hora
    dev = "cuda"
    flags = hora.FLAG_EXACT_INT | hora.FLAG_SHARED_INT_PRIOR
    for N, B_per in ((1 << 18, 3), (100_001, 2)):
        w = wl.make("cfg5", N)
        c, cap = torch.from_numpy(w.c).to(dev), torch.from_numpy(w.cap).to(dev)
        assert hora.hora_allocate_workspace_bytes(N, w.ld, True, flags) <= hora.hora_allocate_static_capacity()
        res = []
        for static in (False, True):
            d = torch.full((N,), -1, dtype=torch.int32, device=dev)
            G = torch.full((N,), -1, dtype=torch.int32, device=dev)
            off = torch.full((N + 1,), -1, dtype=torch.int64, device=dev)
            info = torch.zeros(hora.INFO_BYTES, dtype=torch.uint8, device=dev)
            if static:
                hora.hora_allocate_static(None, None, 1.0, 1.0, c, w.G0, cap, 0, N, w.ld, None, B_per * N, flags, d, G, off, info)
            else:
                ws = torch.empty(hora.hora_allocate_workspace_bytes(N, w.ld, True, flags), dtype=torch.uint8, device=dev)
                hora.hora_allocate(None, None, 1.0, 1.0, c, w.G0, cap, 0, N, w.ld, None, B_per * N, flags, d, G, off, info, ws)
            torch.cuda.synchronize()
            res.append((d, G, off, hora.read_info(info)))
        (d0, G0_, off0, a), (d1, G1, off1, b) = res
        assert a.status == 0 and b.status == 0 and a.first_pass_bits == -1 and b.first_pass_bits == -1
        assert torch.equal(d0, d1) and torch.equal(G0_, G1) and torch.equal(off0, off1) and int(d1.sum()) == B_per * N
        assert (a.n_above, a.n_tied, a.n_tied_taken, a.lambda_, a.objective) == (b.n_above, b.n_tied, b.n_tied_taken, b.lambda_, b.objective)


def test_static_scratch_rejects_problems_beyond_its_capacity():
    from paper_2605_07114_b200 import hora
    N, ld = 1 << 20, 256
    assert hora.hora_allocate_workspace_bytes(N, ld, False, 0) > hora.hora_allocate_static_capacity()
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(hora.HoraError) as e:     # refused from the sizes alone: the buffers are never touched
        hora.hora_allocate_static(None, None, 1.0, 1.0, z, 8, None, ld, N, ld, None, 10, 0, z, z, None, None)
    assert e.value.code == hora.ERR_WORKSPACE
