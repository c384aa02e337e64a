"""ctypes front end of the C oracle (``hora_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Nothing here is imported by the product package; the tests, the smoke check and the
benchmark's CPU-baseline leg are the only callers.  Arrays are numpy, on the host.
Parity pins for every function live in ``tests/test_oracle_pins.py``.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Tuple

import numpy as np

from . import build as _build

OK, BAD_ARG, INFEASIBLE, NOT_INTEGER, OVERFLOW, NOMEM = range(6)
GRPO, RLOO = 0, 1


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__({1: "bad argument", 2: "infeasible: B > sum(cap)", 3: "prior is not integer-valued",
                          4: "exact arithmetic overflowed 128 bits", 5: "out of memory"}.get(code, f"code {code}"))
        self.code = code


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        p = C.c_void_p
        L.oracle_gains.argtypes = [p, p, C.c_double, C.c_double, p, C.c_int32, p, C.c_int64, C.c_int32, p]
        L.oracle_gain_one.argtypes = [C.c_double, C.c_double, C.c_int32]
        L.oracle_gain_one.restype = C.c_double
        L.oracle_utility_one.argtypes = [C.c_double, C.c_double, C.c_int32]
        L.oracle_utility_one.restype = C.c_double
        L.oracle_greedy_real.argtypes = [p, p, C.c_double, C.c_double, p, C.c_int32, p, C.c_int64, C.c_int64,
                                         p, p, p, p]
        L.oracle_greedy_exact.argtypes = [p, p, C.c_double, C.c_double, p, C.c_int32, p, C.c_int64, C.c_int64,
                                          p, p, p, p, p]
        L.oracle_group_advantage.argtypes = [p, p, C.c_int64, C.c_int32, C.c_double, C.c_int32, p]
        L.oracle_token_broadcast.argtypes = [p, p, C.c_int64, p]
        L.oracle_rollout_weights.argtypes = [p, C.c_int64, p, C.c_int32, C.c_double, p]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _prior(alpha, beta, N):
    if alpha is None:
        return None, None
    alpha = np.ascontiguousarray(alpha, dtype=np.float64)
    beta = np.ascontiguousarray(beta, dtype=np.float64)
    assert alpha.shape == (N,) and beta.shape == (N,)
    return alpha, beta


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


def gains(alpha, beta, alpha0, beta0, c, G0, cap, ld) -> np.ndarray:
    """Rows g_i(1..ld) by the paper's recurrence in long double; entries past cap_i are 0."""
    c = np.ascontiguousarray(c, dtype=np.int32)
    cap = np.ascontiguousarray(cap, dtype=np.int32)
    N = c.shape[0]
    alpha, beta = _prior(alpha, beta, N)
    out = np.empty((N, ld), dtype=np.float64)
    _check(lib().oracle_gains(_ptr(alpha), _ptr(beta), alpha0, beta0, _ptr(c), G0, _ptr(cap), N, ld, _ptr(out)))
    return out


def gain_one(a: float, b: float, Delta: int) -> float:
    return lib().oracle_gain_one(a, b, Delta)


def utility_one(a: float, b: float, Delta: int) -> float:
    return lib().oracle_utility_one(a, b, Delta)


def greedy_real(alpha, beta, alpha0, beta0, c, G0, cap, B) -> Tuple[np.ndarray, np.ndarray, float, float]:
    """Heap greedy in long double.  Returns (Delta, G, lambda = last gain handed out, objective)."""
    c = np.ascontiguousarray(c, dtype=np.int32)
    cap = np.ascontiguousarray(cap, dtype=np.int32)
    N = c.shape[0]
    alpha, beta = _prior(alpha, beta, N)
    delta = np.zeros(N, dtype=np.int32)
    G = np.zeros(N, dtype=np.int32)
    lam = C.c_double(0.0)
    obj = C.c_double(0.0)
    _check(lib().oracle_greedy_real(_ptr(alpha), _ptr(beta), alpha0, beta0, _ptr(c), G0, _ptr(cap), N, int(B),
                                    _ptr(delta), _ptr(G), C.addressof(lam), C.addressof(obj)))
    return delta, G, lam.value, obj.value


def greedy_exact(alpha, beta, alpha0, beta0, c, G0, cap, B):
    """Heap greedy on exact rationals (integer-valued priors).

    Returns (Delta, G, (lambda_num, lambda_den) as Python ints, objective)."""
    c = np.ascontiguousarray(c, dtype=np.int32)
    cap = np.ascontiguousarray(cap, dtype=np.int32)
    N = c.shape[0]
    alpha, beta = _prior(alpha, beta, N)
    delta = np.zeros(N, dtype=np.int32)
    G = np.zeros(N, dtype=np.int32)
    num = (C.c_uint64 * 2)()
    den = (C.c_uint64 * 2)()
    obj = C.c_double(0.0)
    _check(lib().oracle_greedy_exact(_ptr(alpha), _ptr(beta), alpha0, beta0, _ptr(c), G0, _ptr(cap), N, int(B),
                                     _ptr(delta), _ptr(G), C.addressof(num), C.addressof(den), C.addressof(obj)))
    return delta, G, (num[0] | (num[1] << 64), den[0] | (den[1] << 64)), obj.value


def group_advantage(rewards, off, mode: int, eps: float, ddof: int) -> np.ndarray:
    rewards = np.ascontiguousarray(rewards, dtype=np.float32)
    off = np.ascontiguousarray(off, dtype=np.int64)
    out = np.zeros_like(rewards)
    _check(lib().oracle_group_advantage(_ptr(rewards), _ptr(off), off.shape[0] - 1, mode, float(eps), ddof, _ptr(out)))
    return out


def token_broadcast(adv, tok_off) -> np.ndarray:
    adv = np.ascontiguousarray(adv, dtype=np.float32)
    tok_off = np.ascontiguousarray(tok_off, dtype=np.int64)
    out = np.empty(int(tok_off[-1]), dtype=np.float32)
    _check(lib().oracle_token_broadcast(_ptr(adv), _ptr(tok_off), adv.shape[0], _ptr(out)))
    return out


def rollout_weights(goff, toff, mode: int, length_const: float = 1.0) -> np.ndarray:
    """Loss weight per rollout: 1/(G_g len_r) (mode 0) or 1/(G_g length_const) (mode 1)."""
    goff = np.ascontiguousarray(goff, dtype=np.int64)
    toff = None if toff is None else np.ascontiguousarray(toff, dtype=np.int64)
    out = np.zeros(int(goff[-1]), dtype=np.float32)
    _check(lib().oracle_rollout_weights(_ptr(goff), goff.shape[0] - 1, _ptr(toff), mode, float(length_const), _ptr(out)))
    return out
