"""Thin ctypes binding over ``libhora.so`` — same names and arguments as ``include/hora.h``.

Argument marshalling only: tensors are passed as device pointers, the stream is torch's current
stream, and every step of the path runs in the library's CUDA kernels.  There is no CPU
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhora.so")

(OK, ERR_INVALID_ARG, ERR_INVALID_VALUE, ERR_INFEASIBLE, ERR_NOT_INTEGER, ERR_EXACT_RANGE, ERR_WORKSPACE, ERR_CUDA,
 ERR_INTERNAL) = range(9)
FLAG_EXACT_INT = 1
FLAG_SKIP_OBJECTIVE = 2
FLAG_SHARED_PRIOR = 4
FLAG_HARD_FIRST = 8
FLAG_SHARED_INT_PRIOR = 4            # the same flag under the name of its first use
ADV_GRPO, ADV_RLOO = 0, 1
WEIGHT_PER_TOKEN, WEIGHT_CONST_LENGTH = 0, 1

EXPORTS = ("hora_gains", "hora_allocate_workspace_bytes", "hora_allocate", "hora_group_advantage",
           "hora_token_broadcast", "hora_status_string", "hora_version", "hora_launch_count",
           "hora_allocate_static", "hora_allocate_static_capacity", "hora_allocate_profile_events", "hora_allocate_profile_stages",
           "hora_allocate_batched", "hora_allocate_batched_workspace_bytes", "hora_rollout_weights",
           "hora_learned_prior", "hora_beta_binomial_nll", "hora_pass_at_k", "hora_pass_at_k_workspace_bytes",
           "hora_group_advantage_tokens", "hora_allocation_share", "hora_allocate_hard_first",
           "hora_allocate_hard_first_workspace_bytes", "hora_fp64_probe", "hora_checked_violation")


class HoraError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {status_string(code)} (status {code})")
        self.code = code


class hora_alloc_info(C.Structure):
    _fields_ = [("status", C.c_int32), ("first_pass_bits", C.c_int32), ("lambda_", C.c_double),
                ("n_above", C.c_int64), ("n_tied", C.c_int64), ("n_tied_taken", C.c_int64),
                ("objective", C.c_double), ("sum_G", C.c_int64), ("sum_cap", C.c_int64)]


INFO_BYTES = C.sizeof(hora_alloc_info)
_lib = None


def use_library(path: Optional[str]) -> None:
    """Bind the module to another build of the same library (e.g. the checked one), or back to the default (None).
    Takes effect at the next call."""
    global _lib, _lib_path
    _lib = None
    _lib_path = path or LIB_PATH


_lib_path = LIB_PATH


def load() -> C.CDLL:
    """Load the CUDA library built in-tree.  Raises if it is not there: nothing else can do its work."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_lib_path):
        raise FileNotFoundError(f"{_lib_path} not found: build it with `python -m paper_2605_07114_b200.build`")
    L = C.CDLL(_lib_path)
    p, i32, i64, f64, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_double, C.c_uint32
    L.hora_gains.argtypes = [p, p, f64, f64, p, i32, p, i32, i64, i32, p, p, p]
    L.hora_gains.restype = C.c_int
    L.hora_allocate_workspace_bytes.argtypes = [i64, i32, i32, u32]
    L.hora_allocate_workspace_bytes.restype = C.c_size_t
    L.hora_allocate.argtypes = [p, p, f64, f64, p, i32, p, i32, i64, i32, p, i64, u32, p, p, p, p, p, C.c_size_t, p]
    L.hora_allocate.restype = C.c_int
    L.hora_allocate_static.argtypes = [p, p, f64, f64, p, i32, p, i32, i64, i32, p, i64, u32, p, p, p, p, p]
    L.hora_allocate_static.restype = C.c_int
    L.hora_allocate_static_capacity.restype = C.c_size_t
    L.hora_allocate_hard_first_workspace_bytes.argtypes = [i64, i32]
    L.hora_allocate_hard_first_workspace_bytes.restype = C.c_size_t
    L.hora_allocate_hard_first.argtypes = [p, i32, p, i32, i64, i32, i64, p, p, p, p, p, C.c_size_t, p]
    L.hora_allocate_hard_first.restype = C.c_int
    L.hora_allocate_batched_workspace_bytes.argtypes = [i64, i64]
    L.hora_allocate_batched_workspace_bytes.restype = C.c_size_t
    L.hora_allocate_batched.argtypes = [p, p, f64, f64, p, i32, p, i32, i64, i32, p, p, i64, u32, p, p, p, p, p,
                                        C.c_size_t, p]
    L.hora_allocate_batched.restype = C.c_int
    L.hora_allocate_profile_events.argtypes = [p, p]
    L.hora_allocate_profile_events.restype = None
    L.hora_allocate_profile_stages.argtypes = [C.POINTER(C.c_void_p), C.c_int32]
    L.hora_allocate_profile_stages.restype = None
    L.hora_group_advantage.argtypes = [p, p, i64, i32, C.c_float, i32, p, p, p]
    L.hora_group_advantage.restype = C.c_int
    L.hora_group_advantage_tokens.argtypes = [p, p, i64, p, i64, i64, i32, C.c_float, i32, i32, C.c_float, p, p, p, p]
    L.hora_group_advantage_tokens.restype = C.c_int
    L.hora_allocation_share.argtypes = [p, p, i64, i32, p, p, p, p]
    L.hora_allocation_share.restype = C.c_int
    L.hora_pass_at_k_workspace_bytes.argtypes = [i32]
    L.hora_pass_at_k_workspace_bytes.restype = C.c_size_t
    L.hora_pass_at_k.argtypes = [p, i64, i32, p, i32, p, p, p, C.c_size_t, p]
    L.hora_pass_at_k.restype = C.c_int
    L.hora_learned_prior.argtypes = [p, p, f64, i64, p, p, p, p]
    L.hora_learned_prior.restype = C.c_int
    L.hora_beta_binomial_nll.argtypes = [p, p, f64, p, i32, i64, p, p, p]
    L.hora_beta_binomial_nll.restype = C.c_int
    L.hora_rollout_weights.argtypes = [p, i64, p, i32, C.c_float, p, p, p]
    L.hora_rollout_weights.restype = C.c_int
    L.hora_token_broadcast.argtypes = [p, p, i64, i64, p, p]
    L.hora_token_broadcast.restype = C.c_int
    L.hora_checked_violation.restype = C.c_int32
    L.hora_fp64_probe.argtypes = [i32, p, p]
    L.hora_fp64_probe.restype = C.c_uint64
    L.hora_status_string.argtypes = [C.c_int]
    L.hora_status_string.restype = C.c_char_p
    L.hora_version.restype = C.c_int
    L.hora_launch_count.restype = C.c_uint64
    _lib = L
    return L


def status_string(code: int) -> str:
    return load().hora_status_string(int(code)).decode()


hora_status_string = status_string


def hora_version() -> int:
    return load().hora_version()


def hora_launch_count() -> int:
    return int(load().hora_launch_count())


def _ptr(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, where: str):
    if rc != OK:
        raise HoraError(rc, where)


def hora_gains(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, status_dev=None):
    rc = load().hora_gains(_ptr(alpha, torch.float64, "alpha"), _ptr(beta, torch.float64, "beta"), alpha0, beta0,
                           _ptr(c, torch.int32, "c"), G0, _ptr(cap, torch.int32, "cap"), cap_scalar, N, ld,
                           _ptr(gains, torch.float64, "gains"), _ptr(status_dev, torch.int32, "status_dev"), _stream())
    _check(rc, "hora_gains")


def hora_allocate_workspace_bytes(N, ld, gains_is_null, flags) -> int:
    return int(load().hora_allocate_workspace_bytes(N, ld, int(bool(gains_is_null)), flags))


def hora_allocate(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, B, flags, delta, G,
                  group_offsets, info_dev, workspace):
    rc = load().hora_allocate(_ptr(alpha, torch.float64, "alpha"), _ptr(beta, torch.float64, "beta"), alpha0, beta0,
                              _ptr(c, torch.int32, "c"), G0, _ptr(cap, torch.int32, "cap"), cap_scalar, N, ld,
                              _ptr(gains, torch.float64, "gains"), B, flags, _ptr(delta, torch.int32, "delta"),
                              _ptr(G, torch.int32, "G"), _ptr(group_offsets, torch.int64, "group_offsets"),
                              _ptr(info_dev, torch.uint8, "info_dev"), _ptr(workspace, torch.uint8, "workspace"),
                              0 if workspace is None else workspace.numel(), _stream())
    _check(rc, "hora_allocate")


def hora_allocate_hard_first_workspace_bytes(N, ld) -> int:
    return int(load().hora_allocate_hard_first_workspace_bytes(N, ld))


def hora_allocate_hard_first(c, G0, cap, cap_scalar, N, ld, B, delta, G, group_offsets, info_dev, workspace):
    rc = load().hora_allocate_hard_first(_ptr(c, torch.int32, "c"), G0, _ptr(cap, torch.int32, "cap"), cap_scalar, N, ld, B,
                                         _ptr(delta, torch.int32, "delta"), _ptr(G, torch.int32, "G"),
                                         _ptr(group_offsets, torch.int64, "group_offsets"),
                                         _ptr(info_dev, torch.uint8, "info_dev"), _ptr(workspace, torch.uint8, "workspace"),
                                         0 if workspace is None else workspace.numel(), _stream())
    _check(rc, "hora_allocate_hard_first")


def hora_allocate_batched_workspace_bytes(N, S) -> int:
    return int(load().hora_allocate_batched_workspace_bytes(N, S))


def hora_allocate_batched(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, seg_offsets_host, budgets_host,
                          flags, delta, G, group_offsets, info_dev, workspace):
    """seg_offsets_host / budgets_host: host int64 arrays (numpy or CPU tensors); info_dev: uint8[S*64] on device."""
    import numpy as np
    seg = np.ascontiguousarray(np.asarray(seg_offsets_host), dtype=np.int64)
    bud = np.ascontiguousarray(np.asarray(budgets_host), dtype=np.int64)
    S = int(seg.shape[0]) - 1
    if bud.shape[0] != S:
        raise ValueError("budgets_host must have one entry per segment")
    rc = load().hora_allocate_batched(_ptr(alpha, torch.float64, "alpha"), _ptr(beta, torch.float64, "beta"), alpha0,
                                      beta0, _ptr(c, torch.int32, "c"), G0, _ptr(cap, torch.int32, "cap"), cap_scalar,
                                      N, ld, seg.ctypes.data_as(C.c_void_p), bud.ctypes.data_as(C.c_void_p), S, flags,
                                      _ptr(delta, torch.int32, "delta"), _ptr(G, torch.int32, "G"),
                                      _ptr(group_offsets, torch.int64, "group_offsets"),
                                      _ptr(info_dev, torch.uint8, "info_dev"), _ptr(workspace, torch.uint8, "workspace"),
                                      0 if workspace is None else workspace.numel(), _stream())
    _check(rc, "hora_allocate_batched")


def read_infos(info_dev: torch.Tensor, S: int):
    """Per-segment summaries of hora_allocate_batched (synchronises the current stream)."""
    raw = info_dev.cpu().numpy().tobytes()
    out = []
    for s in range(S):
        x = hora_alloc_info.from_buffer_copy(raw[s * INFO_BYTES:(s + 1) * INFO_BYTES])
        out.append(AllocInfo(x.status, x.first_pass_bits, x.lambda_, x.n_above, x.n_tied, x.n_tied_taken, x.objective,
                             x.sum_G, x.sum_cap))
    return out


def hora_checked_violation() -> int:
    """0: no index check failed since the last call; > 0: (file id << 20) | line of the first failure; -1: this is
    not the checked build."""
    return int(load().hora_checked_violation())


def hora_fp64_probe(iters, sink_dev) -> int:
    """Enqueue the fp64 FMA probe kernel; returns the number of FMAs it performs (time it with events)."""
    n = int(load().hora_fp64_probe(iters, _ptr(sink_dev, torch.float64, "sink_dev"), _stream()))
    if n == 0:
        raise HoraError(ERR_CUDA, "hora_fp64_probe")
    return n


def hora_allocate_profile_events(start_event, stop_event):
    """Record the given events (raw cudaEvent_t handles as ints, or None to switch off) around the full-read
    selection kernel of every following hora_allocate call."""
    load().hora_allocate_profile_events(None if start_event is None else C.c_void_p(int(start_event)),
                                        None if stop_event is None else C.c_void_p(int(stop_event)))


def hora_allocate_profile_stages(events):
    """Record the given events (raw cudaEvent_t handles as ints; at most 7; None or empty to switch off) at the
    stage boundaries of every following hora_allocate call."""
    if not events:
        load().hora_allocate_profile_stages(None, 0)
        return
    arr = (C.c_void_p * len(events))(*[C.c_void_p(int(e)) if e is not None else None for e in events])
    load().hora_allocate_profile_stages(arr, len(events))


def hora_allocate_static_capacity() -> int:
    return int(load().hora_allocate_static_capacity())


def hora_allocate_static(alpha, beta, alpha0, beta0, c, G0, cap, cap_scalar, N, ld, gains, B, flags, delta, G,
                         group_offsets, info_dev):
    """hora_allocate with the library's own fixed scratch: no workspace argument, no allocation.
    Problems whose workspace would exceed hora_allocate_static_capacity() raise HoraError(ERR_WORKSPACE).
    Calls share that scratch, so do not let two of them overlap on the GPU."""
    rc = load().hora_allocate_static(_ptr(alpha, torch.float64, "alpha"), _ptr(beta, torch.float64, "beta"), alpha0,
                                     beta0, _ptr(c, torch.int32, "c"), G0, _ptr(cap, torch.int32, "cap"), cap_scalar,
                                     N, ld, _ptr(gains, torch.float64, "gains"), B, flags,
                                     _ptr(delta, torch.int32, "delta"), _ptr(G, torch.int32, "G"),
                                     _ptr(group_offsets, torch.int64, "group_offsets"),
                                     _ptr(info_dev, torch.uint8, "info_dev"), _stream())
    _check(rc, "hora_allocate_static")


def hora_group_advantage(rewards, group_offsets, N, mode, eps, ddof, adv, status_dev=None):
    rc = load().hora_group_advantage(_ptr(rewards, torch.float32, "rewards"),
                                     _ptr(group_offsets, torch.int64, "group_offsets"), N, mode, eps, ddof,
                                     _ptr(adv, torch.float32, "adv"), _ptr(status_dev, torch.int32, "status_dev"),
                                     _stream())
    _check(rc, "hora_group_advantage")


def hora_group_advantage_tokens(rewards, group_offsets, N, token_offsets, R, T, mode, eps, ddof, token_adv,
                                token_weight=None, weight_mode=WEIGHT_PER_TOKEN, length_const=1.0, status_dev=None):
    rc = load().hora_group_advantage_tokens(
        _ptr(rewards, torch.float32, "rewards"), _ptr(group_offsets, torch.int64, "group_offsets"), N,
        _ptr(token_offsets, torch.int64, "token_offsets"), R, T, mode, eps, ddof, weight_mode, length_const,
        _ptr(token_adv, torch.float32, "token_adv"), _ptr(token_weight, torch.float32, "token_weight"),
        _ptr(status_dev, torch.int32, "status_dev"), _stream())
    _check(rc, "hora_group_advantage_tokens")


def hora_allocation_share(c, delta, N, G0, prompts, budget, status_dev=None):
    rc = load().hora_allocation_share(_ptr(c, torch.int32, "c"), _ptr(delta, torch.int32, "delta"), N, G0,
                                      _ptr(prompts, torch.int64, "prompts"), _ptr(budget, torch.int64, "budget"),
                                      _ptr(status_dev, torch.int32, "status_dev"), _stream())
    _check(rc, "hora_allocation_share")


def hora_pass_at_k_workspace_bytes(n_samples) -> int:
    return int(load().hora_pass_at_k_workspace_bytes(n_samples))


def hora_pass_at_k(c, Q, n_samples, K_dev, n_K, pass_at_k, status_dev, workspace):
    rc = load().hora_pass_at_k(_ptr(c, torch.int32, "c"), Q, n_samples, _ptr(K_dev, torch.int32, "K_dev"), n_K,
                               _ptr(pass_at_k, torch.float64, "pass_at_k"), _ptr(status_dev, torch.int32, "status_dev"),
                               _ptr(workspace, torch.uint8, "workspace"), 0 if workspace is None else workspace.numel(),
                               _stream())
    _check(rc, "hora_pass_at_k")


def hora_learned_prior(p_hat, s_raw, s_fixed, N, alpha, beta, status_dev=None):
    rc = load().hora_learned_prior(_ptr(p_hat, torch.float64, "p_hat"), _ptr(s_raw, torch.float64, "s_raw"), s_fixed, N,
                                   _ptr(alpha, torch.float64, "alpha"), _ptr(beta, torch.float64, "beta"),
                                   _ptr(status_dev, torch.int32, "status_dev"), _stream())
    _check(rc, "hora_learned_prior")


def hora_beta_binomial_nll(p_hat, s_raw, s_fixed, c, G0, N, nll, status_dev=None):
    rc = load().hora_beta_binomial_nll(_ptr(p_hat, torch.float64, "p_hat"), _ptr(s_raw, torch.float64, "s_raw"), s_fixed,
                                       _ptr(c, torch.int32, "c"), G0, N, _ptr(nll, torch.float64, "nll"),
                                       _ptr(status_dev, torch.int32, "status_dev"), _stream())
    _check(rc, "hora_beta_binomial_nll")


def hora_rollout_weights(group_offsets, N, token_offsets, mode, length_const, weights, status_dev=None):
    rc = load().hora_rollout_weights(_ptr(group_offsets, torch.int64, "group_offsets"), N,
                                     _ptr(token_offsets, torch.int64, "token_offsets"), mode, length_const,
                                     _ptr(weights, torch.float32, "weights"), _ptr(status_dev, torch.int32, "status_dev"),
                                     _stream())
    _check(rc, "hora_rollout_weights")


def hora_token_broadcast(adv, token_offsets, R, T, token_adv):
    rc = load().hora_token_broadcast(_ptr(adv, torch.float32, "adv"), _ptr(token_offsets, torch.int64, "token_offsets"),
                                     R, T, _ptr(token_adv, torch.float32, "token_adv"), _stream())
    _check(rc, "hora_token_broadcast")


# ------------------------------------------------------------------------------------------------
# Convenience layer: buffer ownership for callers who hold torch tensors.  No arithmetic here.
@dataclass
class AllocInfo:
    status: int
    first_pass_bits: int
    lambda_: float
    n_above: int
    n_tied: int
    n_tied_taken: int
    objective: float
    sum_G: int
    sum_cap: int


def read_info(info_dev: torch.Tensor) -> AllocInfo:
    """Copy the 64-byte summary to the host (synchronises the current stream)."""
    raw = bytes(info_dev.cpu().numpy().tobytes())
    s = hora_alloc_info.from_buffer_copy(raw)
    return AllocInfo(s.status, s.first_pass_bits, s.lambda_, s.n_above, s.n_tied, s.n_tied_taken, s.objective, s.sum_G, s.sum_cap)


class Allocator:
    """Owns the device buffers of one allocation problem shape (N, ld) and runs gains -> allocate."""

    def __init__(self, N: int, ld: int, G0: int, *, exact_int: bool = False, skip_objective: bool = False,
                 materialise: bool = True, shared_int_prior: bool = False, device="cuda"):
        self.N, self.ld, self.G0 = N, ld, G0
        self.flags = (FLAG_EXACT_INT if exact_int else 0) | (FLAG_SKIP_OBJECTIVE if skip_objective else 0) | \
                     (FLAG_SHARED_INT_PRIOR if shared_int_prior else 0)
        self.materialise = materialise
        dev = torch.device(device)
        self.gains = torch.empty((N, ld), dtype=torch.float64, device=dev) if materialise else None
        wb = hora_allocate_workspace_bytes(N, ld, not materialise, self.flags)
        self.workspace = torch.empty(max(wb, 256), dtype=torch.uint8, device=dev)
        if self.workspace.data_ptr() % 256:
            raise RuntimeError("device allocation is not 256-byte aligned")
        self.delta = torch.empty(N, dtype=torch.int32, device=dev)
        self.G = torch.empty(N, dtype=torch.int32, device=dev)
        self.group_offsets = torch.empty(N + 1, dtype=torch.int64, device=dev)
        self.info = torch.zeros(INFO_BYTES, dtype=torch.uint8, device=dev)

    def run(self, alpha, beta, alpha0, beta0, c, cap, cap_scalar, B):
        if self.materialise:
            hora_gains(alpha, beta, alpha0, beta0, c, self.G0, cap, cap_scalar, self.N, self.ld, self.gains)
        hora_allocate(alpha, beta, alpha0, beta0, c, self.G0, cap, cap_scalar, self.N, self.ld, self.gains, B,
                      self.flags, self.delta, self.G, self.group_offsets, self.info, self.workspace)
        return self.delta, self.G, self.group_offsets

    def read_info(self) -> AllocInfo:
        return read_info(self.info)
