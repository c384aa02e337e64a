"""The C-ABI library builds, loads without a GPU, and exports every function include/hora.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "hora.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b(hora_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_07114_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_four_calls():
    names = declared_functions()
    for must in ("hora_gains", "hora_allocate", "hora_group_advantage", "hora_token_broadcast",
                 "hora_allocate_workspace_bytes", "hora_status_string", "hora_version"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_names():
    from paper_2605_07114_b200 import hora
    assert sorted(hora.EXPORTS) == declared_functions()
    for name in hora.EXPORTS:
        assert callable(getattr(hora, name))


def test_host_only_entry_points(lib):
    lib.hora_status_string.restype = ctypes.c_char_p
    assert lib.hora_status_string(0) == b"ok"
    assert b"cap" in lib.hora_status_string(3)
    assert lib.hora_version() >= 100
    lib.hora_allocate_workspace_bytes.restype = ctypes.c_size_t
    lib.hora_allocate_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint32]
    small = lib.hora_allocate_workspace_bytes(1024, 64, 0, 0)
    with_gains = lib.hora_allocate_workspace_bytes(1024, 64, 1, 0)
    exact = lib.hora_allocate_workspace_bytes(1024, 64, 0, 1)
    assert small % 256 == 0 and small > 5 * 8192 * 8
    assert with_gains >= small + 1024 * 64 * 8
    assert exact > small
    assert lib.hora_allocate_workspace_bytes(-1, 64, 0, 0) == 0


def test_host_side_argument_checks_need_no_gpu(lib):
    """Bad sizes are refused before anything touches the device."""
    i64, i32, f64, p = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p
    lib.hora_gains.argtypes = [p, p, f64, f64, p, i32, p, i32, i64, i32, p, p, p]
    assert lib.hora_gains(None, None, 1.0, 1.0, None, 4, None, 8, -1, 8, None, None, None) == 1
    assert lib.hora_gains(None, None, 1.0, 1.0, None, 4, None, 8, 10, 0, None, None, None) == 1
    assert lib.hora_gains(None, None, -1.0, 1.0, None, 4, None, 8, 10, 8, None, None, None) == 1
    assert lib.hora_gains(None, None, 1.0, 1.0, None, 4, None, 9, 10, 8, None, None, None) == 1     # cap_scalar > ld
    assert lib.hora_gains(None, None, 1.0, 1.0, None, 4, None, 8, 0, 8, None, None, None) == 0      # N == 0: no-op
    lib.hora_token_broadcast.argtypes = [p, p, i64, i64, p, p]
    assert lib.hora_token_broadcast(None, None, -1, 0, None, None) == 1
    assert lib.hora_token_broadcast(None, None, 0, 0, None, None) == 0
    lib.hora_group_advantage.argtypes = [p, p, i64, i32, ctypes.c_float, i32, p, p, p]
    assert lib.hora_group_advantage(None, None, 5, 7, 0.0, 0, None, None, None) == 1                # unknown mode
    assert lib.hora_group_advantage(None, None, 5, 0, 0.0, 2, None, None, None) == 1                # ddof
    assert lib.hora_group_advantage(None, None, 0, 0, 0.0, 0, None, None, None) == 0


def test_allocate_refuses_what_the_host_can_see(lib):
    """hora_allocate: more than 2^31 - 1 prompts (row indices are kept in 32 bits), negative sizes, a cap above
    ld and unknown flags are refused with INVALID_ARG before the device is touched."""
    i64, i32, f64, p, u32 = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p, ctypes.c_uint32
    lib.hora_allocate.argtypes = [p, p, f64, f64, p, i32, p, i32, i64, i32, p, i64, u32, p, p, p, p, p, ctypes.c_size_t, p]

    def call(N=10, ld=8, G0=4, B=5, cap_scalar=8, flags=0, alpha0=1.0):
        return lib.hora_allocate(None, None, alpha0, 1.0, None, G0, None, cap_scalar, N, ld, None, B, flags, None, None,
                                 None, None, None, 0, None)

    assert call(N=1 << 31) == 1
    assert call(N=(1 << 31) + 12345) == 1
    assert call(N=-1) == 1 and call(ld=0) == 1 and call(G0=-1) == 1 and call(B=-1) == 1
    assert call(cap_scalar=9) == 1 and call(flags=64) == 1 and call(alpha0=0.0) == 1
    assert call(N=(1 << 31) - 1) == 1          # in range, but c / delta / G are missing
    lib.hora_status_string.restype = ctypes.c_char_p
    assert b"internal" in lib.hora_status_string(8)
