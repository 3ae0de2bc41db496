"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, rejects bad arguments before touching the device, and Eq. 5 matches the oracle."""
import ctypes as C
import os
import re

import pytest

from oracle import delta_oracle as O
from paper_2507_19608_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"DELTA_API\s+[\w\s\*]+?\b(delta_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 17
    raw = C.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in include/ but not exported"
    assert set(names) == set(B.EXPORTED)


def test_status_strings():
    assert B.lib.delta_status_string(0) == b"ok"
    assert B.lib.delta_debug_bounds_build() == 0      # the default process loads the regular build
    for s in range(1, 10):
        assert len(B.lib.delta_status_string(s)) > 3


@pytest.mark.parametrize("kw,want", [
    (dict(B=0), B.DELTA_ERR_INVALID_ARG),
    (dict(H=6, H_kv=4), B.DELTA_ERR_INVALID_ARG),
    (dict(d=96), B.DELTA_ERR_UNSUPPORTED),
    (dict(H=12, H_kv=4), B.DELTA_ERR_UNSUPPORTED),          # group of 3 query heads
    (dict(source=B.DELTA_SRC_KEY), B.DELTA_OK),              # key deltas: bf16 only
    (dict(source=B.DELTA_SRC_KEY, dtype="f32"), B.DELTA_ERR_UNSUPPORTED),
    (dict(source=B.DELTA_SRC_QUERY_BOTTOM_UP), B.DELTA_OK),    # strategy (2): bf16 only, prefill only
    (dict(source=B.DELTA_SRC_QUERY_BOTTOM_UP, dtype="f32"), B.DELTA_ERR_UNSUPPORTED),
    (dict(source=3), B.DELTA_ERR_INVALID_ARG),
    (dict(T_max=0), B.DELTA_ERR_INVALID_ARG),
    (dict(dtype=7), B.DELTA_ERR_INVALID_ARG),
])
def test_config_validation(kw, want):
    base = dict(B=1, H=8, H_kv=2, d=64, T_max=256, dtype="bf16")
    base.update(kw)
    cfg = B.make_config(**base)
    n = C.c_size_t(0)
    assert B.lib.delta_state_workspace_bytes(C.byref(cfg), C.byref(n)) == want


def test_workspace_size_grows_with_capacity_and_is_aligned():
    a = B.delta_state_workspace_bytes(B.make_config(1, 8, 2, 64, 256))
    b = B.delta_state_workspace_bytes(B.make_config(1, 8, 2, 64, 512))
    assert a % 256 == 0 and b > a
    # at least the delta values, indices and the score row
    assert a >= 8 * 256 * 64 * 5 + 8 * 256 * 4


def test_null_and_misaligned_arguments_are_rejected_before_any_device_work():
    cfg = B.make_config(1, 8, 2, 64, 256)
    h = C.c_void_p()
    assert B.lib.delta_state_init(C.byref(cfg), None, 1 << 30, None, C.byref(h)) == B.DELTA_ERR_INVALID_ARG
    assert B.lib.delta_state_init(C.byref(cfg), 0x1001, 1 << 30, None, C.byref(h)) == B.DELTA_ERR_WORKSPACE
    assert B.lib.delta_state_init(C.byref(cfg), 0x1000, 16, None, C.byref(h)) == B.DELTA_ERR_WORKSPACE
    assert B.lib.delta_attn_prefill(None, 1, 1, 1, 1, 8, 8, 2, 64, 0.1, 4, None) == B.DELTA_ERR_INVALID_ARG
    assert B.lib.delta_attn_decode_step(None, 1, 1, 1, 1, 1, 1, 0.1, 4, None) == B.DELTA_ERR_INVALID_ARG
    assert B.lib.delta_sparsity_stats(None, None, None) == B.DELTA_ERR_INVALID_ARG
    # decode pointers off the 16-byte grid: rejected on the host (the argument check comes before
    # anything looks at the state, so a dummy handle is enough here and nothing is launched)
    ok = 0x1000
    for bad in range(6):
        ptrs = [ok + (4 if i == bad else 0) for i in range(6)]
        assert B.lib.delta_attn_decode_step(0x10, *ptrs, 0.1, 4, None) == B.DELTA_ERR_INVALID_ARG
        assert B.lib.delta_attn_decode_step_noalloc(*ptrs, ok, ok + 64, ok, 10, 1, 8, 2, 64, 128, B.DELTA_BF16,
                                                    0.1, 4, None) == B.DELTA_ERR_INVALID_ARG
    assert B.lib.delta_noalloc_device_status(None, None) == B.DELTA_ERR_INVALID_ARG
    assert B.lib.delta_attn_prefill_varlen(None, 16, 16, 16, 16, None, None, 0.1, None) == B.DELTA_ERR_INVALID_ARG
    assert B.lib.delta_state_sequence_position(None, 0) == -1
    assert B.lib.delta_state_position(None) == -1


@pytest.mark.parametrize("n,gamma,wmax", [(1000, 0.05, 64), (1000, 0.1, 64), (10, 0.05, 64),
                                          (120, 0.25, 1 << 30), (4096, 0.02, 256), (0, 0.5, 8),
                                          (100, 0.02, 48), (257, 0.1, 16), (640, 0.05, 48)])
def test_window_from_gamma_matches_eq5(n, gamma, wmax):
    assert B.delta_window_from_gamma(n, gamma, wmax) == O.window_from_gamma(n, gamma, wmax)


def test_window_from_gamma_out_of_domain_is_zero():
    assert B.delta_window_from_gamma(-3, 0.5, 8) == 0
    assert B.delta_window_from_gamma(100, -0.1, 8) == 0
    assert B.delta_window_from_gamma(100, float("nan"), 8) == 0
