"""Thin ctypes binding over libdelta_attn.so (argument marshalling only).

The functions carry the names of the C ABI (include/delta_attn.h).  torch supplies device
memory (tensor.data_ptr()) and the current CUDA stream; every step of the hot path runs in
the library's own kernels.  There is no CPU fallback: if the shared library cannot be built
or loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

from . import _build

DELTA_TILE_ROWS = 64

# enums (values of include/delta_attn.h)
DELTA_OK = 0
DELTA_ERR_INVALID_ARG, DELTA_ERR_UNSUPPORTED, DELTA_ERR_WORKSPACE, DELTA_ERR_CAPACITY = 1, 2, 3, 4
DELTA_ERR_STATE, DELTA_ERR_CUDA, DELTA_ERR_TIMEOUT, DELTA_ERR_SCRATCH_LIMIT, DELTA_ERR_BOUNDS = 5, 6, 7, 8, 9
DELTA_F32, DELTA_BF16 = 0, 1
DELTA_SRC_QUERY, DELTA_SRC_KEY, DELTA_SRC_QUERY_BOTTOM_UP = 0, 1, 2
DELTA_WIN_BLOCK, DELTA_WIN_SLIDING = 0, 1
DELTA_INIT_BASIS_EXACT, DELTA_INIT_ZERO_STATE = 0, 1
(DELTA_VIEW_DQ, DELTA_VIEW_MASK, DELTA_VIEW_ROW_NNZ, DELTA_VIEW_TILE_NNZ, DELTA_VIEW_IDX,
 DELTA_VIEW_QHAT_TILE, DELTA_VIEW_QHAT, DELTA_VIEW_R, DELTA_VIEW_COUNTERS) = range(9)

EXPORTED = [
    "delta_state_workspace_bytes", "delta_state_init", "delta_state_reset", "delta_state_destroy",
    "delta_attn_prefill", "delta_prefill_staging_bytes", "delta_attn_prefill_host", "delta_attn_prefill_varlen",
    "delta_state_sequence_position",
    "delta_attn_decode_step", "delta_sparsity_stats", "delta_window_from_gamma", "delta_state_view",
    "delta_state_position", "delta_state_prefill_kernel", "delta_state_decode_kernel",
    "delta_state_set_decode_kernel",
    "delta_state_set_prefill_kernel", "delta_state_set_key_cache", "delta_key_cache_bytes",
    "delta_launch_count", "delta_status_string", "delta_last_cuda_error", "delta_debug_bounds_build",
    "delta_state_enable_profiling", "delta_state_prefill_kernel_ms",
    "delta_attn_decode_step_noalloc", "delta_noalloc_device_status",
]


class delta_config_t(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32),
                ("T_max", C.c_int32), ("dtype", C.c_int), ("source", C.c_int),
                ("prefill_window", C.c_int), ("init", C.c_int)]


class delta_stage_stats_t(C.Structure):
    _fields_ = [("nnz", C.c_uint64), ("elements", C.c_uint64), ("macs_done", C.c_uint64),
                ("macs_dense", C.c_uint64), ("S_m", C.c_double), ("S_c_eq6", C.c_double),
                ("S_c_exact", C.c_double)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class delta_stats_t(C.Structure):
    _fields_ = [("prefill", delta_stage_stats_t), ("decode", delta_stage_stats_t),
                ("combined", delta_stage_stats_t), ("n", C.c_int32), ("device_status", C.c_uint32)]

    def as_dict(self):
        return dict(prefill=self.prefill.as_dict(), decode=self.decode.as_dict(),
                    combined=self.combined.as_dict(), n=self.n, device_status=self.device_status)


class DeltaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.delta_status_string(status).decode()
        if status == DELTA_ERR_CUDA:
            msg += " (" + lib.delta_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [{status}]")


def _load() -> C.CDLL:
    # DELTA_ATTN_DEBUG_BOUNDS=1 selects the bounds-checking build of the library
    debug = os.environ.get("DELTA_ATTN_DEBUG_BOUNDS", "") not in ("", "0")
    path = _build.build(debug_bounds=debug)          # raises if nvcc or the sources are missing
    l = C.CDLL(path)
    vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
    cfgp = C.POINTER(delta_config_t)
    sig = {
        "delta_state_workspace_bytes": (C.c_int, [cfgp, C.POINTER(sz)]),
        "delta_state_init": (C.c_int, [cfgp, vp, sz, vp, C.POINTER(vp)]),
        "delta_state_reset": (C.c_int, [vp, vp]),
        "delta_state_destroy": (C.c_int, [vp]),
        "delta_attn_prefill": (C.c_int, [vp, vp, vp, vp, vp, i32, i32, i32, i32, f32, i32, vp]),
        "delta_prefill_staging_bytes": (C.c_int, [cfgp, i32, C.POINTER(sz)]),
        "delta_attn_prefill_varlen": (C.c_int, [vp, vp, vp, vp, vp, C.POINTER(i32), C.POINTER(i32), f32, vp]),
        "delta_state_sequence_position": (i32, [vp, i32]),
        "delta_attn_prefill_host": (C.c_int, [vp, vp, vp, vp, vp, vp, sz, i32, f32, i32, vp]),
        "delta_attn_decode_step": (C.c_int, [vp, vp, vp, vp, vp, vp, vp, f32, i32, vp]),
        "delta_sparsity_stats": (C.c_int, [vp, C.POINTER(delta_stats_t), vp]),
        "delta_window_from_gamma": (i32, [i32, C.c_double, i32]),
        "delta_state_view": (C.c_int, [vp, i32, C.POINTER(vp), C.POINTER(sz)]),
        "delta_state_position": (i32, [vp]),
        "delta_state_prefill_kernel": (i32, [vp]),
        "delta_state_decode_kernel": (i32, [vp]),
        "delta_state_set_decode_kernel": (C.c_int, [vp, i32]),
        "delta_state_set_prefill_kernel": (C.c_int, [vp, i32]),
        "delta_state_set_key_cache": (C.c_int, [vp, i32]),
        "delta_key_cache_bytes": (C.c_int, [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), vp]),
        "delta_state_enable_profiling": (C.c_int, [vp, i32]),
        "delta_state_prefill_kernel_ms": (C.c_int, [vp, C.POINTER(C.c_float)]),
        "delta_attn_decode_step_noalloc": (C.c_int, [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32,
                                                     i32, i32, C.c_int, f32, i32, vp]),
        "delta_noalloc_device_status": (C.c_int, [C.POINTER(C.c_uint32), vp]),
        "delta_launch_count": (C.c_uint64, []),
        "delta_debug_bounds_build": (i32, []),
        "delta_status_string": (C.c_char_p, [C.c_int]),
        "delta_last_cuda_error": (C.c_char_p, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(l, name)
        fn.restype = res
        fn.argtypes = args
    return l


lib = _load()
LIB_PATH = _build.LIB_DEBUG if lib.delta_debug_bounds_build() else _build.LIB


def _check(status: int, where: str):
    if status != DELTA_OK:
        raise DeltaError(status, where)


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(type(t))


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


def make_config(B, H, H_kv, d, T_max, dtype="bf16", source=DELTA_SRC_QUERY,
                prefill_window=DELTA_WIN_BLOCK, init=DELTA_INIT_BASIS_EXACT) -> delta_config_t:
    dt = {"f32": DELTA_F32, "bf16": DELTA_BF16}.get(dtype, dtype)
    return delta_config_t(B, H, H_kv, d, T_max, dt, source, prefill_window, init)


def delta_state_workspace_bytes(cfg: delta_config_t) -> int:
    n = C.c_size_t(0)
    _check(lib.delta_state_workspace_bytes(C.byref(cfg), C.byref(n)), "delta_state_workspace_bytes")
    return n.value


class DeltaState:
    """Owns the torch workspace tensor and the library's host-side state handle."""

    def __init__(self, cfg: delta_config_t, handle, workspace):
        self.cfg, self.handle, self.workspace = cfg, handle, workspace

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and lib is not None:      # module globals are gone while the interpreter shuts down
            lib.delta_state_destroy(h)


def delta_state_init(cfg: delta_config_t, device="cuda", stream=None, workspace=None) -> DeltaState:
    """Allocates the workspace with torch (unless one is given) and calls delta_state_init."""
    import torch
    nbytes = delta_state_workspace_bytes(cfg)
    if workspace is None:
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
    h = C.c_void_p()
    _check(lib.delta_state_init(C.byref(cfg), _ptr(workspace), workspace.numel(), _stream(stream),
                                C.byref(h)), "delta_state_init")
    return DeltaState(cfg, h, workspace)


def delta_state_reset(st: DeltaState, stream=None):
    _check(lib.delta_state_reset(st.handle, _stream(stream)), "delta_state_reset")


def delta_attn_prefill(st: DeltaState, q, k, v, out, T, H, H_kv, d, theta, window, stream=None):
    _check(lib.delta_attn_prefill(st.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), T, H, H_kv, d,
                                  theta, window, _stream(stream)), "delta_attn_prefill")


def delta_attn_prefill_varlen(st: DeltaState, q, k, v, out, seq_lens, windows, theta, stream=None):
    """q, out packed per sequence ([H, seq_lens[b], d] one behind the other); seq_lens and windows are
    host integer sequences of length B."""
    n = st.cfg.B
    lens = (C.c_int32 * n)(*[int(x) for x in seq_lens])
    wins = (C.c_int32 * n)(*[int(x) for x in windows])
    _check(lib.delta_attn_prefill_varlen(st.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), lens, wins, theta,
                                         _stream(stream)), "delta_attn_prefill_varlen")


def delta_state_sequence_position(st: DeltaState, b: int) -> int:
    return lib.delta_state_sequence_position(st.handle, b)


def delta_prefill_staging_bytes(cfg: delta_config_t, T: int) -> int:
    n = C.c_size_t(0)
    _check(lib.delta_prefill_staging_bytes(C.byref(cfg), T, C.byref(n)), "delta_prefill_staging_bytes")
    return n.value


def delta_attn_prefill_host(st: DeltaState, q_host, k_host, v_host, out_host, staging, T, theta,
                            window, stream=None):
    _check(lib.delta_attn_prefill_host(st.handle, _ptr(q_host), _ptr(k_host), _ptr(v_host),
                                       _ptr(out_host), _ptr(staging), staging.numel(), T, theta,
                                       window, _stream(stream)), "delta_attn_prefill_host")


def delta_attn_decode_step(st: DeltaState, q_new, k_new, v_new, k_cache, v_cache, out, theta, window,
                           stream=None):
    _check(lib.delta_attn_decode_step(st.handle, _ptr(q_new), _ptr(k_new), _ptr(v_new),
                                      _ptr(k_cache), _ptr(v_cache), _ptr(out), theta, window,
                                      _stream(stream)), "delta_attn_decode_step")


def delta_attn_decode_step_noalloc(q_new, k_new, v_new, k_cache, v_cache, out, qhat_in, qhat_out, R,
                                   n, B, H, H_kv, d, T_max, dtype, theta, window, stream=None):
    """Decode step for callers that cannot allocate: the carried state (qhat_in -> qhat_out, R)
    is passed explicitly and the scratch is a fixed array inside the library.  Allocates nothing."""
    dt = {"f32": DELTA_F32, "bf16": DELTA_BF16}.get(dtype, dtype)
    _check(lib.delta_attn_decode_step_noalloc(_ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                              _ptr(v_cache), _ptr(out), _ptr(qhat_in), _ptr(qhat_out),
                                              _ptr(R), n, B, H, H_kv, d, T_max, dt, theta, window,
                                              _stream(stream)), "delta_attn_decode_step_noalloc")


def delta_noalloc_device_status(stream=None) -> int:
    """Reads and clears the status word of the no-alloc decode step on the current device."""
    v = C.c_uint32(0)
    lib.delta_noalloc_device_status(C.byref(v), _stream(stream))
    return v.value


def delta_sparsity_stats(st: DeltaState, stream=None) -> dict:
    s = delta_stats_t()
    _check(lib.delta_sparsity_stats(st.handle, C.byref(s), _stream(stream)), "delta_sparsity_stats")
    return s.as_dict()


def delta_window_from_gamma(n: int, gamma: float, w_max: int) -> int:
    return lib.delta_window_from_gamma(n, gamma, w_max)


def delta_state_position(st: DeltaState) -> int:
    return lib.delta_state_position(st.handle)


def delta_state_prefill_kernel(st: DeltaState) -> int:
    return lib.delta_state_prefill_kernel(st.handle)


def delta_state_decode_kernel(st: DeltaState) -> int:
    return lib.delta_state_decode_kernel(st.handle)


def delta_state_set_decode_kernel(st: DeltaState, which: int) -> None:
    _check(lib.delta_state_set_decode_kernel(st.handle, which), "delta_state_set_decode_kernel")


def delta_state_set_prefill_kernel(st: DeltaState, which: int):
    _check(lib.delta_state_set_prefill_kernel(st.handle, which), "delta_state_set_prefill_kernel")


def delta_state_set_key_cache(st: DeltaState, packed: bool):
    _check(lib.delta_state_set_key_cache(st.handle, int(packed)), "delta_state_set_key_cache")


def delta_key_cache_bytes(st: DeltaState, stream=None):
    """(bytes of the packed key-delta encoding in use, bytes of the dense reference-key rows)."""
    a, b = C.c_uint64(0), C.c_uint64(0)
    _check(lib.delta_key_cache_bytes(st.handle, C.byref(a), C.byref(b), _stream(stream)), "delta_key_cache_bytes")
    return a.value, b.value


def delta_state_enable_profiling(st: DeltaState, enable: bool):
    _check(lib.delta_state_enable_profiling(st.handle, int(enable)), "delta_state_enable_profiling")


def delta_state_prefill_kernel_ms(st: DeltaState) -> list:
    ms = (C.c_float * 4)()
    _check(lib.delta_state_prefill_kernel_ms(st.handle, ms), "delta_state_prefill_kernel_ms")
    return list(ms)


def delta_launch_count() -> int:
    return lib.delta_launch_count()


_VIEW_DTYPES = {DELTA_VIEW_DQ: "float32", DELTA_VIEW_MASK: "int32", DELTA_VIEW_ROW_NNZ: "int16",
                DELTA_VIEW_TILE_NNZ: "int32", DELTA_VIEW_IDX: "uint8", DELTA_VIEW_QHAT_TILE: "float32",
                DELTA_VIEW_QHAT: "float32", DELTA_VIEW_R: "float32", DELTA_VIEW_COUNTERS: "int64"}


def delta_state_view(st: DeltaState, what: int):
    """A torch tensor aliasing one of the state's arrays (shape per include/delta_attn.h)."""
    import torch
    p, n = C.c_void_p(), C.c_size_t(0)
    _check(lib.delta_state_view(st.handle, what, C.byref(p), C.byref(n)), "delta_state_view")
    off = p.value - st.workspace.data_ptr()
    raw = st.workspace[off:off + n.value]
    c = st.cfg
    nt = (c.T_max + DELTA_TILE_ROWS - 1) // DELTA_TILE_ROWS
    shapes = {DELTA_VIEW_DQ: (c.B, c.H, c.T_max, c.d), DELTA_VIEW_MASK: (c.B, c.H, c.T_max, c.d // 32),
              DELTA_VIEW_ROW_NNZ: (c.B, c.H, c.T_max), DELTA_VIEW_TILE_NNZ: (c.B, c.H, nt),
              DELTA_VIEW_IDX: (c.B, c.H, c.T_max, c.d), DELTA_VIEW_QHAT_TILE: (c.B, c.H, nt, c.d),
              DELTA_VIEW_QHAT: (c.B, c.H, c.d), DELTA_VIEW_R: (c.B, c.H, c.T_max),
              DELTA_VIEW_COUNTERS: (n.value // 8,)}
    return raw.view(getattr(torch, _VIEW_DTYPES[what])).view(shapes[what])
