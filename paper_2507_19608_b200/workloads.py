"""Seeded synthetic Q/K/V streams for the delta-attention tests and benchmark.

This module only *draws inputs*: it contains none of the method's arithmetic
(no thresholding, no scores, no softmax).  It is the one module that both the
CPU oracle's tests and the CUDA path's tests/bench import, so that both sides
see byte-identical host buffers.

Recipe.  Every (tensor, batch element, head, channel) is an independent AR(1)
chain along the token axis,

    x_0 = eps_0,   x_t = rho * x_{t-1} + sqrt(1 - rho^2) * eps_t,   eps ~ N(0,1)

drawn in float64 from numpy's PCG64, multiplied by a per-channel scale s_c and
then rounded (round-to-nearest-even) to the storage type.  Temporal
correlation along tokens is what gives the delta method something to skip;
the per-channel log-normal scale mimics the channel-magnitude spread of real
attention projections.

bf16 tensors are returned twice: as float32 arrays whose values are exactly
bf16-representable (what the oracle consumes) and as the uint16 bit patterns
(what is copied to the GPU).
"""
from __future__ import annotations

import dataclasses
import numpy as np

__all__ = [
    "Workload", "WORKLOADS", "ar1", "round_to_bf16", "bf16_bits", "bits_to_f32",
    "make_qkv", "make_decode_tokens",
]


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) & 0xFFFF0000
    # NaN stays NaN (quiet), never rounds to inf
    nan = np.isnan(x)
    out = r.astype(np.uint32).view(np.float32).copy()
    if nan.any():
        out[nan] = np.float32(np.nan)
    return out.reshape(x.shape)


def bf16_bits(x_bf16_as_f32: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    u = np.ascontiguousarray(x_bf16_as_f32, dtype=np.float32).view(np.uint32)
    assert not np.any(u & 0xFFFF), "value is not bf16-representable"
    return (u >> 16).astype(np.uint16)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen uint16 bf16 bit patterns to float32 (exact)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def ar1(rng: np.random.Generator, shape_prefix: tuple, T: int, d: int, rho: float,
        x_prev: np.ndarray | None = None) -> np.ndarray:
    """AR(1) chains along the token axis; returns float64 [*shape_prefix, T, d].

    x_prev (shape [*shape_prefix, d]) continues existing chains; otherwise the
    chain starts at x_0 = eps_0.
    """
    eps = rng.standard_normal(size=(*shape_prefix, T, d))
    out = np.empty_like(eps)
    c = float(np.sqrt(1.0 - rho * rho))
    if x_prev is None:
        out[..., 0, :] = eps[..., 0, :]
        start = 1
        prev = out[..., 0, :]
    else:
        start = 0
        prev = x_prev
    for t in range(start, T):
        prev = rho * prev + c * eps[..., t, :]
        out[..., t, :] = prev
    return out


@dataclasses.dataclass(frozen=True)
class Workload:
    """One attention-layer workload (shape + generator parameters)."""
    name: str
    B: int
    H: int
    H_kv: int
    T: int
    d: int
    dtype: str            # "f32" | "bf16"
    rho: float
    lognormal_sigma: float  # 0 => unit channel scale
    window: int
    thetas: tuple
    seed: int
    n_decode: int = 0
    layers: int = 1

    @property
    def T_max(self) -> int:
        return self.T + self.n_decode


# Shapes follow the two models the paper evaluates (their attention layers) and
# the decode scenario; the seeds are fixed so every run sees the same bytes.
WORKLOADS = {
    # single head, fp32, small enough for the oracle to finish in well under a second
    "single_head_fp32": Workload("single_head_fp32", 1, 1, 1, 128, 64, "f32", 0.9, 0.0, 16,
                                 (0.1,), seed=0),
    # Llama-3.2-1B attention layer: 32 query heads, 8 KV heads, head_dim 64
    "llama32_1b_prefill": Workload("llama32_1b_prefill", 1, 32, 8, 1024, 64, "bf16", 0.95, 0.5, 64,
                                   (0.05, 0.1, 0.2), seed=2000),
    # BitNet-b1.58-2B-4T attention layer: 20 query heads, 5 KV heads, head_dim 128
    "bitnet_2b_prefill": Workload("bitnet_2b_prefill", 1, 20, 5, 2048, 128, "bf16", 0.95, 0.0, 128,
                                  (0.29,), seed=3000),
    # decode at the Llama shape: cache prefilled to 2048, then 256 single-token steps
    "llama32_1b_decode_b1": Workload("llama32_1b_decode_b1", 1, 32, 8, 2048, 64, "bf16", 0.95, 0.5, 64,
                                     (0.1,), seed=4000, n_decode=256),
    "llama32_1b_decode_b16": Workload("llama32_1b_decode_b16", 16, 32, 8, 2048, 64, "bf16", 0.95, 0.5, 64,
                                      (0.1,), seed=4000, n_decode=256),
    # one layer of the 16-layer stack (layers are independent draws: seed + 100*layer)
    "llama32_1b_stack_layer": Workload("llama32_1b_stack_layer", 8, 32, 8, 4096, 64, "bf16", 0.95, 0.5, 256,
                                       (0.05, 0.1, 0.2), seed=5000, n_decode=128, layers=16),
}


def _cast(x64: np.ndarray, dtype: str) -> np.ndarray:
    x32 = x64.astype(np.float32)
    if dtype == "f32":
        return x32
    if dtype == "bf16":
        return round_to_bf16(x32)
    raise ValueError(dtype)


def _one_tensor(seed: int, B: int, heads: int, T: int, d: int, rho: float, sigma: float,
                dtype: str, n_extra: int):
    rng = np.random.default_rng(seed)
    if sigma > 0.0:
        scale = np.exp(sigma * rng.standard_normal(size=(1, heads, 1, d)))
    else:
        scale = np.ones((1, heads, 1, d))
    x = ar1(rng, (B, heads), T + n_extra, d, rho)
    x = _cast(x * scale, dtype)
    return x[:, :, :T, :].copy(), x[:, :, T:, :].copy()


def make_qkv(w: Workload, layer: int = 0, *, T: int | None = None, B: int | None = None,
             n_decode: int | None = None):
    """Draw Q [B,H,T,d], K, V [B,H_kv,T,d] (float32 arrays; bf16-representable when
    w.dtype == "bf16") plus the decode continuation of the same chains:
    q_dec [B,H,n_decode,d], k_dec, v_dec [B,H_kv,n_decode,d].

    Seeds: w.seed + 100*layer + {0: Q, 1: K, 2: V}.
    """
    T = w.T if T is None else T
    B = w.B if B is None else B
    nd = w.n_decode if n_decode is None else n_decode
    base = w.seed + 100 * layer
    q, qd = _one_tensor(base + 0, B, w.H, T, w.d, w.rho, w.lognormal_sigma, w.dtype, nd)
    k, kd = _one_tensor(base + 1, B, w.H_kv, T, w.d, w.rho, w.lognormal_sigma, w.dtype, nd)
    v, vd = _one_tensor(base + 2, B, w.H_kv, T, w.d, w.rho, w.lognormal_sigma, w.dtype, nd)
    return dict(q=q, k=k, v=v, q_dec=qd, k_dec=kd, v_dec=vd)


def make_decode_tokens(w: Workload, layer: int = 0):
    """Only the decode continuation (convenience wrapper around make_qkv)."""
    t = make_qkv(w, layer)
    return t["q_dec"], t["k_dec"], t["v_dec"]
