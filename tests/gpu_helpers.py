"""Helpers for the GPU parity tests: numpy <-> device marshalling around the C-ABI binding."""
import numpy as np
import torch

from paper_2507_19608_b200 import workloads as WL


def to_dev(x_f32: np.ndarray, dtype: str):
    """Host float32 array -> device tensor of the storage type (exact for bf16-representable input)."""
    t = torch.from_numpy(np.ascontiguousarray(x_f32))
    if dtype == "bf16":
        bits = torch.from_numpy(WL.bf16_bits(x_f32).view(np.int16))
        return bits.cuda().view(torch.bfloat16)
    return t.cuda()


def to_cache(x_f32: np.ndarray, T_max: int, dtype: str):
    """[B,H_kv,T,d] host array -> [B,H_kv,T_max,d] device cache (rows >= T filled with NaN so
    that any read of an unwritten row shows up)."""
    B, Hk, T, d = x_f32.shape
    full = np.full((B, Hk, T_max, d), np.nan, np.float32)
    full[:, :, :T] = x_f32
    t = torch.from_numpy(full)
    return t.to(torch.bfloat16).cuda() if dtype == "bf16" else t.cuda()


def to_host_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def run_prefill(B, q, k, v, theta, W, dtype, shape="block", init="basis_exact", T_max=None, kernel=None):
    """Runs delta_attn_prefill on numpy inputs; returns (state, out tensor, k_cache, v_cache)."""
    Bn, H, T, d = q.shape
    Hk = k.shape[1]
    T_max = T_max or T
    cfg = B.make_config(Bn, H, Hk, d, T_max, dtype,
                        prefill_window=B.DELTA_WIN_BLOCK if shape == "block" else B.DELTA_WIN_SLIDING,
                        init=B.DELTA_INIT_BASIS_EXACT if init == "basis_exact" else B.DELTA_INIT_ZERO_STATE)
    st = B.delta_state_init(cfg)
    if kernel is not None:
        B.delta_state_set_prefill_kernel(st, kernel)
    dq, kc, vc = to_dev(q, dtype), to_cache(k, T_max, dtype), to_cache(v, T_max, dtype)
    out = torch.full_like(dq, float("nan"))
    B.delta_attn_prefill(st, dq, kc, vc, out, T, H, Hk, d, float(theta), int(W))
    torch.cuda.synchronize()
    return st, out, kc, vc
