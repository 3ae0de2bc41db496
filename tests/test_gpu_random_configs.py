"""GPU parity on randomly drawn configurations (fixed seeds): shapes, head groupings, lengths around
the tile and checkpoint boundaries, thresholds, windows and kernels are drawn together, so that
combinations no hand-written case lists are met.  Same bars as the other parity tests: masks
bit-exact, outputs within 1e-4 (fp32) / 2e-2 relative (bf16) of the oracle."""
import numpy as np
import pytest
import torch

from oracle import delta_oracle as O
from paper_2507_19608_b200 import workloads as WL
from tests.test_gpu_parity import _check_out

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2507_19608_b200 import binding
    return binding


def _draw(rng, mode, large):
    d = int(rng.choice([64, 64, 128]))
    dtype = str(rng.choice(["bf16", "bf16", "f32"])) if mode == "query" else "bf16"
    g, Hk, Bn = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 3])), int(rng.choice([1, 1, 2]))
    H = g * Hk
    if large:
        T = int(rng.integers(130, 2200))
    else:
        T = int(rng.choice([1, 2, 7, 8, 9, 63, 64, 65, 127, 128, 129, int(rng.integers(1, 400))]))
    T = max(1, min(T, 10000 // (Bn * H)))
    return dict(
        mode=mode, Bn=Bn, H=H, Hk=Hk, T=T, d=d, dtype=dtype,
        W=int(rng.choice([0, 1, 3, 8, 64, 100, 128, 10000, int(rng.integers(0, 400))])),
        shape=str(rng.choice(["block", "sliding"])), theta=float(rng.choice([0.0, 0.05, 0.2, 0.4, 1e9])),
        init=str(rng.choice(["basis_exact", "basis_exact", "zero_state"])) if mode != "key" else "basis_exact",
        steps=int(rng.integers(1, 4)), seed=int(rng.integers(1, 1 << 30)),
        kernel=int(rng.choice([0, 1, 2, 3, 4, 5])), decode_kernel=int(rng.choice([0, 1])),
        W_d=int(rng.choice([0, 2, 64, 200, 5000])))


def _run(B, c):
    from tests.gpu_helpers import to_cache, to_dev, to_host_f64
    mode, Bn, H, Hk, T, d, dtype = (c[k] for k in ("mode", "Bn", "H", "Hk", "T", "d", "dtype"))
    theta, W, shape, init, steps = (c[k] for k in ("theta", "W", "shape", "init", "steps"))
    g = H // Hk
    w = WL.Workload("t", Bn, H, Hk, T, d, dtype, 0.95, 0.5, W, (), c["seed"], n_decode=steps)
    t = WL.make_qkv(w)
    T_max = T + steps
    src = {"query": B.DELTA_SRC_QUERY, "key": B.DELTA_SRC_KEY, "bottom_up": B.DELTA_SRC_QUERY_BOTTOM_UP}[mode]
    cfg = B.make_config(Bn, H, Hk, d, T_max, dtype, source=src,
                        prefill_window=B.DELTA_WIN_BLOCK if shape == "block" else B.DELTA_WIN_SLIDING,
                        init=B.DELTA_INIT_BASIS_EXACT if init == "basis_exact" else B.DELTA_INIT_ZERO_STATE)
    st = B.delta_state_init(cfg)
    for setter, which in ((B.delta_state_set_prefill_kernel, c["kernel"]),
                          (B.delta_state_set_decode_kernel, c["decode_kernel"])):
        if mode == "query" or setter is B.delta_state_set_decode_kernel:
            try:
                setter(st, which)
            except B.DeltaError as e:       # no such kernel for this configuration: the default runs
                assert e.status == B.DELTA_ERR_UNSUPPORTED
    dq_, kc, vc = to_dev(t["q"], dtype), to_cache(t["k"], T_max, dtype), to_cache(t["v"], T_max, dtype)
    out = torch.full_like(dq_, float("nan"))
    B.delta_attn_prefill(st, dq_, kc, vc, out, T, H, Hk, d, theta, W)
    torch.cuda.synchronize()
    if mode == "query":
        ref, heads = O.prefill_mha(t["q"], t["k"], t["v"], theta, W, shape, init=init)
    elif mode == "key":
        ref, heads = O.prefill_mha(t["q"], t["k"], t["v"], theta, W, shape, source="key")
    else:
        ref, heads = O.prefill_mha(t["q"], t["k"], t["v"], theta, W, shape, init, source="query", order="bottom_up")
    _check_out(to_host_f64(out), ref, dtype, "prefill out")
    mask = B.delta_state_view(st, B.DELTA_VIEW_MASK).cpu().numpy().view(np.uint32)
    if mode == "key":
        mk = mask.reshape(Bn * H, *mask.shape[2:])
        for b in range(Bn):
            for kvh in range(Hk):
                assert np.array_equal(mk[b * Hk + kvh, :T], heads[(b, kvh * g)]["delta"]["mask"])
    else:
        for (b, h), r in heads.items():
            m = r["delta"]["mask"]
            assert np.array_equal(mask[b, h, :T], m[::-1] if mode == "bottom_up" else m)
    if mode == "bottom_up":     # the method has no decode stage
        assert B.delta_sparsity_stats(st)["device_status"] == 0
        return
    if mode == "query":
        states = {key: r["state"] for key, r in heads.items()}
    else:
        states = {(b, kvh): heads[(b, kvh * g)]["state"] for b in range(Bn) for kvh in range(Hk)}
    for s in range(steps):
        qn, kn, vn = t["q_dec"][:, :, s], t["k_dec"][:, :, s], t["v_dec"][:, :, s]
        dqn, dkn, dvn = to_dev(qn, dtype), to_dev(kn, dtype), to_dev(vn, dtype)
        o = torch.full_like(dqn, float("nan"))
        B.delta_attn_decode_step(st, dqn, dkn, dvn, kc, vc, o, theta, c["W_d"])
        torch.cuda.synchronize()
        if mode == "query":
            oref, _ = O.decode_mha(states, qn, kn, vn, theta, c["W_d"])
        else:
            oref, _ = O.decode_mha_key(states, qn, kn, vn, theta, c["W_d"])
        _check_out(to_host_f64(o), oref, dtype, f"decode step {s}")
        n = T + s
        assert torch.equal(kc[:, :, n], dkn) and torch.equal(vc[:, :, n], dvn)
        ref_state = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy()
        if mode == "query":
            for (b, h), stt in states.items():
                assert np.array_equal(ref_state[b, h].view(np.uint32), stt["qhat"].view(np.uint32))
        else:
            kh = ref_state.reshape(Bn * H, d)
            for (b, kvh), stt in states.items():
                assert np.array_equal(kh[b * Hk + kvh].view(np.uint32), stt["khat"].view(np.uint32))
    assert B.delta_sparsity_stats(st)["device_status"] == 0


@pytest.mark.parametrize("mode,large,count,seed", [
    ("query", False, 200, 11), ("query", True, 40, 12),
    ("key", False, 120, 21), ("key", True, 30, 22),
    ("bottom_up", False, 120, 31), ("bottom_up", True, 30, 32),
])
def test_random_configurations_match_oracle(B, mode, large, count, seed):
    rng = np.random.default_rng(seed)
    for i in range(count):
        c = _draw(rng, mode, large)
        try:
            _run(B, c)
        except AssertionError as e:
            raise AssertionError(f"case {i}: {c}: {e}") from e
