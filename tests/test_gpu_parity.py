"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Bars: masks, counts, indices, delta values and reference states are bit-exact; attention
outputs agree within max-abs 1e-4 for fp32 inputs and within 2e-2 relative for bf16 (per output
row: its largest error against its own largest reference magnitude; the normalised RMS error of
the whole tensor is held to 5e-3 as well).
"""
import numpy as np
import pytest
import torch

from oracle import delta_oracle as O
from paper_2507_19608_b200 import workloads as WL

pytestmark = pytest.mark.gpu

FP32_ATOL = 1e-4
BF16_REL = 2e-2
BF16_NRMS = 5e-3


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2507_19608_b200 import binding
    return binding


def _inputs(Bn, H, Hk, T, d, dtype, seed, rho=0.95, sigma=0.5):
    w = WL.Workload("t", Bn, H, Hk, T, d, dtype, rho, sigma, 0, (), seed)
    t = WL.make_qkv(w)
    return t["q"], t["k"], t["v"]


def _check_out(gpu, ref, dtype, what=""):
    err = np.abs(gpu - ref)
    if dtype == "f32":
        assert err.max() <= FP32_ATOL, f"{what}: max abs err {err.max():.3e}"
    else:
        # relative 2e-2, taken row by row: the largest error of an output row against the largest
        # reference magnitude of that same row (a small row cannot hide behind a large one)
        row_scale = np.abs(ref).max(axis=-1, keepdims=True)
        rel = err.max(axis=-1, keepdims=True) / np.maximum(row_scale, 1e-30)
        assert rel.max() <= BF16_REL, f"{what}: worst row rel err {rel.max():.3e}"
        nrms = np.sqrt(np.mean(err ** 2)) / np.sqrt(np.mean(ref ** 2))
        assert nrms <= BF16_NRMS, f"{what}: nrms {nrms:.3e}"
    assert np.isfinite(gpu).all()


def _check_delta_arrays(B, st, q, theta, init, T):
    Bn, H, _, d = q.shape
    dq = B.delta_state_view(st, B.DELTA_VIEW_DQ).cpu().numpy()
    mask = B.delta_state_view(st, B.DELTA_VIEW_MASK).cpu().numpy().view(np.uint32)
    rnz = B.delta_state_view(st, B.DELTA_VIEW_ROW_NNZ).cpu().numpy().view(np.uint16)
    tnz = B.delta_state_view(st, B.DELTA_VIEW_TILE_NNZ).cpu().numpy().view(np.uint32)
    idx = B.delta_state_view(st, B.DELTA_VIEW_IDX).cpu().numpy()
    qht = B.delta_state_view(st, B.DELTA_VIEW_QHAT_TILE).cpu().numpy()
    qh = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy()
    nt = (T + 63) // 64
    total = 0
    for b in range(Bn):
        for h in range(H):
            r = O.delta_construct(q[b, h], theta, init)
            assert np.array_equal(dq[b, h, :T].view(np.uint32), r["dq"].view(np.uint32)), (b, h)
            assert np.array_equal(mask[b, h, :T], r["mask"]), (b, h)
            assert np.array_equal(rnz[b, h, :T], r["row_nnz"]), (b, h)
            assert np.array_equal(tnz[b, h, :nt], r["tile_nnz"]), (b, h)
            assert np.array_equal(idx[b, h, :T], r["idx"]), (b, h)
            assert np.array_equal(qht[b, h, :nt].view(np.uint32), r["ahat_tile"].view(np.uint32)), (b, h)
            assert np.array_equal(qh[b, h].view(np.uint32), r["ahat"].view(np.uint32)), (b, h)
            total += int(r["row_nnz"].astype(np.int64).sum())
    return total


# ------------------------------------------------------------------ delta construction: bit-exact
@pytest.mark.parametrize("Bn,H,T,d,dtype,theta,init", [
    (1, 1, 128, 64, "f32", 0.1, "basis_exact"),
    (2, 3, 200, 128, "bf16", 0.2, "basis_exact"),
    (1, 2, 1, 64, "bf16", 0.1, "basis_exact"),
    (1, 2, 64, 64, "f32", 0.3, "zero_state"),
    (1, 2, 65, 128, "f32", 0.0, "basis_exact"),
    (1, 4, 1000, 64, "bf16", 0.29, "zero_state"),
    (1, 2, 17, 64, "bf16", 1e9, "basis_exact"),
    (2, 80, 70, 64, "bf16", 0.2, "basis_exact"),       # more heads than SMs: the row-by-row chain kernel
    (1, 80, 130, 128, "f32", 0.1, "zero_state"),
])
def test_delta_construction_bit_exact(B, Bn, H, T, d, dtype, theta, init):
    from tests.gpu_helpers import run_prefill
    q, k, v = _inputs(Bn, H, H, T, d, dtype, seed=7 + T)
    st, out, _, _ = run_prefill(B, q, k, v, theta, 16, dtype, init=init)
    total = _check_delta_arrays(B, st, q, theta, init, T)
    s = B.delta_sparsity_stats(st)
    assert s["prefill"]["nnz"] == total and s["prefill"]["elements"] == Bn * H * T * d


@pytest.mark.parametrize("T,d,dtype,theta,init", [
    (1024, 64, "bf16", 0.4, "basis_exact"),
    (1000, 64, "f32", 0.3, "zero_state"),
    (777, 128, "bf16", 0.25, "basis_exact"),
    (2048, 64, "bf16", 0.5, "basis_exact"),
])
def test_delta_construction_hard_streams(B, T, d, dtype, theta, init):
    """Structured streams across several ring stages, checkpoint blocks and tiles: a steady drift
    (the reference trails the input by a constant phase, so a chain restarted anywhere else
    would never agree with it again), a constant (nothing ever fires), a staircase, a drift that
    reverses, noise around a drift, a slow sine below the threshold, NaN and infinities in the
    middle of a stage."""
    from tests.gpu_helpers import run_prefill
    H = 3
    q, k, v = _inputs(1, H, H, T, d, dtype, seed=11 + T)
    t = np.arange(T, dtype=np.float64)
    rng = np.random.default_rng(5)
    for h in range(H):
        for c in range(d):
            kind = (c + h) % 8
            slope = theta * (0.011 + 0.0007 * c)
            if kind == 0:
                x = slope * t
            elif kind == 1:
                x = np.full(T, 0.5 + c)
            elif kind == 2:
                x = np.floor(t / 37.0) * theta * 0.75
            elif kind == 3:
                x = slope * np.abs(t - T * 0.6)
            elif kind == 4:
                x = slope * t + 0.2 * theta * rng.standard_normal(T)
            elif kind == 5:
                x = -slope * t * 3.0
            elif kind == 6:
                x = theta * 0.9 * np.sin(t / 50.0 + c)
            else:
                continue                      # keep the AR(1) stream
            q[0, h, :, c] = x.astype(np.float32)
    q[0, 0, T // 2 + 3, 5] = np.nan
    q[0, 1, T // 3, 9] = np.inf
    q[0, 1, T // 3 + 40, 9] = -np.inf
    if dtype == "bf16":
        q = WL.round_to_bf16(q)
    st, out, _, _ = run_prefill(B, q, k, v, theta, 64, dtype, init=init)
    _check_delta_arrays(B, st, q, theta, init, T)


def test_delta_special_values_bit_exact(B):
    from tests.gpu_helpers import run_prefill
    T, d = 70, 64
    q, k, v = _inputs(1, 1, 1, T, d, "f32", seed=3)
    th = np.float32(0.1)
    q[0, 0, :6, 0] = [1.0, np.float32(1.0) + th, 1.0, 1.0, 1.0, 1.0]     # |diff| vs theta at rounding level
    q[0, 0, :6, 1] = [0.0, -0.0, 0.0, 1e-40, 0.0, 0.0]                   # signed zero, subnormal
    q[0, 0, :6, 2] = [1.0, 1.0 + 0.1, 1.0, 2.0, 2.0, 2.0]
    q[0, 0, 10:20, 3] = 5.0                                             # constant run: nothing fires inside
    for theta in (0.1, 0.0):
        st, out, _, _ = run_prefill(B, q, k, v, theta, 8, "f32")
        _check_delta_arrays(B, st, q, theta, "basis_exact", T)


# ------------------------------------------------------------------ prefill outputs
CASES = [
    # Bn, H, Hk, T,   d,  dtype, theta, W,  shape
    (1, 1, 1, 128, 64, "f32", 0.1, 16, "block"),       # the single-head fp32 configuration
    (1, 1, 1, 128, 64, "f32", 0.1, 16, "sliding"),
    (1, 2, 1, 130, 64, "f32", 0.2, 0, "block"),        # no window at all, ragged tail
    (1, 2, 2, 100, 128, "f32", 0.3, 100, "block"),     # window covers everything: dense
    (2, 4, 2, 200, 64, "bf16", 0.2, 64, "block"),      # GQA, batch 2, ragged
    (1, 4, 1, 257, 128, "bf16", 0.29, 50, "block"),    # window not a multiple of the tile
    (1, 4, 4, 192, 64, "bf16", 0.1, 37, "sliding"),
    (1, 2, 2, 64, 128, "bf16", 0.0, 5, "sliding"),     # theta = 0
    (1, 2, 1, 1, 64, "bf16", 0.1, 4, "block"),         # one token
    (1, 8, 2, 320, 64, "bf16", 1e9, 16, "block"),      # nothing fires after the basis row
    (1, 4, 2, 700, 64, "bf16", 0.3, 64, "block"),      # six 128-row tiles, ragged last tile
    (2, 2, 1, 513, 64, "bf16", 0.15, 200, "sliding"),  # window wider than a tile, one row in the last tile
    (1, 2, 2, 384, 64, "bf16", 0.25, 1000, "sliding"), # every tile exact
    (1, 2, 1, 300, 64, "bf16", 0.2, 0, "sliding"),     # no exact score at all
    (1, 2, 2, 260, 64, "bf16", 0.2, 128, "block", "zero_state"),
]


@pytest.mark.parametrize("case", CASES, ids=[f"{c[5]}-T{c[3]}-d{c[4]}-W{c[7]}{c[8][0]}-th{c[6]}{'-zs' if len(c) > 9 else ''}" for c in CASES])
@pytest.mark.parametrize("kernel", [0, 1, 2, 3, 4, 5], ids=["generic", "tc_delta", "tc_telescoped", "tc_telescoped_one_head", "tc_telescoped_two_heads", "tc_telescoped_both_forms"])
def test_prefill_output_matches_oracle(B, case, kernel):
    from tests.gpu_helpers import run_prefill, to_host_f64
    Bn, H, Hk, T, d, dtype, theta, W, shape = case[:9]
    init = case[9] if len(case) > 9 else "basis_exact"
    q, k, v = _inputs(Bn, H, Hk, T, d, dtype, seed=100 + T + d)
    if kernel >= 1:
        cfg = B.make_config(Bn, H, Hk, d, T, dtype)
        ws = torch.empty(B.delta_state_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        st0 = B.delta_state_init(cfg, workspace=ws)
        try:
            B.delta_state_set_prefill_kernel(st0, kernel)
        except B.DeltaError as e:
            assert e.status == B.DELTA_ERR_UNSUPPORTED
            pytest.skip("no tensor-core kernel for this configuration")
    st, out, _, _ = run_prefill(B, q, k, v, theta, W, dtype, shape=shape, init=init, kernel=kernel)
    assert B.delta_state_prefill_kernel(st) == kernel
    ref, heads = O.prefill_mha(q, k, v, theta, W, shape, init=init)
    _check_out(to_host_f64(out), ref, dtype, "prefill out")
    assert B.delta_sparsity_stats(st)["device_status"] == 0
    # hand-off state for decode: reference query and the last score row
    R = B.delta_state_view(st, B.DELTA_VIEW_R).cpu().numpy()
    for b in range(Bn):
        for h in range(H):
            Rref = heads[(b, h)]["state"]["R"]
            tol = 1e-4 * max(1.0, np.abs(Rref).max())
            assert np.abs(R[b, h, :T] - Rref).max() <= tol
    # counters (Eq. 6 inputs) are integers: exact
    s = B.delta_sparsity_stats(st)["prefill"]
    done = dense = nnz = 0
    for b in range(Bn):
        for h in range(H):
            c = O.prefill_stats(heads[(b, h)]["delta"]["row_nnz"], T, d, W, shape)
            done += c["macs_done"]; dense += c["macs_dense"]; nnz += c["nnz"]
    assert (s["nnz"], s["macs_done"], s["macs_dense"]) == (nnz, done, dense)
    one = O.finish_stats(dict(nnz=nnz, elements=Bn * H * T * d, macs_done=done, macs_dense=dense), min(W, T), T)
    assert s["S_m"] == pytest.approx(one["S_m"], abs=1e-12)
    assert s["S_c_eq6"] == pytest.approx(one["S_c_eq6"], abs=1e-12)
    assert s["S_c_exact"] == pytest.approx(one["S_c_exact"], abs=1e-12)


def test_theta0_full_window_equals_dense_attention(B):
    """theta = 0 with W >= T must be plain causal attention (checked against torch SDPA in fp64)."""
    from tests.gpu_helpers import run_prefill, to_host_f64
    q, k, v = _inputs(1, 4, 2, 150, 64, "f32", seed=5, sigma=0.0)
    st, out, _, _ = run_prefill(B, q, k, v, 0.0, 150, "f32")
    tq = torch.from_numpy(q.astype(np.float64))
    tk = torch.from_numpy(k.astype(np.float64)).repeat_interleave(2, dim=1)
    tv = torch.from_numpy(v.astype(np.float64)).repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).numpy()
    assert np.abs(to_host_f64(out) - ref).max() <= FP32_ATOL


@pytest.mark.parametrize("T_max", [160, 150], ids=["cache_longer_than_prompt", "cache_full"])
def test_prefill_host_entry_matches_device_entry(B, T_max):
    from tests.gpu_helpers import run_prefill
    Bn, H, Hk, T, d, dtype = 1, 4, 2, 150, 64, "bf16"
    q, k, v = _inputs(Bn, H, Hk, T, d, dtype, seed=9)
    st, out, _, _ = run_prefill(B, q, k, v, 0.2, 32, dtype, T_max=T_max)
    cfg = B.make_config(Bn, H, Hk, d, T_max, dtype)
    st2 = B.delta_state_init(cfg)
    staging = torch.empty(B.delta_prefill_staging_bytes(cfg, T), dtype=torch.uint8, device="cuda")
    hq = torch.from_numpy(WL.bf16_bits(q).view(np.int16)).pin_memory()
    hk = torch.from_numpy(WL.bf16_bits(k).view(np.int16)).pin_memory()
    hv = torch.from_numpy(WL.bf16_bits(v).view(np.int16)).pin_memory()
    ho = torch.empty_like(hq).pin_memory()
    B.delta_attn_prefill_host(st2, hq, hk, hv, ho, staging, T, 0.2, 32)
    assert torch.equal(ho.view(torch.bfloat16), out.cpu())


# ------------------------------------------------------------------ decode
@pytest.mark.parametrize("Bn,H,Hk,T,d,dtype,theta,W,steps", [
    (1, 2, 1, 100, 64, "f32", 0.2, 8, 6),
    (2, 4, 2, 130, 64, "bf16", 0.1, 64, 5),
    (1, 4, 1, 700, 128, "bf16", 0.29, 4, 4),      # several key splits per head group
    (1, 8, 1, 90, 64, "bf16", 0.1, 0, 3),         # no exact window, group of 8 heads
    (1, 2, 2, 40, 128, "f32", 0.0, 1000, 3),      # window covers the whole cache
    (1, 1, 1, 1, 64, "bf16", 0.1, 2, 4),          # decode right after a one-token prefill
    (1, 4, 1, 700, 64, "bf16", 0.29, 4, 4),       # several key slices, ragged tiles
    (3, 4, 4, 1500, 64, "bf16", 0.2, 200, 3),     # one head per KV head, window wider than a tile, 12 tiles
    (2, 4, 2, 255, 64, "bf16", 0.15, 1000, 3),    # window covers the cache; the new key opens a tile at step 2
    (40, 4, 4, 1100, 64, "bf16", 0.2, 64, 2),     # 160 KV heads: one slice of 9 tiles per head
    (19, 16, 8, 600, 64, "bf16", 0.25, 16, 2),    # 152 KV heads, groups of 2: one slice of 5 tiles
])
@pytest.mark.parametrize("decode_kernel", [0, 1], ids=["fp32_pipes", "tc_scores"])
def test_decode_steps_match_oracle(B, Bn, H, Hk, T, d, dtype, theta, W, steps, decode_kernel):
    from tests.gpu_helpers import run_prefill, to_dev, to_host_f64
    if decode_kernel == 1 and not (dtype == "bf16" and d == 64):
        pytest.skip("tensor-core decode scores: bf16, d = 64")
    w = WL.Workload("t", Bn, H, Hk, T, d, dtype, 0.95, 0.5, W, (), 77 + T, n_decode=steps)
    t = WL.make_qkv(w)
    st, out, kc, vc = run_prefill(B, t["q"], t["k"], t["v"], theta, W, dtype, shape="sliding", T_max=T + steps)
    B.delta_state_set_decode_kernel(st, decode_kernel)
    assert B.delta_state_decode_kernel(st) == decode_kernel
    ref, heads = O.prefill_mha(t["q"], t["k"], t["v"], theta, W, "sliding")
    states = {key: r["state"] for key, r in heads.items()}
    nnz = done = dense = 0
    for s in range(steps):
        qn, kn, vn = t["q_dec"][:, :, s], t["k_dec"][:, :, s], t["v_dec"][:, :, s]
        dqn, dkn, dvn = to_dev(qn, dtype), to_dev(kn, dtype), to_dev(vn, dtype)
        o = torch.full_like(dqn, float("nan"))
        B.delta_attn_decode_step(st, dqn, dkn, dvn, kc, vc, o, float(theta), int(W))
        torch.cuda.synchronize()
        oref, infos = O.decode_mha(states, qn, kn, vn, theta, W)
        _check_out(to_host_f64(o), oref, dtype, f"decode step {s}")
        n = T + s
        assert B.delta_state_position(st) == n + 1
        # the cache row was appended
        assert torch.equal(kc[:, :, n], dkn) and torch.equal(vc[:, :, n], dvn)
        R = B.delta_state_view(st, B.DELTA_VIEW_R).cpu().numpy()
        qh = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy()
        for (b, h), stt in states.items():
            tol = (1e-4 if dtype == "f32" else 1e-3) * max(1.0, np.abs(stt["R"]).max())
            assert np.abs(R[b, h, :n + 1] - stt["R"]).max() <= tol
            assert np.array_equal(qh[b, h].view(np.uint32), stt["qhat"].view(np.uint32))
            c = O.stage_stats([infos[(b, h)]["row_nnz"]], [n], d, W, "sliding")
            nnz += c["nnz"]; done += c["macs_done"]; dense += c["macs_dense"]
    stats = B.delta_sparsity_stats(st)
    sd = stats["decode"]
    assert (sd["nnz"], sd["elements"], sd["macs_done"], sd["macs_dense"]) == (nnz, Bn * H * d * steps, done, dense)
    # Eq. 6 per stage and over both stages against the oracle's aggregates
    want_dec = O.decode_stage_stats(dict(nnz=nnz, elements=Bn * H * d * steps, macs_done=done, macs_dense=dense),
                                    [W] * steps, [T + s + 1 for s in range(steps)])
    pre = [O.prefill_stats(r["delta"]["row_nnz"], T, d, W, "sliding") for r in heads.values()]
    want_pre = O.finish_stats({key: sum(c[key] for c in pre) for key in ("nnz", "elements", "macs_done", "macs_dense")},
                              min(W, T), T)
    want_all = O.combined_stats(want_pre, want_dec)
    for name, want in (("prefill", want_pre), ("decode", want_dec), ("combined", want_all)):
        for key in ("nnz", "elements", "macs_done", "macs_dense"):
            assert stats[name][key] == want[key], (name, key)
        for key in ("S_m", "S_c_eq6", "S_c_exact"):
            assert stats[name][key] == pytest.approx(want[key], abs=1e-12), (name, key)


# ------------------------------------------------------------------ device status word -> host
def test_device_status_word_reaches_the_host(B):
    """A kernel whose bounded wait runs out records DELTA_ERR_TIMEOUT in the device status word.
    No wait is made to run out here: the word is written by the host, through the counters view,
    and delta_sparsity_stats must report it (return value and device_status) until a reset."""
    from tests.gpu_helpers import run_prefill
    q, k, v = _inputs(1, 2, 1, 40, 64, "bf16", seed=2)
    st, out, _, _ = run_prefill(B, q, k, v, 0.1, 8, "bf16")
    assert B.delta_sparsity_stats(st)["device_status"] == 0
    counters = B.delta_state_view(st, B.DELTA_VIEW_COUNTERS)
    assert counters.numel() == 144
    counters[8] = B.DELTA_ERR_TIMEOUT
    torch.cuda.synchronize()
    with pytest.raises(B.DeltaError) as e:
        B.delta_sparsity_stats(st)
    assert e.value.status == B.DELTA_ERR_TIMEOUT
    B.delta_state_reset(st)
    assert B.delta_sparsity_stats(st)["device_status"] == 0
    # the word itself is cleared by the next prefill
    from tests.gpu_helpers import to_cache, to_dev
    o2 = torch.empty_like(out)
    B.delta_attn_prefill(st, to_dev(q, "bf16"), to_cache(k, 40, "bf16"), to_cache(v, 40, "bf16"), o2, 40, 2, 1, 64, 0.1, 8)
    torch.cuda.synchronize()
    assert int(B.delta_state_view(st, B.DELTA_VIEW_COUNTERS)[8].item()) == 0
    assert B.delta_sparsity_stats(st)["device_status"] == 0 and torch.equal(o2, out)


# ------------------------------------------------------------------ call-order and capacity errors
def test_state_errors(B):
    from tests.gpu_helpers import run_prefill, to_dev
    q, k, v = _inputs(1, 2, 1, 32, 64, "bf16", seed=1)
    st, out, kc, vc = run_prefill(B, q, k, v, 0.1, 4, "bf16", T_max=33)
    first = B.delta_sparsity_stats(st)["prefill"]
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_prefill(st, out, kc, vc, out, 32, 2, 1, 64, 0.1, 4)
    assert e.value.status == B.DELTA_ERR_STATE
    qn, kn = to_dev(q[:, :, 0], "bf16"), to_dev(k[:, :, 0], "bf16")
    o = torch.empty_like(qn)
    B.delta_attn_decode_step(st, qn, kn, kn, kc, vc, o, 0.1, 4)
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_decode_step(st, qn, kn, kn, kc, vc, o, 0.1, 4)
    assert e.value.status == B.DELTA_ERR_CAPACITY
    B.delta_state_reset(st)
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_decode_step(st, qn, kn, kn, kc, vc, o, 0.1, 4)
    assert e.value.status == B.DELTA_ERR_STATE
    for bad in (dict(theta=-1.0), dict(theta=float("nan")), dict(window=-1), dict(T=0), dict(H=3)):
        a = dict(T=32, H=2, theta=0.1, window=4); a.update(bad)
        with pytest.raises(B.DeltaError) as e:
            B.delta_attn_prefill(st, out, kc, vc, out, a["T"], a["H"], 1, 64, a["theta"], a["window"])
        assert e.value.status == B.DELTA_ERR_INVALID_ARG
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_prefill(st, out, kc, vc, out, 34, 2, 1, 64, 0.1, 4)
    assert e.value.status == B.DELTA_ERR_CAPACITY
    # a reset state takes a new prefill and reproduces the first result
    out2 = torch.empty_like(out)
    from tests.gpu_helpers import to_dev as td
    B.delta_attn_prefill(st, td(q, "bf16"), kc, vc, out2, 32, 2, 1, 64, 0.1, 4)
    torch.cuda.synchronize()
    assert torch.equal(out2, out)
    # ... with counters that started from zero again (the reset's clearing is done by the prefill)
    again = B.delta_sparsity_stats(st)
    assert again["prefill"] == first and again["decode"]["macs_dense"] == 0 and again["device_status"] == 0
    assert B.delta_launch_count() > 0


# ------------------------------------------------------------------ full-size configurations
@pytest.mark.parametrize("name,theta,heads,kernel", [
    ("llama32_1b_prefill", 0.1, (0, 13, 31), 2),
    ("llama32_1b_prefill", 0.3, (5, 18), 2),
    ("llama32_1b_prefill", 0.3, (7, 30), 1),
    ("llama32_1b_prefill", 0.05, (11,), 1),
    ("bitnet_2b_prefill", 0.29, (0, 19), 0),
    ("bitnet_2b_prefill", 0.29, (3, 12), 2),
])
def test_full_size_prefill_sampled_heads(B, name, theta, heads, kernel):
    """The benchmark's launch configuration at full size: delta arrays of the sampled heads are
    bit-exact, outputs of the sampled heads match the oracle, global counters match a recount
    over all heads."""
    from tests.gpu_helpers import run_prefill, to_host_f64
    w = WL.WORKLOADS[name]
    t = WL.make_qkv(w)
    st, out, _, _ = run_prefill(B, t["q"], t["k"], t["v"], theta, w.window, w.dtype, kernel=kernel)
    g = w.H // w.H_kv
    dq = B.delta_state_view(st, B.DELTA_VIEW_DQ)
    mask = B.delta_state_view(st, B.DELTA_VIEW_MASK)
    idx = B.delta_state_view(st, B.DELTA_VIEW_IDX)
    rnz = B.delta_state_view(st, B.DELTA_VIEW_ROW_NNZ).cpu().numpy().view(np.uint16)
    nnz_all = 0
    for h in range(w.H):
        r = O.delta_construct(t["q"][0, h], theta)
        assert np.array_equal(rnz[0, h], r["row_nnz"])
        assert np.array_equal(mask[0, h].cpu().numpy().view(np.uint32), r["mask"])
        nnz_all += int(r["row_nnz"].astype(np.int64).sum())
        if h in heads:
            assert np.array_equal(dq[0, h].cpu().numpy().view(np.uint32), r["dq"].view(np.uint32))
            assert np.array_equal(idx[0, h].cpu().numpy(), r["idx"])
    s = B.delta_sparsity_stats(st)["prefill"]
    assert s["nnz"] == nnz_all
    o = to_host_f64(out)
    for h in heads:
        ref = O.prefill_head(t["q"][0, h], t["k"][0, h // g], t["v"][0, h // g], theta, w.window, "block")
        _check_out(o[0, h], ref["out"], w.dtype, f"{name} head {h}")


@pytest.mark.parametrize("name,source,units", [
    ("llama32_1b_decode_b16", "query", ((0, 0), (9, 5), (15, 7))),
    ("llama32_1b_decode_b1", "query", ((0, 2), (0, 6))),
    ("llama32_1b_decode_b16", "key", ((3, 1), (12, 4))),
])
def test_full_size_decode_sampled_units(B, name, source, units):
    """The decode leg as the benchmark runs it (cache prefilled to 2048 tokens through
    delta_attn_prefill with a sliding window, kernels chosen by the library, then decode steps):
    outputs, carried references and score rows of sampled (batch, KV head) units against the
    oracle, step by step."""
    from tests.gpu_helpers import to_dev, to_host_f64
    w = WL.WORKLOADS[name]
    theta, steps = w.thetas[0], 3
    t = WL.make_qkv(w, n_decode=steps)
    key = source == "key"
    cfg = B.make_config(w.B, w.H, w.H_kv, w.d, w.T_max, w.dtype, prefill_window=B.DELTA_WIN_SLIDING,
                        source=B.DELTA_SRC_KEY if key else B.DELTA_SRC_QUERY)
    st = B.delta_state_init(cfg)
    g = w.H // w.H_kv

    def cache(x):
        full = np.zeros((w.B, w.H_kv, w.T_max, w.d), np.float32)
        full[:, :, :w.T] = x
        return to_dev(full, w.dtype)
    q, kc, vc = to_dev(t["q"], w.dtype), cache(t["k"]), cache(t["v"])
    out = torch.empty_like(q)
    B.delta_attn_prefill(st, q, kc, vc, out, w.T, w.H, w.H_kv, w.d, float(theta), int(w.window))
    assert B.delta_state_decode_kernel(st) == 1          # the tensor-core score kernel serves this shape
    o_pre = to_host_f64(out)
    states = {}
    for (b, kvh) in units:
        for hh in range(1 if key else g):
            h = kvh * g + hh
            r = O.prefill_head(t["q"][b, h], t["k"][b, kvh], t["v"][b, kvh], theta, w.window, "sliding",
                               source=source)
            _check_out(o_pre[b, h], r["out"], w.dtype, f"prefill unit {(b, h)}")
            states[(b, kvh) if key else (b, h)] = r["state"]
    for s_ in range(steps):
        qn, kn, vn = t["q_dec"][:, :, s_], t["k_dec"][:, :, s_], t["v_dec"][:, :, s_]
        o = torch.empty_like(to_dev(qn, w.dtype))
        B.delta_attn_decode_step(st, to_dev(qn, w.dtype), to_dev(kn, w.dtype), to_dev(vn, w.dtype), kc, vc, o,
                                 float(theta), int(w.window))
        og = to_host_f64(o)
        n = w.T + s_
        if key:
            for (b, kvh) in list(states):
                stt, _ = O.decode_key_step(states[(b, kvh)], kn[b, kvh], vn[b, kvh], theta)
                states[(b, kvh)] = stt
                for hh in range(g):
                    ref_o = O.decode_key_attend(stt, qn[b, kvh * g + hh], w.window)
                    _check_out(og[b, kvh * g + hh], np.asarray(ref_o), w.dtype,
                               f"key decode step {s_} unit {(b, kvh, hh)}")
        else:
            R = B.delta_state_view(st, B.DELTA_VIEW_R).cpu().numpy()
            qh = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy()
            for (b, h) in list(states):
                ref_o, stt, _ = O.decode_head(states[(b, h)], qn[b, h], kn[b, h // g], vn[b, h // g], theta, w.window)
                states[(b, h)] = stt
                _check_out(og[b, h], np.asarray(ref_o), w.dtype, f"decode step {s_} unit {(b, h)}")
                assert np.array_equal(qh[b, h].view(np.uint32), stt["qhat"].view(np.uint32))
                tol = 1e-3 * max(1.0, np.abs(stt["R"]).max())
                assert np.abs(R[b, h, :n + 1] - stt["R"]).max() <= tol
    assert B.delta_sparsity_stats(st)["device_status"] == 0


@pytest.mark.parametrize("kernel,theta", [(2, 0.1), (1, 0.2)])
def test_stack_layer_sampled_units(B, kernel, theta):
    """One layer of the 16-layer stack configuration (batch 8, T = 4096, block window 256) at full
    size: outputs of sampled (batch, head) units against the oracle, masks of the sampled units
    bit-exact, no device-side time-out."""
    from tests.gpu_helpers import run_prefill, to_host_f64
    w = WL.WORKLOADS["llama32_1b_stack_layer"]
    t = WL.make_qkv(w, layer=3, n_decode=0)
    st, out, _, _ = run_prefill(B, t["q"], t["k"], t["v"], theta, w.window, w.dtype, kernel=kernel)
    assert B.delta_sparsity_stats(st)["device_status"] == 0
    g = w.H // w.H_kv
    mask = B.delta_state_view(st, B.DELTA_VIEW_MASK)
    for (b, h) in ((0, 0), (7, 31), (3, 14)):
        ref = O.prefill_head(t["q"][b, h], t["k"][b, h // g], t["v"][b, h // g], theta, w.window, "block")
        assert np.array_equal(mask[b, h].cpu().numpy().view(np.uint32), ref["delta"]["mask"])
        _check_out(to_host_f64(out[b, h]), ref["out"], w.dtype, f"stack layer unit {(b, h)}")


# ------------------------------------------------------------------ key deltas (strategy 3)
KEY_CASES = [
    # Bn, H, Hk, T,  d,  theta, W,  shape
    (1, 4, 1, 200, 64, 0.2, 64, "block"),
    (2, 4, 2, 513, 64, 0.15, 100, "sliding"),
    (1, 2, 2, 300, 64, 0.3, 0, "block"),
    (1, 8, 2, 384, 128, 0.25, 128, "block"),
    (1, 2, 1, 130, 64, 0.1, 1000, "block"),        # window covers everything
    (1, 2, 1, 1, 64, 0.1, 4, "block"),
    (2, 80, 80, 150, 64, 0.2, 64, "block"),        # more KV heads than SMs: the row-by-row chain kernel
]


@pytest.mark.parametrize("case", KEY_CASES, ids=[f"T{c[3]}-d{c[4]}-W{c[6]}{c[7][0]}" for c in KEY_CASES])
@pytest.mark.parametrize("form", [2, 3, 4, 5], ids=["auto", "one_head", "two_heads", "both_forms"])
def test_key_delta_prefill_matches_oracle(B, case, form):
    """Strategy (3): the key stream of every KV head becomes the delta matrix (every form of the
    attention kernel's grid that the configuration has)."""
    from tests.gpu_helpers import to_cache, to_dev, to_host_f64
    Bn, H, Hk, T, d, theta, W, shape = case
    q, k, v = _inputs(Bn, H, Hk, T, d, "bf16", seed=300 + T + d)
    cfg = B.make_config(Bn, H, Hk, d, T, "bf16", source=B.DELTA_SRC_KEY,
                        prefill_window=B.DELTA_WIN_BLOCK if shape == "block" else B.DELTA_WIN_SLIDING)
    st = B.delta_state_init(cfg)
    try:
        B.delta_state_set_prefill_kernel(st, form)
    except B.DeltaError as e:
        assert e.status == B.DELTA_ERR_UNSUPPORTED and form in (4, 5)
        pytest.skip("no two-head form for this configuration")
    dq_, kc, vc = to_dev(q, "bf16"), to_cache(k, T, "bf16"), to_cache(v, T, "bf16")
    out = torch.full_like(dq_, float("nan"))
    B.delta_attn_prefill(st, dq_, kc, vc, out, T, H, Hk, d, float(theta), int(W))
    torch.cuda.synchronize()
    ref, heads = O.prefill_mha(q, k, v, theta, W, shape, source="key")
    _check_out(to_host_f64(out), ref, "bf16", "key-delta prefill out")
    # delta arrays are those of the key stream, one set per KV head (the leading H_kv heads of the views)
    g = H // Hk
    dk = B.delta_state_view(st, B.DELTA_VIEW_DQ).cpu().numpy()
    mask = B.delta_state_view(st, B.DELTA_VIEW_MASK).cpu().numpy().view(np.uint32)
    rnz = B.delta_state_view(st, B.DELTA_VIEW_ROW_NNZ).cpu().numpy().view(np.uint16)
    idx = B.delta_state_view(st, B.DELTA_VIEW_IDX).cpu().numpy()
    dk, mask, rnz, idx = (x.reshape(Bn * H, *x.shape[2:]) for x in (dk, mask, rnz, idx))
    nnz = done = dense = 0
    for b in range(Bn):
        for kvh in range(Hk):
            r = heads[(b, kvh * g)]["delta"]
            u = b * Hk + kvh
            assert np.array_equal(dk[u, :T].view(np.uint32), r["dq"].view(np.uint32))
            assert np.array_equal(mask[u, :T], r["mask"])
            assert np.array_equal(rnz[u, :T], r["row_nnz"])
            assert np.array_equal(idx[u, :T], r["idx"])
            c = O.stage_stats_key(r["row_nnz"], T, d, W, shape, g)
            nnz += c["nnz"]; done += c["macs_done"]; dense += c["macs_dense"]
    s = B.delta_sparsity_stats(st)["prefill"]
    assert (s["nnz"], s["elements"], s["macs_done"], s["macs_dense"]) == (nnz, Bn * Hk * T * d, done, dense)
    assert B.delta_sparsity_stats(st)["device_status"] == 0


@pytest.mark.parametrize("Bn,H,Hk,T,d,theta,W,steps", [
    (1, 4, 1, 100, 64, 0.2, 8, 5),
    (2, 4, 2, 300, 64, 0.15, 64, 4),
    (1, 8, 2, 700, 128, 0.29, 4, 4),       # several key slices
    (1, 2, 1, 90, 64, 0.1, 0, 3),          # no exact window at all
    (1, 2, 2, 40, 64, 0.0, 1000, 3),       # window covers the whole cache
    (1, 1, 1, 1, 64, 0.1, 2, 4),
    (2, 4, 2, 700, 64, 0.2, 100, 3),       # the window's edge inside a tile, several slices
    (3, 4, 4, 1500, 64, 0.2, 300, 2),      # window over three tiles: key-cache tiles, one mixed tile
    (40, 4, 4, 1100, 64, 0.2, 64, 2),      # 160 KV heads: one slice of 9 tiles per head
])
@pytest.mark.parametrize("decode_kernel", [0, 1, 2], ids=["fp32_pipes", "tc_scores", "packed_cache"])
def test_key_delta_decode_steps_match_oracle(B, Bn, H, Hk, T, d, theta, W, steps, decode_kernel):
    """Strategy (3) carried into decoding: the reference key per KV head is the carried state,
    old keys are scored through the reference-key rows, the W_d most recent ones exactly.
    packed_cache: the reference-key rows are rebuilt from the compressed key-delta cache (mask,
    packed fired values, segment bases), which the prefill builds and every step extends."""
    from tests.gpu_helpers import to_cache, to_dev, to_host_f64
    w = WL.Workload("t", Bn, H, Hk, T, d, "bf16", 0.95, 0.5, W, (), 500 + T, n_decode=steps)
    t = WL.make_qkv(w)
    T_max = T + steps
    cfg = B.make_config(Bn, H, Hk, d, T_max, "bf16", source=B.DELTA_SRC_KEY, prefill_window=B.DELTA_WIN_SLIDING)
    st = B.delta_state_init(cfg)
    if decode_kernel == 1 and d != 64:
        pytest.skip("tensor-core decode scores: d = 64")
    packed = decode_kernel == 2
    if packed:
        B.delta_state_set_key_cache(st, True)
    else:
        B.delta_state_set_decode_kernel(st, decode_kernel)
        assert B.delta_state_decode_kernel(st) == decode_kernel
    dq_, kc, vc = to_dev(t["q"], "bf16"), to_cache(t["k"], T_max, "bf16"), to_cache(t["v"], T_max, "bf16")
    out = torch.full_like(dq_, float("nan"))
    B.delta_attn_prefill(st, dq_, kc, vc, out, T, H, Hk, d, float(theta), int(W))
    ref, heads = O.prefill_mha(t["q"], t["k"], t["v"], theta, W, "sliding", source="key")
    _check_out(to_host_f64(out), ref, "bf16", "key-delta prefill out")
    g = H // Hk
    states = {(b, kvh): heads[(b, kvh * g)]["state"] for b in range(Bn) for kvh in range(Hk)}
    row_nnz = {key: list(heads[(key[0], key[1] * g)]["delta"]["row_nnz"]) for key in states}
    nnz = done = dense = 0
    for s in range(steps):
        qn, kn, vn = t["q_dec"][:, :, s], t["k_dec"][:, :, s], t["v_dec"][:, :, s]
        dqn, dkn, dvn = to_dev(qn, "bf16"), to_dev(kn, "bf16"), to_dev(vn, "bf16")
        o = torch.full_like(dqn, float("nan"))
        B.delta_attn_decode_step(st, dqn, dkn, dvn, kc, vc, o, float(theta), int(W))
        torch.cuda.synchronize()
        oref, infos = O.decode_mha_key(states, qn, kn, vn, theta, W)
        _check_out(to_host_f64(o), oref, "bf16", f"key-delta decode step {s}")
        n = T + s
        assert B.delta_state_position(st) == n + 1
        assert torch.equal(kc[:, :, n], dkn) and torch.equal(vc[:, :, n], dvn)
        khat = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy().reshape(Bn * H, d)
        for (b, kvh), stt in states.items():
            assert np.array_equal(khat[b * Hk + kvh].view(np.uint32), stt["khat"].view(np.uint32))
            row_nnz[(b, kvh)].append(infos[(b, kvh)]["row_nnz"])
            nnz += infos[(b, kvh)]["row_nnz"]
            for j in range(n + 1):
                done += g * (d if O.in_window(n, j, W, "sliding") else int(row_nnz[(b, kvh)][j]))
            dense += g * (n + 1) * d
    sd = B.delta_sparsity_stats(st)
    assert sd["device_status"] == 0
    sd = sd["decode"]
    assert (sd["nnz"], sd["elements"], sd["macs_done"], sd["macs_dense"]) == (nnz, Bn * Hk * d * steps, done, dense)
    if packed:
        # bytes of the encoding in use: values (2 bytes per fired element, segments padded to 8
        # values), mask words, counts, segment bases and offsets -- recounted from the oracle's masks
        got_packed, got_dense = B.delta_key_cache_bytes(st)
        n_tok = T + steps
        want = 0
        for key in states:
            rn = row_nnz[key]
            vals = 0
            for s0 in range(0, n_tok, 32):
                seg = int(sum(rn[s0:s0 + 32]))
                vals = (vals + 7) // 8 * 8 if s0 else 0        # a segment starts on a multiple of 8 values
                vals += seg
            segs = (n_tok + 31) // 32
            want += 2 * vals + n_tok * (d // 8) + n_tok * 2 + segs * d * 2 + (segs + 1) * 4
        assert got_dense == Bn * Hk * n_tok * d * 2
        assert got_packed == want


# ------------------------------------------------------------------ strategy (2): bottom-up query deltas
BOTTOM_UP_CASES = [
    # Bn, H, Hk, T,  d,  theta, W,  shape,    init
    (1, 4, 2, 200, 64, 0.2, 64, "block", "basis_exact"),       # ragged: the basis row sits inside a block
    (2, 4, 2, 513, 64, 0.15, 100, "sliding", "basis_exact"),
    (1, 2, 2, 256, 64, 0.3, 0, "block", "basis_exact"),        # no window: every score from the recursion
    (1, 8, 2, 384, 128, 0.25, 128, "block", "basis_exact"),
    (1, 2, 1, 1000, 64, 0.29, 64, "block", "zero_state"),
    (1, 2, 1, 1, 64, 0.1, 4, "block", "basis_exact"),
    (1, 96, 96, 150, 64, 0.2, 64, "block", "basis_exact"),      # more heads than SMs: the row-by-row chain kernel
]


@pytest.mark.parametrize("case", BOTTOM_UP_CASES, ids=[f"T{c[3]}-d{c[4]}-W{c[6]}{c[7][0]}" for c in BOTTOM_UP_CASES])
def test_bottom_up_query_delta_prefill_matches_oracle(B, case):
    """Strategy (2) of Section III-A: Eq. 2-3 and Eq. 4 run from the last row up; the basis is
    the last row.  Outputs within the bf16 bar; delta arrays (indexed by token row) bit-exact."""
    from tests.gpu_helpers import to_cache, to_dev, to_host_f64
    Bn, H, Hk, T, d, theta, W, shape, init = case
    q, k, v = _inputs(Bn, H, Hk, T, d, "bf16", seed=500 + T + d)
    cfg = B.make_config(Bn, H, Hk, d, T, "bf16", source=B.DELTA_SRC_QUERY_BOTTOM_UP,
                        prefill_window=B.DELTA_WIN_BLOCK if shape == "block" else B.DELTA_WIN_SLIDING,
                        init=B.DELTA_INIT_BASIS_EXACT if init == "basis_exact" else B.DELTA_INIT_ZERO_STATE)
    st = B.delta_state_init(cfg)
    dq_, kc, vc = to_dev(q, "bf16"), to_cache(k, T, "bf16"), to_cache(v, T, "bf16")
    out = torch.full_like(dq_, float("nan"))
    B.delta_attn_prefill(st, dq_, kc, vc, out, T, H, Hk, d, float(theta), int(W))
    torch.cuda.synchronize()
    ref, heads = O.prefill_mha(q, k, v, theta, W, shape, init, source="query", order="bottom_up")
    _check_out(to_host_f64(out), ref, "bf16", "bottom-up prefill out")
    dq = B.delta_state_view(st, B.DELTA_VIEW_DQ).cpu().numpy()
    mask = B.delta_state_view(st, B.DELTA_VIEW_MASK).cpu().numpy().view(np.uint32)
    rnz = B.delta_state_view(st, B.DELTA_VIEW_ROW_NNZ).cpu().numpy().view(np.uint16)
    idx = B.delta_state_view(st, B.DELTA_VIEW_IDX).cpu().numpy()
    qh = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy()
    nnz = done = dense = 0
    for b in range(Bn):
        for h in range(H):
            r = heads[(b, h)]["delta"]          # the oracle's arrays are in processing order: flip to token rows
            assert np.array_equal(dq[b, h, :T].view(np.uint32), r["dq"][::-1].view(np.uint32)), (b, h)
            assert np.array_equal(mask[b, h, :T], r["mask"][::-1]), (b, h)
            assert np.array_equal(rnz[b, h, :T], r["row_nnz"][::-1]), (b, h)
            assert np.array_equal(idx[b, h, :T], r["idx"][::-1]), (b, h)
            assert np.array_equal(qh[b, h].view(np.uint32), r["ahat"].view(np.uint32)), (b, h)
            c = O.stage_stats(r["row_nnz"][::-1], list(range(T)), d, W, shape)
            nnz += c["nnz"]; done += c["macs_done"]; dense += c["macs_dense"]
    s = B.delta_sparsity_stats(st)
    assert (s["prefill"]["nnz"], s["prefill"]["macs_done"], s["prefill"]["macs_dense"]) == (nnz, done, dense)
    assert s["device_status"] == 0
    # the method has no decode stage
    with pytest.raises(B.DeltaError):
        B.delta_attn_decode_step(st, dq_[:, :, 0].contiguous(), kc[:, :, 0].contiguous(), vc[:, :, 0].contiguous(),
                                 kc, vc, out[:, :, 0].contiguous(), float(theta), 4)


# ------------------------------------------------------------------ Eq. 5: window from the input length
@pytest.mark.parametrize("n", [100, 257, 640])
@pytest.mark.parametrize("gamma", [0.02, 0.05, 0.1])
def test_eq5_dynamic_window_prefill_and_decode(B, n, gamma):
    """Section III-B: the prefill window follows the input length, W = min(floor(gamma n), W_max),
    squares along the diagonal; decode uses the paper's fixed W_d = 4.  Outputs and the Eq. 6
    statistics of both stages against the oracle."""
    from tests.gpu_helpers import run_prefill, to_dev, to_host_f64
    H, Hk, d, theta, W_max, W_d, steps = 4, 2, 64, 0.25, 48, 4, 3
    W = B.delta_window_from_gamma(n, gamma, W_max)
    assert W == O.window_from_gamma(n, gamma, W_max)
    w = WL.Workload("t", 1, H, Hk, n, d, "bf16", 0.95, 0.5, W, (), 900 + n)
    t = WL.make_qkv(w, n_decode=steps)
    q, k, v = t["q"], t["k"], t["v"]
    st, out, kc, vc = run_prefill(B, q, k, v, theta, W, "bf16", T_max=n + steps)
    ref, heads = O.prefill_mha(q, k, v, theta, W, "block")
    _check_out(to_host_f64(out), ref, "bf16", f"prefill n={n} gamma={gamma} W={W}")
    states = {key: h["state"] for key, h in heads.items()}
    for s_ in range(steps):
        qn, kn, vn = t["q_dec"][:, :, s_], t["k_dec"][:, :, s_], t["v_dec"][:, :, s_]
        o = torch.empty_like(to_dev(qn, "bf16"))
        B.delta_attn_decode_step(st, to_dev(qn, "bf16"), to_dev(kn, "bf16"), to_dev(vn, "bf16"), kc, vc, o,
                                 float(theta), W_d)
        ref_o, _ = O.decode_mha(states, qn, kn, vn, theta, W_d)
        _check_out(to_host_f64(o), ref_o, "bf16", f"decode step {s_}")
    stats = B.delta_sparsity_stats(st)
    rn = np.concatenate([heads[(0, h)]["delta"]["row_nnz"] for h in range(H)])
    want = O.finish_stats(O.stage_stats(rn, [i for _ in range(H) for i in range(n)], d, W, "block"), min(W, n), n)
    got = stats["prefill"]
    assert (got["nnz"], got["macs_done"], got["macs_dense"]) == (want["nnz"], want["macs_done"], want["macs_dense"])
    assert abs(got["S_c_eq6"] - want["S_c_eq6"]) < 1e-6 and abs(got["S_c_exact"] - want["S_c_exact"]) < 1e-9
    assert stats["device_status"] == 0


# ------------------------------------------------------------------ streams
def test_two_states_on_two_streams_match_the_default_stream(B):
    """The library works on the stream it is given: two independent states, each driven on a
    stream of its own with their calls interleaved, give bit for bit what one state gives on
    the default stream (outputs, cache rows, reference state, counters)."""
    from tests.gpu_helpers import to_cache, to_dev
    Bn, H, Hk, T, d, dtype, theta, W, steps = 2, 8, 2, 700, 64, "bf16", 0.2, 64, 4
    sets = []
    for seed in (41, 42):
        w = WL.Workload("t", Bn, H, Hk, T, d, dtype, 0.95, 0.5, W, (), seed, n_decode=steps)
        sets.append(WL.make_qkv(w))

    def run(t, stream_ctx, other=None):
        """Generator: yields after every call so that two runs can be interleaved."""
        with stream_ctx():
            cfg = B.make_config(Bn, H, Hk, d, T + steps, dtype, prefill_window=B.DELTA_WIN_SLIDING)
            st = B.delta_state_init(cfg)
            dq_, kc, vc = to_dev(t["q"], dtype), to_cache(t["k"], T + steps, dtype), to_cache(t["v"], T + steps, dtype)
            out = torch.full_like(dq_, float("nan"))
            outs = []
        yield
        with stream_ctx():
            B.delta_attn_prefill(st, dq_, kc, vc, out, T, H, Hk, d, theta, W)
        yield
        for s in range(steps):
            with stream_ctx():
                dqn, dkn, dvn = (to_dev(t[n][:, :, s], dtype) for n in ("q_dec", "k_dec", "v_dec"))
                o = torch.full_like(dqn, float("nan"))
                B.delta_attn_decode_step(st, dqn, dkn, dvn, kc, vc, o, theta, W)
                outs.append(o)
            yield
        with stream_ctx():
            stats = B.delta_sparsity_stats(st)
            qh = B.delta_state_view(st, B.DELTA_VIEW_QHAT).clone()
        torch.cuda.synchronize()
        res.append((out, outs, kc, vc, qh, stats))
        yield

    import contextlib
    res = []
    for t in sets:                                  # one after the other on the default stream
        for _ in run(t, contextlib.nullcontext):
            pass
    want = list(res)
    res.clear()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    g1 = run(sets[0], lambda: torch.cuda.stream(s1))
    g2 = run(sets[1], lambda: torch.cuda.stream(s2))
    for _ in zip(g1, g2):                           # interleaved, each on its own stream
        pass
    torch.cuda.synchronize()
    assert len(res) == 2
    for got, ref in zip(res, want):
        assert torch.equal(got[0], ref[0])
        for a, b in zip(got[1], ref[1]):
            assert torch.equal(a, b)
        assert torch.equal(got[2][:, :, :T + steps], ref[2][:, :, :T + steps])
        assert torch.equal(got[3][:, :, :T + steps], ref[3][:, :, :T + steps])
        assert torch.equal(got[4], ref[4])
        assert got[5] == ref[5] and got[5]["device_status"] == 0


# ------------------------------------------------------------------ long decode runs
@pytest.mark.parametrize("source", ["query", "key"])
@pytest.mark.parametrize("decode_kernel", [0, 1, 2], ids=["fp32_pipes", "tc_scores", "packed_cache"])
def test_long_decode_run_crosses_tile_and_slice_boundaries(B, source, decode_kernel):
    """300 decode steps from a 100-token prompt: the cache grows across three 128-key tile
    boundaries and the number of key slices per head changes on the way; every step's output is
    held to the oracle's, the carried reference state bit for bit."""
    from tests.gpu_helpers import to_cache, to_dev, to_host_f64
    Bn, H, Hk, T, d, dtype, theta, W, W_d, steps = 1, 4, 2, 100, 64, "bf16", 0.2, 32, 4, 300
    g = H // Hk
    w = WL.Workload("t", Bn, H, Hk, T, d, dtype, 0.95, 0.5, W, (), 900, n_decode=steps)
    t = WL.make_qkv(w)
    T_max = T + steps
    cfg = B.make_config(Bn, H, Hk, d, T_max, dtype, prefill_window=B.DELTA_WIN_SLIDING,
                        source=B.DELTA_SRC_KEY if source == "key" else B.DELTA_SRC_QUERY)
    st = B.delta_state_init(cfg)
    if decode_kernel == 2:
        if source != "key":
            pytest.skip("the compressed cache belongs to key deltas")
        B.delta_state_set_key_cache(st, True)
    else:
        B.delta_state_set_decode_kernel(st, decode_kernel)
    dq_, kc, vc = to_dev(t["q"], dtype), to_cache(t["k"], T_max, dtype), to_cache(t["v"], T_max, dtype)
    out = torch.full_like(dq_, float("nan"))
    B.delta_attn_prefill(st, dq_, kc, vc, out, T, H, Hk, d, theta, W)
    ref, heads = O.prefill_mha(t["q"], t["k"], t["v"], theta, W, "sliding", source=source)
    if source == "key":
        states = {(b, kvh): heads[(b, kvh * g)]["state"] for b in range(Bn) for kvh in range(Hk)}
    else:
        states = {key: r["state"] for key, r in heads.items()}
    qd, kd, vd = (to_dev(np.ascontiguousarray(t[n].transpose(2, 0, 1, 3)), dtype) for n in ("q_dec", "k_dec", "v_dec"))
    od = torch.full_like(qd, float("nan"))
    for s in range(steps):
        B.delta_attn_decode_step(st, qd[s], kd[s], vd[s], kc, vc, od[s], theta, W_d)
    torch.cuda.synchronize()
    got = to_host_f64(od)
    for s in range(steps):
        qn, kn, vn = t["q_dec"][:, :, s], t["k_dec"][:, :, s], t["v_dec"][:, :, s]
        if source == "key":
            oref, _ = O.decode_mha_key(states, qn, kn, vn, theta, W_d)
        else:
            oref, _ = O.decode_mha(states, qn, kn, vn, theta, W_d)
        _check_out(got[s], oref, dtype, f"decode step {s}")
    assert B.delta_state_position(st) == T_max
    ref_state = B.delta_state_view(st, B.DELTA_VIEW_QHAT).cpu().numpy()
    if source == "key":
        kh = ref_state.reshape(Bn * H, d)
        for (b, kvh), stt in states.items():
            assert np.array_equal(kh[b * Hk + kvh].view(np.uint32), stt["khat"].view(np.uint32))
    else:
        R = B.delta_state_view(st, B.DELTA_VIEW_R).cpu().numpy()
        for (b, h), stt in states.items():
            assert np.array_equal(ref_state[b, h].view(np.uint32), stt["qhat"].view(np.uint32))
            assert np.abs(R[b, h, :T_max] - stt["R"]).max() <= 1e-3 * max(1.0, np.abs(stt["R"]).max())
    assert B.delta_sparsity_stats(st)["device_status"] == 0
    # the cache is full now
    with pytest.raises(B.DeltaError) as e:
        B.delta_attn_decode_step(st, qd[0], kd[0], vd[0], kc, vc, od[0], theta, W_d)
    assert e.value.status == B.DELTA_ERR_CAPACITY
