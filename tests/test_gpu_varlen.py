"""One prefill over sequences of different lengths (Section III-B, Eq. 5: the window follows the
input length), followed by decode steps from the positions the sequences stand at, against the
oracle run sequence by sequence."""
import numpy as np
import pytest
import torch

from oracle import delta_oracle as O
from paper_2507_19608_b200 import workloads as WL
from tests.test_gpu_parity import _check_out

pytestmark = pytest.mark.gpu

LENGTHS = (1, 63, 64, 257, 1000)
W_MAX = 64


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2507_19608_b200 import binding
    return binding


def _batch(H, Hk, d, steps, seed):
    """Independent AR(1) sequences of the test lengths: per sequence q [H,T+steps,d], k, v [Hk,T+steps,d]."""
    seqs = []
    for i, T in enumerate(LENGTHS):
        w = WL.Workload("v", 1, H, Hk, T, d, "bf16", 0.95, 0.5, 0, (), seed + 10 * i, n_decode=steps)
        t = WL.make_qkv(w)
        seqs.append({key: val[0] for key, val in t.items()})
    return seqs


@pytest.mark.parametrize("gamma", [0.02, 0.05, 0.1])
@pytest.mark.parametrize("source", ["query", "key"])
def test_ragged_batch_prefill_and_decode_match_oracle(B, gamma, source):
    from tests.gpu_helpers import to_dev, to_host_f64
    H, Hk, d, steps, theta, W_d = 4, 2, 64, 2, 0.25, 4
    g = H // Hk
    key = source == "key"
    seqs = _batch(H, Hk, d, steps, seed=900)
    Bn = len(LENGTHS)
    T_max = max(LENGTHS) + steps
    windows = [O.window_from_gamma(T, gamma, W_MAX) for T in LENGTHS]
    assert windows == [B.delta_window_from_gamma(T, gamma, W_MAX) for T in LENGTHS]
    cfg = B.make_config(Bn, H, Hk, d, T_max, "bf16", source=B.DELTA_SRC_KEY if key else B.DELTA_SRC_QUERY)
    st = B.delta_state_init(cfg)
    # packed queries, cache-layout keys and values (rows past a sequence's end NaN)
    q_packed = np.concatenate([s["q"].reshape(-1) for s in seqs])
    kc = np.full((Bn, Hk, T_max, d), np.nan, np.float32)
    vc = np.full((Bn, Hk, T_max, d), np.nan, np.float32)
    for b, s in enumerate(seqs):
        kc[b, :, :LENGTHS[b]] = s["k"]
        vc[b, :, :LENGTHS[b]] = s["v"]
    dq_, dk_, dv_ = to_dev(q_packed, "bf16"), torch.from_numpy(kc).to(torch.bfloat16).cuda(), \
        torch.from_numpy(vc).to(torch.bfloat16).cuda()
    out = torch.full_like(dq_, float("nan"))
    B.delta_attn_prefill_varlen(st, dq_, dk_, dv_, out, LENGTHS, windows, theta)
    torch.cuda.synchronize()
    assert B.delta_state_position(st) == max(LENGTHS)
    assert [B.delta_state_sequence_position(st, b) for b in range(Bn)] == list(LENGTHS)
    o = to_host_f64(out)
    states, off = {}, 0
    pre = []
    for b, (s, T, W) in enumerate(zip(seqs, LENGTHS, windows)):
        ref, heads = O.prefill_mha(s["q"][None], s["k"][None], s["v"][None], theta, W, "block", source=source)
        _check_out(o[off:off + H * T * d].reshape(H, T, d), ref[0], "bf16", f"sequence {b} (T={T}, W={W})")
        off += H * T * d
        for h in range(H):
            r = heads[(0, h)]
            if key:
                if h % g == 0:
                    states[(b, h // g)] = r["state"]
                    pre.append(O.stage_stats_key(r["delta"]["row_nnz"], T, d, W, "block", g))
            else:
                states[(b, h)] = r["state"]
                pre.append(O.stage_stats(r["delta"]["row_nnz"], list(range(T)), d, W, "block"))
    # Eq. 6 over the ragged batch: counters add, W/n is sum min(W_b, n_b) / sum n_b
    want = O.finish_stats({key_: sum(c[key_] for c in pre) for key_ in ("nnz", "elements", "macs_done", "macs_dense")},
                          sum(min(W, T) for W, T in zip(windows, LENGTHS)), sum(LENGTHS))
    got = B.delta_sparsity_stats(st)
    assert got["device_status"] == 0
    for key_ in ("nnz", "elements", "macs_done", "macs_dense"):
        assert got["prefill"][key_] == want[key_], key_
    assert got["prefill"]["S_c_eq6"] == pytest.approx(want["S_c_eq6"], abs=1e-12)
    # decode: every sequence advances from where it stands
    for step in range(steps):
        qn = np.stack([s["q_dec"][:, step] for s in seqs])
        kn = np.stack([s["k_dec"][:, step] for s in seqs])
        vn = np.stack([s["v_dec"][:, step] for s in seqs])
        od = torch.full((Bn, H, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.delta_attn_decode_step(st, to_dev(qn, "bf16"), to_dev(kn, "bf16"), to_dev(vn, "bf16"), dk_, dv_, od, theta, W_d)
        torch.cuda.synchronize()
        og = to_host_f64(od)
        for b in range(Bn):
            if key:
                sub = {(0, kvh): states[(b, kvh)] for kvh in range(Hk)}
                oref, _ = O.decode_mha_key(sub, qn[b:b + 1], kn[b:b + 1], vn[b:b + 1], theta, W_d)
                for kvh in range(Hk):
                    states[(b, kvh)] = sub[(0, kvh)]
            else:
                sub = {(0, h): states[(b, h)] for h in range(H)}
                oref, _ = O.decode_mha(sub, qn[b:b + 1], kn[b:b + 1], vn[b:b + 1], theta, W_d)
                for h in range(H):
                    states[(b, h)] = sub[(0, h)]
            _check_out(og[b], oref[0], "bf16", f"decode step {step}, sequence {b}")
            assert B.delta_state_sequence_position(st, b) == LENGTHS[b] + step + 1
            n = LENGTHS[b] + step
            assert torch.equal(dk_[b, :, n], to_dev(kn[b], "bf16"))
    assert B.delta_sparsity_stats(st)["device_status"] == 0


def test_varlen_argument_checks(B):
    cfg = B.make_config(2, 4, 2, 64, 128, "bf16")
    st = B.delta_state_init(cfg)
    x = torch.zeros(4 * 2 * 128 * 64, dtype=torch.bfloat16, device="cuda")
    for lens, wins, want in (((0, 5), (1, 1), B.DELTA_ERR_INVALID_ARG), ((5, 129), (1, 1), B.DELTA_ERR_CAPACITY),
                             ((5, 5), (1, -1), B.DELTA_ERR_INVALID_ARG)):
        with pytest.raises(B.DeltaError) as e:
            B.delta_attn_prefill_varlen(st, x, x, x, x, lens, wins, 0.1)
        assert e.value.status == want
    assert B.delta_state_position(st) == 0
