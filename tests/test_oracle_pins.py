"""Pins for the CPU oracle: it is checked against things other than itself.

Each test fixes the oracle to something the paper or the mathematics fixes:
textbook dense attention (Eq. 1) through an independent library routine,
hand-worked chains (tests/golden/), closed forms that follow from Eq. 2-4,
brute-force recounts written independently in this file, and the structural
statements of Section III-A (strategy 1 keeps row 0 exact, strategy 3 keeps
column 0 exact).  A planted mistake (dropped term, wrong sign, transposed
operand, off-by-one window) fails at least one of them; see
test_planted_mistakes_are_caught.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import delta_oracle as O
from paper_2507_19608_b200 import workloads as WL

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _ar1(T, d, seed, rho=0.9, bf16=False):
    rng = np.random.default_rng(seed)
    x = WL.ar1(rng, (), T, d, rho).astype(np.float32)
    return WL.round_to_bf16(x) if bf16 else x


def _qkv(T, d, seed, bf16=False):
    return _ar1(T, d, seed, bf16=bf16), _ar1(T, d, seed + 1, bf16=bf16), _ar1(T, d, seed + 2, bf16=bf16)


def _sdpa_causal(q, k, v):
    """Independent textbook routine for Eq. 1 with the causal mask (torch, float64)."""
    tq, tk, tv = (torch.from_numpy(np.asarray(x, np.float64))[None, None] for x in (q, k, v))
    return torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0, 0].numpy()


# ------------------------------------------------------------------ golden chains (Eq. 2-3)
def _read_chains():
    rows = []
    with open(os.path.join(GOLDEN, "delta_chains.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, init, theta, a, dq, ahat, fired = [x.strip() for x in line.split("|")]
            f32 = lambda s: np.array([float(x) for x in s.split()], np.float32)
            rows.append((name, init, float(theta), f32(a), f32(dq), f32(ahat),
                         np.array([int(x) for x in fired.split()], bool)))
    return rows


@pytest.mark.parametrize("chain", _read_chains(), ids=lambda c: c[0])
def test_golden_chain(chain):
    name, init, theta, a, dq, ahat, fired = chain
    T = len(a)
    # put the chain in channel 5 of a 32-wide stream; the other channels hold a constant
    x = np.full((T, 32), 7.0, np.float32)
    x[:, 5] = a
    r = O.delta_construct(x, theta, init)
    assert np.array_equal(r["dq"][:, 5], dq)
    assert np.array_equal(r["ahat_rows"][:, 5], ahat)
    assert np.array_equal(r["fired"][:, 5], fired)
    assert np.array_equal((r["mask"][:, 0] >> 5) & 1, fired.astype(np.uint32))
    # the constant channels fire only where the init rule says row 0 fires
    other_fired_row0 = (init == "basis_exact") or (7.0 > theta)
    assert r["fired"][0, 0] == other_fired_row0
    assert not r["fired"][1:, 0].any()


def test_golden_tiny_hybrid():
    rows = {}
    with open(os.path.join(GOLDEN, "tiny_hybrid.txt")) as f:
        for line in f:
            if line.startswith("row"):
                name, vals = line.split("|")
                rows[name.strip()] = [float(x) for x in vals.split()]
    # head_dim must be a multiple of 32 for the mask layout: pad with zero channels, which add
    # nothing to any dot product.  The worked example has head_dim 1, so the softmax is re-run
    # below on the oracle's un-scaled hybrid scores with d_head = 1.
    d = 32
    q = np.zeros((3, d), np.float32); k = np.zeros((3, d), np.float32); v = np.zeros((3, d), np.float32)
    q[:, 0] = [1.0, 1.0625, 2.0]
    k[:, 0] = [1.0, 2.0, 3.0]
    v[0, 0] = v[1, 1] = v[2, 2] = 1.0
    r = O.prefill_head(q, k, v, theta=0.125, W=1, shape="block")
    assert np.allclose(r["S_star"][1, :2], [1.0, 2.125], atol=0, rtol=0)
    assert np.allclose(r["S_star"][2, :3], [2.0, 4.0, 6.0], atol=0, rtol=0)
    assert np.array_equal(r["delta"]["dq"][:, 0], np.array([1.0, 0.0, 1.0], np.float32))
    out = O.causal_softmax_v(r["S_star"], v, d_head=1)
    for i in range(3):
        assert np.allclose(out[i, :3], rows[f"row{i}"], atol=1e-15)


# ------------------------------------------------------------------ P1/P3/P10: dense special cases
@pytest.mark.parametrize("shape", ["block", "sliding"])
def test_theta0_full_window_is_dense_attention(shape):
    q, k, v = _qkv(96, 64, 11)
    r = O.prefill_head(q, k, v, theta=0.0, W=96, shape=shape)
    ref = _sdpa_causal(q, k, v)
    assert np.max(np.abs(r["out"] - ref)) < 1e-12


def test_any_theta_full_window_is_dense_attention():
    q, k, v = _qkv(80, 32, 12)
    r = O.prefill_head(q, k, v, theta=0.7, W=200, shape="block")
    assert np.max(np.abs(r["out"] - _sdpa_causal(q, k, v))) < 1e-12


def test_theta0_no_window_is_dense_up_to_rounding():
    q, k, v = _qkv(200, 64, 13)
    r = O.prefill_head(q, k, v, theta=0.0, W=0, shape="block")
    ref = _sdpa_causal(q, k, v)
    assert np.max(np.abs(r["out"] - ref)) < 1e-5
    # and for bf16 inputs every delta is exact in float32, so the match is at float64 level
    q, k, v = _qkv(200, 64, 13, bf16=True)
    r = O.prefill_head(q, k, v, theta=0.0, W=0, shape="block")
    assert np.max(np.abs(r["out"] - _sdpa_causal(q, k, v))) < 1e-10


def test_constant_stream_is_exact_and_maximally_sparse():
    T, d = 50, 32
    q = np.tile(_ar1(1, d, 3), (T, 1))
    _, k, v = _qkv(T, d, 4)
    r = O.prefill_head(q, k, v, theta=0.3, W=4, shape="block")
    assert np.max(np.abs(r["out"] - _sdpa_causal(q, k, v))) < 1e-12
    st = O.prefill_stats(r["delta"]["row_nnz"], T, d, 4, "block")
    assert st["S_m"] == pytest.approx((T - 1) / T)


# ------------------------------------------------------------------ P2: in-window scores are exact
@pytest.mark.parametrize("shape,W", [("block", 16), ("sliding", 16), ("block", 7), ("sliding", 1)])
def test_in_window_scores_equal_full_attention(shape, W):
    T, d = 70, 64
    q, k, v = _qkv(T, d, 21)
    r = O.prefill_head(q, k, v, theta=0.4, W=W, shape=shape)
    n_diff = 0
    for i in range(T):
        for j in range(i + 1):
            exact = float(np.dot(q[i].astype(np.float64), k[j].astype(np.float64)))
            inside = (i // W == j // W) if shape == "block" else (i - j < W)
            if inside:
                assert abs(r["S_star"][i, j] - exact) < 1e-12
            else:
                n_diff += abs(r["S_star"][i, j] - exact) > 1e-3
    assert n_diff > 100        # outside the window the scores really are approximate


# ------------------------------------------------------------------ P4: closed form of Eq. 4
def test_recursion_telescopes_to_reference_state():
    T, d = 150, 64
    q, k, _ = _qkv(T, d, 31, bf16=True)
    dl = O.delta_construct(q, 0.2)
    R = O.delta_scores_query(dl["dq"], k)
    closed = dl["ahat_rows"].astype(np.float64) @ k.astype(np.float64).T
    assert np.max(np.abs(R - closed)) < 1e-10      # bf16 - bf16 is exact in float32
    qf, kf, _ = _qkv(T, d, 32, bf16=False)
    dl = O.delta_construct(qf, 0.2)
    R = O.delta_scores_query(dl["dq"], kf)
    closed = dl["ahat_rows"].astype(np.float64) @ kf.astype(np.float64).T
    assert np.max(np.abs(R - closed)) < 1e-4       # float32 subtraction rounding only
    assert np.max(np.abs(R - closed)) > 0.0


def test_key_recursion_telescopes_to_reference_keys():
    T, d = 90, 32
    q, k, _ = _qkv(T, d, 33, bf16=True)
    dl = O.delta_construct(k, 0.25)
    S = O.delta_scores_key(q, dl["dq"])
    closed = q.astype(np.float64) @ dl["ahat_rows"].astype(np.float64).T
    assert np.max(np.abs(S - closed)) < 1e-10


# ------------------------------------------------------------------ P5: huge threshold
def test_huge_theta_freezes_the_basis_row():
    T, d = 40, 32
    q, k, v = _qkv(T, d, 41)
    r = O.prefill_head(q, k, v, theta=1e9, W=0, shape="block")
    first = k.astype(np.float64) @ q[0].astype(np.float64)
    for i in range(T):
        assert np.max(np.abs(r["S_delta"][i] - first)) < 1e-12
    st = O.prefill_stats(r["delta"]["row_nnz"], T, d, 0, "block")
    assert st["S_m"] == pytest.approx((T - 1) / T)
    assert st["nnz"] == d


# ------------------------------------------------------------------ P6: brute-force recount
@pytest.mark.parametrize("T,d,theta,init", [(130, 64, 0.3, "basis_exact"), (65, 128, 0.1, "zero_state"),
                                            (1, 32, 0.5, "basis_exact"), (64, 32, 0.0, "basis_exact")])
def test_mask_counts_indices_match_bruteforce_recount(T, d, theta, init):
    a = _ar1(T, d, 51)
    r = O.delta_construct(a, theta, init)
    # independent scalar re-run of Eq. 2-3, element by element, in float32
    th = np.float32(theta)
    nnz_total = 0
    for c in range(d):
        ref = np.float32(0.0)
        for t in range(T):
            if t == 0 and init == "basis_exact":
                fire, delta = True, a[0, c]
            else:
                diff = np.float32(a[t, c] - ref)
                fire = bool(abs(diff) > th)
                delta = diff if fire else np.float32(0.0)
            if fire:
                ref = a[t, c]
            assert r["dq"][t, c] == delta
            assert bool((r["mask"][t, c // 32] >> np.uint32(c % 32)) & 1) == fire
            assert r["ahat_rows"][t, c] == ref
            nnz_total += fire
    for t in range(T):
        bits = [c for c in range(d) if (int(r["mask"][t, c // 32]) >> (c % 32)) & 1]
        assert r["row_nnz"][t] == len(bits)
        assert list(r["idx"][t, :len(bits)]) == bits
        assert np.all(r["idx"][t, len(bits):] == 0xFF)
        if not (t == 0 and init == "basis_exact"):
            assert set(np.nonzero(r["dq"][t])[0]) == set(bits)      # fired <=> non-zero delta
    for tile in range((T + 63) // 64):
        assert r["tile_nnz"][tile] == int(r["row_nnz"][tile * 64:(tile + 1) * 64].astype(np.int64).sum())
    assert int(r["tile_nnz"].astype(np.int64).sum()) == nnz_total
    # per-tile snapshots: state before the tile's first row
    for tile in range((T + 63) // 64):
        want = np.zeros(d, np.float32) if tile == 0 else r["ahat_rows"][tile * 64 - 1]
        assert np.array_equal(r["ahat_tile"][tile], want)


def test_ties_negative_zero_nan_subnormal():
    th = np.float32(0.1)
    a = np.zeros((6, 32), np.float32)
    a[:, 0] = [1.0, np.float32(1.0) + th, 1.0, 1.0, 1.0, 1.0]          # |diff| vs theta at rounding level
    a[:, 1] = [0.0, -0.0, 0.0, 1e-40, 0.0, 0.0]                        # -0.0 and a subnormal
    a[:, 2] = [1.0, np.nan, 1.0, 2.0, 2.0, 2.0]                        # NaN never fires, state survives
    r = O.delta_construct(a, th)
    d1 = np.float32(a[1, 0] - a[0, 0])
    assert r["fired"][1, 0] == bool(abs(d1) > th)
    assert not r["fired"][1, 1] and not np.signbit(r["dq"][1, 1])      # stored as +0.0
    r0 = O.delta_construct(a, 0.0)
    assert r0["fired"][3, 1] and r0["dq"][3, 1] == np.float32(1e-40)   # subnormal difference fires at theta=0
    assert not r["fired"][1, 2] and r["ahat_rows"][1, 2] == 1.0
    assert not r["fired"][2, 2] and r["fired"][3, 2]


# ------------------------------------------------------------------ P7: what stays exact (Section III-A)
def test_query_deltas_keep_row0_exact_key_deltas_keep_col0_exact():
    T, d = 60, 32
    q, k, v = _qkv(T, d, 61)
    exact = q.astype(np.float64) @ k.astype(np.float64).T
    rq = O.prefill_head(q, k, v, theta=0.5, W=0, source="query")
    assert np.max(np.abs(rq["S_delta"][0] - exact[0])) < 1e-12
    assert np.max(np.abs(rq["S_delta"][1:] - exact[1:])) > 1e-2
    rk = O.prefill_head(q, k, v, theta=0.5, W=0, source="key")
    assert np.max(np.abs(rk["S_delta"][:, 0] - exact[:, 0])) < 1e-12
    assert np.max(np.abs(rk["S_delta"][:, 1:] - exact[:, 1:])) > 1e-2
    # strategy (2): the basis is the last row
    rb = O.prefill_head(q, k, v, theta=0.5, W=0, source="query", order="bottom_up")
    assert np.max(np.abs(rb["S_delta"][T - 1] - exact[T - 1])) < 1e-12
    assert np.max(np.abs(rb["S_delta"][:T - 1] - exact[:T - 1])) > 1e-2


def test_bottom_up_scores_follow_the_reverse_chain_closed_form():
    """Strategy (2): with the rows taken from the last to the first, the score row of token i is
    the reference after rows T-1 .. i, dotted with the keys (Eq. 4 telescoped).  The reference is
    re-derived here by a scalar loop of Eq. 2-3 that shares nothing with the oracle."""
    T, d, theta = 40, 32, 0.4
    q, k, v = _qkv(T, d, 83)
    r = O.prefill_head(q, k, v, theta=theta, W=0, source="query", order="bottom_up")
    ref = np.zeros(d, np.float32)
    want = np.zeros((T, T))
    for i in range(T - 1, -1, -1):
        for c in range(d):
            if i == T - 1:
                ref[c] = q[i, c]                       # the basis row is kept whole
            else:
                diff = np.float32(q[i, c]) - ref[c]
                if abs(diff) > np.float32(theta):
                    ref[c] = q[i, c]
        want[i] = ref.astype(np.float64) @ k.astype(np.float64).T
    assert np.max(np.abs(r["S_delta"] - want)) < 1e-4
    # a wrong direction would put the exact row at the top
    assert np.max(np.abs(r["S_delta"][0] - q[0].astype(np.float64) @ k.astype(np.float64).T)) > 1e-2


def test_bottom_up_is_top_down_on_the_mirrored_sequence():
    """Delta construction of strategy (2) over q equals that of strategy (1) over q reversed,
    row for row (Section III-A describes the two as the same procedure from opposite ends)."""
    T, d, theta = 70, 32, 0.3
    q, k, v = _qkv(T, d, 19)
    rb = O.prefill_head(q, k, v, theta=theta, W=5, source="query", order="bottom_up")
    rt = O.delta_construct(q[::-1], theta)
    assert np.array_equal(rb["delta"]["mask"], rt["mask"])
    assert np.array_equal(rb["delta"]["dq"].view(np.uint32), rt["dq"].view(np.uint32))
    # and the hybrid output still takes exact scores inside the window
    exact = q.astype(np.float64) @ k.astype(np.float64).T
    win = O.window_matrix(T, 5, "block")
    assert np.array_equal(rb["S_star"][win], exact[win])


# ------------------------------------------------------------------ P8: window geometry and Eq. 5-6
@pytest.mark.parametrize("T,W", [(128, 16), (100, 16), (64, 64), (33, 7), (10, 0), (10, 50)])
def test_window_pair_counts_closed_form(T, W):
    blk = O.window_matrix(T, W, "block").sum()
    sld = O.window_matrix(T, W, "sliding").sum()
    if W == 0:
        assert blk == 0 and sld == 0
        return
    full, rem = divmod(T, W)
    assert blk == full * W * (W + 1) // 2 + rem * (rem + 1) // 2
    assert sld == sum(min(i + 1, W) for i in range(T))
    # sliding window holds exactly the W most recent tokens, the current one included
    m = O.window_matrix(T, W, "sliding")
    i = T - 1
    if W <= i:
        assert m[i, i - W + 1] and not m[i, i - W]
    assert not np.triu(O.window_matrix(T, W, "block"), 1).any()


def test_eq5_window_from_gamma():
    assert O.window_from_gamma(1000, 0.05, 64) == 50
    assert O.window_from_gamma(1000, 0.1, 64) == 64
    assert O.window_from_gamma(10, 0.05, 64) == 0
    assert O.window_from_gamma(120, 0.25, 1 << 30) == 30


def test_exact_sparsity_close_to_eq6_and_counts_recounted():
    T, d, W = 256, 64, 16
    q = _ar1(T, d, 71, rho=0.95)
    dl = O.delta_construct(q, 0.3)
    st = O.prefill_stats(dl["row_nnz"], T, d, W, "block")
    # independent recount straight from the delta values and the predicate
    done = dense = 0
    for i in range(T):
        nz = d if i == 0 else int(np.count_nonzero(dl["dq"][i]))
        for j in range(i + 1):
            done += d if (i // W == j // W) else nz
            dense += d
    assert st["macs_done"] == done and st["macs_dense"] == dense
    assert st["nnz"] == d + int(np.count_nonzero(dl["dq"][1:]))
    assert st["S_c_eq6"] == pytest.approx(st["S_m"] * (1 - W / T))
    assert abs(st["S_c_exact"] - st["S_c_eq6"]) < 0.05
    assert 0.2 < st["S_m"] < 0.9


# ------------------------------------------------------------------ P12: prefill/decode consistency
@pytest.mark.parametrize("W", [0, 1, 5, 40])
def test_decode_continues_prefill(W):
    T, d, steps = 37, 32, 6
    q, k, v = _qkv(T + steps, d, 81)
    full = O.prefill_head(q, k, v, theta=0.3, W=W, shape="sliding")
    part = O.prefill_head(q[:T], k[:T], v[:T], theta=0.3, W=W, shape="sliding")
    st = part["state"]
    for s in range(steps):
        out, st, info = O.decode_head(st, q[T + s], k[T + s], v[T + s], 0.3, W)
        assert np.max(np.abs(out - full["out"][T + s])) < 1e-12
        assert info["row_nnz"] == full["delta"]["row_nnz"][T + s]
        assert np.array_equal(info["dq"], full["delta"]["dq"][T + s])
    assert np.max(np.abs(st["R"] - full["S_delta"][T + steps - 1])) < 1e-12
    assert np.array_equal(st["qhat"], full["delta"]["ahat"])


def test_decode_new_key_score_is_reference_dot_key():
    T, d = 20, 32
    q, k, v = _qkv(T + 1, d, 91, bf16=True)
    st = O.prefill_head(q[:T], k[:T], v[:T], 0.3, 4, "sliding")["state"]
    _, st2, _ = O.decode_head(st, q[T], k[T], v[T], 0.3, 4)
    assert abs(st2["R"][T] - float(st2["qhat"].astype(np.float64) @ k[T].astype(np.float64))) < 1e-10


# ------------------------------------------------------------------ GQA mapping and multi-head wrapper
def test_gqa_head_mapping():
    B, H, Hkv, T, d = 2, 4, 2, 24, 32
    rng = np.random.default_rng(5)
    q = rng.standard_normal((B, H, T, d)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, T, d)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, T, d)).astype(np.float32)
    out, _ = O.prefill_mha(q, k, v, theta=0.0, W=T, shape="block")
    tk = torch.from_numpy(k.astype(np.float64)).repeat_interleave(H // Hkv, dim=1)
    tv = torch.from_numpy(v.astype(np.float64)).repeat_interleave(H // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q.astype(np.float64)), tk, tv,
                                                           is_causal=True).numpy()
    assert np.max(np.abs(out - ref)) < 1e-12


# ------------------------------------------------------------------ the pins bite
def test_planted_mistakes_are_caught(monkeypatch):
    """Each planted mistake (on the CPU, in the oracle) must break at least one pin above."""
    q, k, v = _qkv(48, 32, 101, bf16=True)
    dl = O.delta_construct(q, 0.2)
    closed = dl["ahat_rows"].astype(np.float64) @ k.astype(np.float64).T

    # (a) recursion without the carried term: R(t) = Delta q(t) K^T only
    bad = dl["dq"].astype(np.float64) @ k.astype(np.float64).T
    assert np.max(np.abs(bad - closed)) > 1e-2
    # (b) sign flipped in Eq. 2
    bad = np.cumsum((-dl["dq"][1:]).astype(np.float64) @ k.astype(np.float64).T, axis=0)
    assert np.max(np.abs(bad - closed[1:])) > 1e-2
    # (c) reference = previous input instead of last fired value: golden chain B fails
    a = np.array([0.25 * t for t in range(10)], np.float32)
    prev_diff_fires = np.abs(np.diff(a)) > 0.5
    assert not prev_diff_fires.any()          # that reading would never fire, golden B says it fires 3 times
    # (d) no 1/sqrt(d) scale: dense special case breaks
    S = O.dense_scores(q, k)
    wrong = O.causal_softmax_v(S, v, d_head=1)
    assert np.max(np.abs(wrong - _sdpa_causal(q, k, v))) > 1e-3


# ------------------------------------------------------------------ input generator sanity (host logic)
def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(100000) * 10.0 ** rng.integers(-10, 10, 100000)).astype(np.float32)
    mine = WL.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(mine, ref)
    assert np.array_equal(WL.bits_to_f32(WL.bf16_bits(mine)), mine)


def test_workload_generator_is_seeded_and_ar1():
    w = WL.WORKLOADS["single_head_fp32"]
    a = WL.make_qkv(w)
    b = WL.make_qkv(w)
    assert all(np.array_equal(a[n], b[n]) for n in a)
    assert a["q"].shape == (1, 1, 128, 64) and a["q"].dtype == np.float32
    w2 = WL.WORKLOADS["llama32_1b_prefill"]
    t = WL.make_qkv(w2, T=512)
    x = t["q"][0, 0].astype(np.float64)
    r1 = np.mean([np.corrcoef(x[1:, c], x[:-1, c])[0, 1] for c in range(x.shape[1])])
    assert 0.85 < r1 < 0.99                       # lag-1 autocorrelation near rho = 0.95
    assert np.array_equal(WL.round_to_bf16(t["k"]), t["k"])


def test_key_delta_counters_closed_forms():
    """Key-delta counters: all-dense deltas cost exactly the dense multiply-adds; all-zero deltas
    outside a block window cost only the in-window pairs (closed form of the block sizes)."""
    T, d, W = 50, 64, 8
    full = O.stage_stats_key(np.full(T, d), T, d, W, "block", g=4)
    assert full["macs_done"] == full["macs_dense"] == 4 * d * T * (T + 1) // 2
    none = O.stage_stats_key(np.zeros(T, int), T, d, W, "block", g=1)
    blocks, rem = divmod(T, W)
    n_in = blocks * W * (W + 1) // 2 + rem * (rem + 1) // 2
    assert none["macs_done"] == d * n_in and none["nnz"] == 0 and none["elements"] == T * d
    slid = O.stage_stats_key(np.zeros(T, int), T, d, W, "sliding")
    assert slid["macs_done"] == d * sum(min(i + 1, W) for i in range(T))


@pytest.mark.parametrize("W", [0, 3, 8, 100])
def test_key_delta_decode_continues_prefill(W):
    """Strategy (3): prefill over T + s tokens (sliding window) and prefill over T tokens followed
    by s decode steps give the same rows (the decode step is the column recursion continued)."""
    rng = np.random.default_rng(11)
    T, s_steps, d, theta = 20, 5, 32, 0.4
    q = rng.standard_normal((T + s_steps, d)).astype(np.float32)
    k = np.cumsum(0.3 * rng.standard_normal((T + s_steps, d)), axis=0).astype(np.float32)
    v = rng.standard_normal((T + s_steps, d)).astype(np.float32)
    full = O.prefill_head(q, k, v, theta, W, "sliding", source="key")
    st = O.prefill_head(q[:T], k[:T], v[:T], theta, W, "sliding", source="key")["state"]
    for s in range(s_steps):
        st, info = O.decode_key_step(st, k[T + s], v[T + s], theta)
        out = O.decode_key_attend(st, q[T + s], W)
        assert np.allclose(out, full["out"][T + s], rtol=1e-12, atol=1e-12)
        assert np.array_equal(info["dk"], full["delta"]["dq"][T + s])
    assert np.array_equal(st["khat"], full["delta"]["ahat"])


# ------------------------------------------------------------------ key-delta counters, non-uniform counts
@pytest.mark.parametrize("shape,W,g", [("block", 5, 1), ("block", 8, 4), ("sliding", 3, 2), ("sliding", 7, 1)])
def test_key_delta_counters_recounted_with_uneven_rows(shape, W, g):
    """stage_stats_key against a recount written out here: the cost of an out-of-window pair
    (i, j) is the fired count of KEY row j (its column), not of the query row i.  The fired
    counts differ from row to row, so taking the wrong index changes the total."""
    T, d = 23, 32
    k = np.cumsum(0.25 * np.random.default_rng(17).standard_normal((T, d)), axis=0).astype(np.float32)
    dl = O.delta_construct(k, 0.35)
    rn = dl["row_nnz"].astype(int)
    assert len(set(rn.tolist())) > 5                      # really uneven
    done = dense = 0
    for i in range(T):                                    # query row
        for j in range(i + 1):                            # key column
            inside = W > 0 and ((i // W == j // W) if shape == "block" else (i - j < W))
            nz_key_j = d if j == 0 else int(np.count_nonzero(dl["dq"][j]))
            done += d if inside else nz_key_j
            dense += d
    got = O.stage_stats_key(dl["row_nnz"], T, d, W, shape, g)
    assert got["macs_done"] == g * done and got["macs_dense"] == g * dense
    assert got["nnz"] == int(rn.sum()) and got["elements"] == T * d
    # the transposed reading (query row's count) gives another total on this input
    wrong = sum((d if (W > 0 and ((i // W == j // W) if shape == "block" else (i - j < W))) else rn[i])
                for i in range(T) for j in range(i + 1))
    assert wrong != done


# ------------------------------------------------------------------ GQA mapping of the decode wrappers
def _sdpa_last_row_gqa(q_new, k_all, v_all):
    """fp64 attention of one new query per head over all keys, KV heads repeated per group."""
    H, Hkv = q_new.shape[1], k_all.shape[1]
    tq = torch.from_numpy(q_new.astype(np.float64))[:, :, None, :]
    tk = torch.from_numpy(k_all.astype(np.float64)).repeat_interleave(H // Hkv, dim=1)
    tv = torch.from_numpy(v_all.astype(np.float64)).repeat_interleave(H // Hkv, dim=1)
    return torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[:, :, 0].numpy()


def test_decode_wrappers_gqa_head_mapping_against_sdpa():
    """decode_mha and decode_mha_key with theta = 0 and a window over the whole cache are plain
    attention of the new query: query head h must read KV head h // (H / H_kv) -- checked against
    torch SDPA in fp64 with the KV heads repeated per group, on heads that all differ."""
    B, H, Hkv, T, d, steps = 2, 4, 2, 9, 32, 2
    rng = np.random.default_rng(23)
    q = rng.standard_normal((B, H, T + steps, d)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, T + steps, d)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, T + steps, d)).astype(np.float32)
    W = T + steps + 1
    _, heads_q = O.prefill_mha(q[:, :, :T], k[:, :, :T], v[:, :, :T], 0.0, W, "sliding")
    _, heads_k = O.prefill_mha(q[:, :, :T], k[:, :, :T], v[:, :, :T], 0.0, W, "sliding", source="key")
    st_q = {key: r["state"] for key, r in heads_q.items()}
    st_k = {(b, kvh): heads_k[(b, kvh * (H // Hkv))]["state"] for b in range(B) for kvh in range(Hkv)}
    for s in range(steps):
        n = T + s
        ref = _sdpa_last_row_gqa(q[:, :, n], k[:, :, :n + 1], v[:, :, :n + 1])
        out_q, _ = O.decode_mha(st_q, q[:, :, n], k[:, :, n], v[:, :, n], 0.0, W)
        out_k, _ = O.decode_mha_key(st_k, q[:, :, n], k[:, :, n], v[:, :, n], 0.0, W)
        assert np.max(np.abs(out_q - ref)) < 1e-12
        assert np.max(np.abs(out_k - ref)) < 1e-12
    # the other mapping (h % H_kv) is a different function on this input
    wrong_k = np.stack([k[:, h % Hkv] for h in range(H)], axis=1)
    wrong_v = np.stack([v[:, h % Hkv] for h in range(H)], axis=1)
    wrong = _sdpa_last_row_gqa(q[:, :, T], wrong_k[:, :, :T + 1], wrong_v[:, :, :T + 1])
    assert np.max(np.abs(wrong - _sdpa_last_row_gqa(q[:, :, T], k[:, :, :T + 1], v[:, :, :T + 1]))) > 1e-3


# ------------------------------------------------------------------ Eq. 6 over stages (hand-worked fixture)
def _read_eq6_fixture():
    rows = {}
    with open(os.path.join(GOLDEN, "eq6_two_stage.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, *vals = [x.strip() for x in line.split("|")]
            rows[name] = dict(nnz=int(vals[0]), elements=int(vals[1]), macs_done=int(vals[2]), macs_dense=int(vals[3]),
                              S_m=float(vals[4]), S_c_eq6=float(vals[5]), S_c_exact=float(vals[6]))
    return rows


def test_eq6_stage_aggregates_match_hand_worked_example():
    want = _read_eq6_fixture()
    d = 2
    pre = O.prefill_stats([2, 1], 2, d, 1, "block")
    steps = [O.stage_stats([0], [2], d, 1, "sliding"), O.stage_stats([2], [3], d, 1, "sliding")]
    raw = {key: sum(s[key] for s in steps) for key in ("nnz", "elements", "macs_done", "macs_dense")}
    dec = O.decode_stage_stats(raw, windows=[1, 1], lengths=[3, 4])
    both = O.combined_stats(pre, dec)
    for name, got in (("prefill", pre), ("decode", dec), ("combined", both)):
        for key in ("nnz", "elements", "macs_done", "macs_dense"):
            assert got[key] == want[name][key], (name, key)
        for key in ("S_m", "S_c_eq6", "S_c_exact"):
            assert got[key] == pytest.approx(want[name][key], abs=1e-15), (name, key)
    # a window longer than a step's sequence counts as the sequence length
    assert O.decode_stage_stats(raw, [10, 10], [3, 4])["S_c_eq6"] == 0.0
