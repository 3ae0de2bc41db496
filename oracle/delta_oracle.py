"""CPU oracle for DeltaLLM's delta attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library must compute.
Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import it; the product (the CUDA library and its Python binding) never does,
and the two share no code.  Everything here is numpy: Eq. 2-3 run in float32
(that is the precision in which the fire/no-fire decision is defined), every
dot product, the softmax and the weighted sum run in float64.  There is no
tiling, fusion or reordering beyond what the equations state.

Notation follows the paper: a(t) input vector, a_hat(t) reference state,
Delta a(t) delta vector, theta threshold (Eq. 2-3); R(t) recursive product
(Eq. 4); W context window (Section III-B); S_m, S_c sparsities (Eq. 6).

Readings of points the paper leaves open (each one is a named argument so the
tests can exercise the alternatives):
  * init="basis_exact": row 0 is the un-thresholded basis vector, Delta a(0) =
    a(0) and a_hat(0) = a(0) (the delta matrix of Section II-C has the basis
    vector as its first row; strategy 1 of Section III-A keeps the first
    attention row dense).  init="zero_state": the reference starts at zero, as
    the sentence after Eq. 3 has it, and Eq. 2-3 are applied at t = 0 as well.
  * the threshold is per element; |diff| == theta does not fire (Eq. 2 uses >).
  * window shape "block": squares of side W along the diagonal anchored at
    token 0 (Section III-B, prefill); "sliding": the most recent W tokens
    (Section III-B, decode).  W = 0 means no exact score at all.
  * source="query" is strategy (1) of Section III-A (deltas of Q, top-down);
    source="key" is strategy (3); order="bottom_up" with source="query" is
    strategy (2).
  * R(t) is its own stream: exact in-window scores never overwrite it.
  * 1/sqrt(d_head) scales exact and approximate scores alike (Eq. 1).

Parity pins: every function below is pinned by tests/test_oracle_pins.py
(dense-attention special cases, closed forms, hand-worked chains in
tests/golden/, brute-force recounts).  The paper's Table 1-3 sparsity values
are NOT reproduced (they need the models' weights and the benchmark text):
parity unpinned for those numbers only.
"""
from __future__ import annotations

import functools

import numpy as np

TILE_ROWS = 64  # rows per delta tile (per-tile counters and per-tile reference snapshots)

F32 = np.float32
F64 = np.float64


# --------------------------------------------------------------------------- Eq. 2-3
def delta_construct(a, theta, init="basis_exact"):
    """Thresholded delta vectors and reference states of one stream (Eq. 2-3).

    a: [T, d] float32 (rows are a(0..T-1)).  Returns a dict with
      dq        [T, d] float32  Delta a(t); +0.0 where the element did not fire
      fired     [T, d] bool
      mask      [T, d/32] uint32  bit (c % 32) of word (c // 32) set iff fired
      row_nnz   [T] uint16,  tile_nnz [ceil(T/64)] uint32
      idx       [T, d] uint8  fired channel ids ascending, padded with 0xFF
      ahat_rows [T, d] float32  reference state a_hat(t) after row t
      ahat_tile [ceil(T/64), d] float32  reference state before each tile's first row
      ahat      [d] float32  final reference state
    """
    a = np.ascontiguousarray(a, dtype=F32)
    T, d = a.shape
    assert d % 32 == 0 and d <= 256
    theta = F32(theta)
    n_tiles = (T + TILE_ROWS - 1) // TILE_ROWS
    ahat = np.zeros(d, F32)
    dq = np.zeros((T, d), F32)
    fired = np.zeros((T, d), bool)
    ahat_rows = np.zeros((T, d), F32)
    ahat_tile = np.zeros((n_tiles, d), F32)
    for t in range(T):
        if t % TILE_ROWS == 0:
            ahat_tile[t // TILE_ROWS] = ahat
        if t == 0 and init == "basis_exact":
            fire = np.ones(d, bool)                 # the basis vector is kept whole
            delta = a[0].copy()
        elif init in ("basis_exact", "zero_state"):
            diff = a[t] - ahat                      # one float32 subtraction (Eq. 2)
            fire = np.abs(diff) > theta             # strict >, NaN compares false
            delta = np.where(fire, diff, F32(0.0))
        else:
            raise ValueError(init)
        ahat = np.where(fire, a[t], ahat).astype(F32)   # Eq. 3
        dq[t] = delta
        fired[t] = fire
        ahat_rows[t] = ahat
    mask = np.zeros((T, d // 32), np.uint32)
    for c in range(d):
        mask[:, c // 32] |= (fired[:, c].astype(np.uint32) << np.uint32(c % 32))
    row_nnz = fired.sum(axis=1).astype(np.uint16)
    tile_nnz = np.zeros(n_tiles, np.uint32)
    for t in range(T):
        tile_nnz[t // TILE_ROWS] += row_nnz[t]
    idx = np.full((T, d), 0xFF, np.uint8)
    for t in range(T):
        ch = np.nonzero(fired[t])[0]
        idx[t, :len(ch)] = ch
    return dict(dq=dq, fired=fired, mask=mask, row_nnz=row_nnz, tile_nnz=tile_nnz, idx=idx,
                ahat_rows=ahat_rows, ahat_tile=ahat_tile, ahat=ahat)


# --------------------------------------------------------------------------- windows
def in_window(i, j, W, shape):
    """Is the causal pair (query i, key j <= i) inside the exact-attention window?"""
    if W <= 0:
        return False
    if shape == "block":
        return (i // W) == (j // W)
    if shape == "sliding":
        return (i - j) < W
    raise ValueError(shape)


@functools.lru_cache(maxsize=16)
def window_matrix(T, W, shape):
    """[T, T] bool, True where the pair is causal and in-window (cached per (T, W, shape))."""
    m = np.zeros((T, T), bool)
    for i in range(T):
        for j in range(i + 1):
            m[i, j] = in_window(i, j, W, shape)
    return m


def window_from_gamma(n, gamma, w_max):
    """Eq. 5: W_p,max = min(floor(gamma * n), W_max)."""
    return int(min(np.floor(F64(gamma) * n), w_max))


# --------------------------------------------------------------------------- Eq. 4
def delta_scores_query(dq, k):
    """Strategy (1): R(t) = Delta q(t) K^T + R(t-1), R(0) = Delta q(0) K^T (Eq. 4).

    Every key column takes part in the recursion, also the ones above the
    diagonal that the causal mask hides later.  Returns R as [T, T] float64,
    row t = R(t).
    """
    D = np.asarray(dq, F64) @ np.asarray(k, F64).T      # row t = Delta q(t) K^T
    return np.cumsum(D, axis=0)                         # running sum over t


def delta_scores_key(q, dk):
    """Strategy (3): column recursion S[:, j] = S[:, j-1] + Q Delta k(j)^T."""
    D = np.asarray(q, F64) @ np.asarray(dk, F64).T      # column j = Q Delta k(j)
    return np.cumsum(D, axis=1)


# --------------------------------------------------------------------------- Eq. 1
def causal_softmax_v(S, v, d_head):
    """softmax_{j<=i}(S[i][j] / sqrt(d_head)) @ V, row by row, float64."""
    S = np.asarray(S, F64)
    v = np.asarray(v, F64)
    T = S.shape[0]
    out = np.zeros((T, v.shape[1]), F64)
    scale = 1.0 / np.sqrt(F64(d_head))
    for i in range(T):
        s = S[i, :i + 1] * scale
        p = np.exp(s - s.max())
        p /= p.sum()
        out[i] = p @ v[:i + 1]
    return out


def dense_scores(q, k):
    return np.asarray(q, F64) @ np.asarray(k, F64).T


# --------------------------------------------------------------------------- prefill, one head
def prefill_head(q, k, v, theta, W, shape="block", init="basis_exact", source="query",
                 order="top_down"):
    """Hybrid delta attention of one head over T tokens (Section III).

    q, k, v: [T, d] float32.  Returns dict(out [T, d] float64, S_star [T, T]
    float64 (un-scaled hybrid scores; entries with j > i are meaningless),
    delta (the delta_construct dict of the source stream), state (decode state
    for source="query": n, qhat, R, dq_hist, k, v)).
    """
    q = np.ascontiguousarray(q, F32)
    k = np.ascontiguousarray(k, F32)
    v = np.ascontiguousarray(v, F32)
    T, d = q.shape
    if source == "query":
        if order == "top_down":
            delta = delta_construct(q, theta, init)
            S_delta = delta_scores_query(delta["dq"], k)
        elif order == "bottom_up":                     # strategy (2): basis is the last row
            delta = delta_construct(q[::-1], theta, init)
            S_delta = delta_scores_query(delta["dq"], k)[::-1]
        else:
            raise ValueError(order)
    elif source == "key":
        delta = delta_construct(k, theta, init)
        S_delta = delta_scores_key(q, delta["dq"])
    else:
        raise ValueError(source)
    S_exact = dense_scores(q, k)
    win = window_matrix(T, W, shape)
    S_star = np.where(win, S_exact, S_delta)           # exact inside the window, delta outside
    out = causal_softmax_v(S_star, v, d)
    state = None
    if source == "query" and order == "top_down":
        state = dict(n=T, qhat=delta["ahat"].copy(), R=S_delta[T - 1].copy(),
                     dq_hist=delta["dq"].copy(), k=k.copy(), v=v.copy())
    elif source == "key":
        state = dict(n=T, khat=delta["ahat"].copy(), dk_hist=delta["dq"].copy(), k=k.copy(), v=v.copy())
    return dict(out=out, S_star=S_star, S_delta=S_delta, S_exact=S_exact, delta=delta, state=state)


# --------------------------------------------------------------------------- decode, one head
def decode_head(state, q_new, k_new, v_new, theta, W_d):
    """One decode step of strategy (1) carried past prefill (Sections III-A/B/C).

    The new query row n continues Eq. 2-4: Delta q(n) against the carried
    reference, R(n)[j] = R(n-1)[j] + Delta q(n).k_j for the cached keys, and for
    the key that arrives with this step R(n)[n] = sum_{s<=n} Delta q(s).k_n
    (every past delta row is kept here so that this sum is literal).  The W_d
    most recent keys (the new one included) get the exact score q_new.k_j.
    Returns (out [d] float64, new_state, info dict with row_nnz and dq).
    """
    n = state["n"]
    d = q_new.shape[0]
    theta = F32(theta)
    q_new = np.asarray(q_new, F32)
    diff = q_new - state["qhat"]
    fire = np.abs(diff) > theta
    dq = np.where(fire, diff, F32(0.0)).astype(F32)
    qhat = np.where(fire, q_new, state["qhat"]).astype(F32)
    k_all = np.vstack([state["k"], np.asarray(k_new, F32)[None, :]])
    v_all = np.vstack([state["v"], np.asarray(v_new, F32)[None, :]])
    dq_hist = np.vstack([state["dq_hist"], dq[None, :]])
    R = np.empty(n + 1, F64)
    R[:n] = state["R"] + k_all[:n].astype(F64) @ dq.astype(F64)
    R[n] = np.sum(dq_hist.astype(F64) @ k_all[n].astype(F64))
    s = np.empty(n + 1, F64)
    for j in range(n + 1):
        s[j] = (q_new.astype(F64) @ k_all[j].astype(F64)) if in_window(n, j, W_d, "sliding") else R[j]
    s *= 1.0 / np.sqrt(F64(d))
    p = np.exp(s - s.max())
    p /= p.sum()
    out = p @ v_all.astype(F64)
    new_state = dict(n=n + 1, qhat=qhat, R=R, dq_hist=dq_hist, k=k_all, v=v_all)
    return out, new_state, dict(row_nnz=int(fire.sum()), dq=dq, fired=fire)


def decode_key_step(state, k_new, v_new, theta):
    """Key side of one decode step of strategy (3) for one KV head: Delta k(n) against the
    carried reference key (Eq. 2-3); the delta, the key and the value are appended to the
    cached histories.  Returns (new_state, info with row_nnz / dk / fired)."""
    theta = F32(theta)
    k_new = np.asarray(k_new, F32)
    diff = k_new - state["khat"]
    fire = np.abs(diff) > theta
    dk = np.where(fire, diff, F32(0.0)).astype(F32)
    khat = np.where(fire, k_new, state["khat"]).astype(F32)
    new_state = dict(n=state["n"] + 1, khat=khat, dk_hist=np.vstack([state["dk_hist"], dk[None, :]]),
                     k=np.vstack([state["k"], k_new[None, :]]),
                     v=np.vstack([state["v"], np.asarray(v_new, F32)[None, :]]))
    return new_state, dict(row_nnz=int(fire.sum()), dk=dk, fired=fire)


def decode_key_attend(state, q_new, W_d):
    """Query side of a strategy-(3) decode step, after decode_key_step appended the new key:
    the score of key j is q_new.k_j for the W_d most recent keys (the new one included) and the
    prefix sum of the cached delta products q_new.Delta k(0..j) for the older ones (the column
    recursion of Section III-A carried into decoding, Section III-C).  Returns out [d] float64."""
    n = state["n"] - 1                                   # index of the token that just arrived
    d = q_new.shape[0]
    q64 = np.asarray(q_new, F32).astype(F64)
    s_delta = np.cumsum(state["dk_hist"].astype(F64) @ q64)   # S[n][j] = S[n][j-1] + q.Delta k(j)
    s = np.empty(n + 1, F64)
    for j in range(n + 1):
        s[j] = (q64 @ state["k"][j].astype(F64)) if in_window(n, j, W_d, "sliding") else s_delta[j]
    s *= 1.0 / np.sqrt(F64(d))
    p = np.exp(s - s.max())
    p /= p.sum()
    return p @ state["v"].astype(F64)


def decode_mha_key(states, q_new, k_new, v_new, theta, W_d):
    """states: dict (b, kv head) -> key-delta state.  q_new [B,H,d], k_new,v_new [B,H_kv,d]."""
    B, H, d = q_new.shape
    H_kv = k_new.shape[1]
    g = H // H_kv
    out = np.zeros((B, H, d), F64)
    infos = {}
    for b in range(B):
        for kvh in range(H_kv):
            states[(b, kvh)], infos[(b, kvh)] = decode_key_step(states[(b, kvh)], k_new[b, kvh], v_new[b, kvh], theta)
            for hh in range(g):
                out[b, kvh * g + hh] = decode_key_attend(states[(b, kvh)], q_new[b, kvh * g + hh], W_d)
    return out, infos


# --------------------------------------------------------------------------- Eq. 6 and exact counts
def stage_stats(row_nnz, rows, d, W, shape):
    """Counters of one stage.  row_nnz[r] is the fired count of query row rows[r]
    (rows[r] = its token index, which has rows[r]+1 causal keys).

    nnz / elements give S_m; macs_done counts d per in-window pair and
    row_nnz per out-of-window pair; macs_dense = d per causal pair.  win_sum
    and len_sum aggregate Eq. 6's W and n over the rows' sequences.
    """
    nnz = int(np.sum(np.asarray(row_nnz, np.int64)))
    elements = len(rows) * d
    done = 0
    dense = 0
    for r, i in enumerate(rows):
        n_in = sum(1 for j in range(i + 1) if in_window(i, j, W, shape))
        n_out = (i + 1) - n_in
        done += n_in * d + n_out * int(row_nnz[r])
        dense += (i + 1) * d
    return dict(nnz=nnz, elements=elements, macs_done=done, macs_dense=dense)


def stage_stats_key(row_nnz, T, d, W, shape, g=1):
    """Counters of a prefill with key deltas (strategy 3): row_nnz[j] is the fired count of key
    row j of one KV head, which g query heads read.  A causal pair (i, j) costs d multiply-adds
    inside the window and row_nnz[j] outside it; nnz / elements count the key delta matrix."""
    nnz = int(np.sum(np.asarray(row_nnz, np.int64)))
    done = 0
    dense = 0
    for j in range(T):
        for i in range(j, T):
            done += d if in_window(i, j, W, shape) else int(row_nnz[j])
            dense += d
    return dict(nnz=nnz, elements=T * d, macs_done=g * done, macs_dense=g * dense)


def finish_stats(c, win_sum, len_sum):
    """S_m, Eq. 6 and the exact MAC-weighted sparsity from raw counters."""
    S_m = 1.0 - c["nnz"] / c["elements"] if c["elements"] else 0.0
    S_c_eq6 = S_m * (1.0 - win_sum / len_sum) if len_sum else 0.0
    S_c_exact = 1.0 - c["macs_done"] / c["macs_dense"] if c["macs_dense"] else 0.0
    return dict(c, S_m=S_m, S_c_eq6=S_c_eq6, S_c_exact=S_c_exact)


def prefill_stats(row_nnz, T, d, W, shape):
    c = stage_stats(row_nnz, list(range(T)), d, W, shape)
    return finish_stats(c, min(W, T), T)


def decode_stage_stats(counters, windows, lengths):
    """Decode stage of Eq. 6: the stage is a run of steps, step s attends lengths[s] keys (the
    new one included) with window windows[s]; Eq. 6's W/n becomes sum(min(W_s, n_s)) / sum(n_s)
    over the steps.  counters: the summed raw counters of the steps."""
    win_sum = sum(min(int(w), int(n)) for w, n in zip(windows, lengths))
    return finish_stats(counters, win_sum, sum(int(n) for n in lengths))


def combined_stats(prefill, decode):
    """Prefill and decode taken together (the paper's "both stages" figure): the raw counters add,
    S_m and the exact multiply-add sparsity follow from the sums, and the Eq. 6 value is the mean
    of the two stages' Eq. 6 values weighted by their dense multiply-adds."""
    c = {key: prefill[key] + decode[key] for key in ("nnz", "elements", "macs_done", "macs_dense")}
    out = finish_stats(c, 0, 0)
    dense = c["macs_dense"]
    out["S_c_eq6"] = ((prefill["S_c_eq6"] * prefill["macs_dense"] + decode["S_c_eq6"] * decode["macs_dense"]) / dense
                      if dense else 0.0)
    return out


# --------------------------------------------------------------------------- multi-head wrappers
def prefill_mha(q, k, v, theta, W, shape="block", init="basis_exact", source="query", order="top_down"):
    """q [B,H,T,d], k,v [B,H_kv,T,d] -> out [B,H,T,d] float64 plus per-head results.
    Query head h reads KV head h // (H / H_kv)."""
    B, H, T, d = q.shape
    H_kv = k.shape[1]
    g = H // H_kv
    out = np.zeros((B, H, T, d), F64)
    heads = {}
    for b in range(B):
        for h in range(H):
            r = prefill_head(q[b, h], k[b, h // g], v[b, h // g], theta, W, shape, init, source, order)
            out[b, h] = r["out"]
            heads[(b, h)] = r
    return out, heads


def decode_mha(states, q_new, k_new, v_new, theta, W_d):
    """states: dict (b,h) -> state.  q_new [B,H,d], k_new,v_new [B,H_kv,d]."""
    B, H, d = q_new.shape
    g = H // k_new.shape[1]
    out = np.zeros((B, H, d), F64)
    infos = {}
    for b in range(B):
        for h in range(H):
            o, st, info = decode_head(states[(b, h)], q_new[b, h], k_new[b, h // g], v_new[b, h // g],
                                      theta, W_d)
            out[b, h] = o
            states[(b, h)] = st
            infos[(b, h)] = info
    return out, infos
