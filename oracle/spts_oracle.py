"""CPU oracle for Self-Predictive Token Skipping (SPTS) -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the paper's token-selective prefill
layer computes (Algorithm 1 with Eq. 2, 4, 5, 6, 12-16), written from the
paper's definitions.  It shares no code with the CUDA path and must never be
imported by it; only tests, the smoke check and the benchmark's CPU-baseline
leg may call it.

Conventions
  * weights are [out_features, in_features]; y = x @ W.T
  * all arithmetic is float64; `rnd` is the identity ("exact" mode) or rounds
    to bf16 at the storage points the bf16 kernels declare ("bf16" mode):
    cached K/V, projected Q, attention output, SwiGLU intermediate, proxy
    intermediates, and the residual stream after each update.
  * Algorithm 1 leaves out normalisation and positional embedding; they are
    placed as in a pre-norm LLaMA block: RMSNorm before the attention block
    (feeds PAP's K, q and the reduced attention), RMSNorm of the updated
    residual before the FFN block (feeds the proxy and the FFN), rotary
    embedding (rotate-half pairing, original token positions) on q, Q and K.
  * index sets are emitted ascending; ties go to the lower index; with
    force_last the last candidate is always a member (it carries the output).

Pinned by tests/test_oracle_pins.py (library routines, closed forms, the
paper's Table 3 and Table 6 values, brute force).  Unpinned: nothing in this
file; accuracy on LongBench and the paper's speed-up ratios are out of reach
offline ("parity unpinned" for those, they are not computed here).
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# rounding points
# ----------------------------------------------------------------------------
def identity(a):
    return a


def round_bf16(a):
    """Round float64 values to the nearest bf16 (ties to even); result float64.

    Works on the fp64 bit pattern directly (keeps 7 explicit mantissa bits), so
    there is no double rounding through float32.  Values are assumed to lie in
    bf16's normal range.
    """
    a = np.ascontiguousarray(a, dtype=F64)
    u = a.view(np.uint64)
    drop = np.uint64(45)
    lsb = (u >> drop) & np.uint64(1)
    u2 = (u + (np.uint64((1 << 44) - 1) + lsb)) & ~np.uint64((1 << 45) - 1)
    return u2.view(F64).reshape(a.shape)


def rounding(mode: str):
    return round_bf16 if mode == "bf16" else identity


# ----------------------------------------------------------------------------
# standard ops the paper omits from Algorithm 1
# ----------------------------------------------------------------------------
def rmsnorm(X, g, eps):
    X = np.asarray(X, F64)
    ms = np.mean(X * X, axis=-1, keepdims=True)
    return X / np.sqrt(ms + eps) * np.asarray(g, F64)


def rope(x, pos, theta):
    """Rotary embedding, rotate-half pairing (i, i + d/2).  x: [n, heads, d]."""
    x = np.asarray(x, F64)
    n, _, d = x.shape
    half = d // 2
    inv_freq = theta ** (-(np.arange(half, dtype=F64) * 2.0) / d)
    ang = np.asarray(pos, F64)[:, None] * inv_freq[None, :]          # [n, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


# ----------------------------------------------------------------------------
# Eq. 4: partial attention probing
# ----------------------------------------------------------------------------
def pap_score(A, pos, wk, wq, shape):
    """K = A Wk (all rows), q = A_N Wq (last row); S_n = mean_h softmax_n(q_h K_h / sqrt d).

    Returns (K [N,Hkv,d] post-RoPE unrounded, q [H,d], S [N]).
    """
    N = A.shape[0]
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    G = H // Hkv
    K = rope((A @ wk.T).reshape(N, Hkv, d), pos, shape.rope_theta)
    q = rope((A[N - 1:N] @ wq.T).reshape(1, H, d), pos[N - 1:N], shape.rope_theta)[0]
    S = np.zeros(N, F64)
    for h in range(H):
        z = K[:, h // G, :] @ q[h] / math.sqrt(d)
        z = z - z.max()
        e = np.exp(z)
        S += e / e.sum()
    return K, q, S / H


def pap_score_window(A, pos, wk, wq, shape, window, rnd=identity):
    """The probe score with a window of query tokens (the query-length ablation of the paper's Appendix C): the
    attention rows of the last `window` candidates, each over its causal range n <= i, averaged over the window and
    the H heads.  window = 1 is Eq. 4.  K and the window's queries are rounded with `rnd` (they are taken as stored).
    Returns (K [N,Hkv,d] after rnd, S [N])."""
    N = A.shape[0]
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    G = H // Hkv
    w = min(window, N)
    K = rnd(rope((A @ wk.T).reshape(N, Hkv, d), pos, shape.rope_theta))
    Q = rnd(rope((A[N - w:] @ wq.T).reshape(w, H, d), pos[N - w:], shape.rope_theta))
    S = np.zeros(N, F64)
    for a in range(w):
        i = N - w + a                          # the query's own index: it sees keys 0..i
        for h in range(H):
            z = K[: i + 1, h // G, :] @ Q[a, h] / math.sqrt(d)
            z = z - z.max()
            e = np.exp(z)
            S[: i + 1] += e / e.sum()
    return K, S / (w * H)


# ----------------------------------------------------------------------------
# Eq. 5 / 15 / 16: TopK
# ----------------------------------------------------------------------------
def topk_select(scores, k, force_last=False):
    """Indices of the k largest scores, ascending.  Order: score descending,
    then index ascending; -0.0 counts as +0.0; NaN ranks below everything.
    With force_last the last index is ranked first."""
    s = np.array(scores, dtype=F64).copy()
    n = s.shape[0]
    assert 1 <= k <= n
    s[np.isnan(s)] = -np.inf
    s = s + 0.0                       # -0.0 -> +0.0
    key = -s
    if force_last:
        key[n - 1] = -np.inf
    order = np.lexsort((np.arange(n), key))   # primary key, then index
    # NaN entries (now -inf scores) tie with genuine -inf; acceptable: both rank last
    return np.sort(order[:k]).astype(np.int64)


# ----------------------------------------------------------------------------
# reduced / dense causal GQA attention
# ----------------------------------------------------------------------------
def causal_gqa_attention(Q, K, V, row_chunk=1024):
    """Q [m,H,d], K,V [m,Hkv,d]; row i attends to rows j <= i.  Returns [m, H*d]."""
    m, H, d = Q.shape
    Hkv = K.shape[1]
    G = H // Hkv
    out = np.zeros((m, H, d), F64)
    for h in range(H):
        Kh = K[:, h // G, :]
        Vh = V[:, h // G, :]
        for r0 in range(0, m, row_chunk):
            r1 = min(m, r0 + row_chunk)
            z = Q[r0:r1, h, :] @ Kh[:r1].T / math.sqrt(d)
            ii = np.arange(r0, r1)[:, None]
            jj = np.arange(r1)[None, :]
            z = np.where(jj <= ii, z, -np.inf)
            z = z - z.max(axis=1, keepdims=True)
            p = np.exp(z)
            p /= p.sum(axis=1, keepdims=True)
            out[r0:r1, h, :] = p @ Vh[:r1]
    return out.reshape(m, H * d)


def causal_gqa_attention_rows(Q_rows, rows, K, V):
    """The rows `rows` of causal_gqa_attention(Q, K, V) without forming the others:
    Q_rows [s,H,d] holds the queries of those rows; row i attends to K[j], V[j] for j <= i
    (compact order, Algorithm 1's F_MHA on the active rows).  Returns [s, H*d]."""
    Q_rows = np.asarray(Q_rows, F64)
    s, H, d = Q_rows.shape
    G = H // K.shape[1]
    out = np.zeros((s, H, d), F64)
    for a, i in enumerate(rows):
        for h in range(H):
            z = K[: i + 1, h // G, :] @ Q_rows[a, h] / math.sqrt(d)
            z = z - z.max()
            e = np.exp(z)
            out[a, h] = (e / e.sum()) @ V[: i + 1, h // G, :]
    return out.reshape(s, H * d)


# ----------------------------------------------------------------------------
# Eq. 6 and Eq. 12-14
# ----------------------------------------------------------------------------
def ffn(B, w_gate, w_up, w_down, rnd=identity):
    hm = rnd(silu(B @ w_gate.T) * (B @ w_up.T))
    return hm @ w_down.T


def ltp_proxy(B, W, rnd=identity):
    """f(B) = (silu(B Ug Vg) * (B Uu Vu)) Vd^T Ud^T, with the factors stored [out,in]."""
    tg = rnd(B @ W["ug"].T)
    tu = rnd(B @ W["uu"].T)
    h = rnd(silu(tg @ W["vg"].T) * (tu @ W["vu"].T))
    td = rnd(h @ W["vd"].T)
    return td @ W["ud"].T


def ltp_score(B, S_mha, W, rnd=identity):
    o = ltp_proxy(B, W, rnd)
    C = np.sqrt(np.sum(o * o, axis=1))
    return C, C * S_mha


# ----------------------------------------------------------------------------
# one layer of Algorithm 1
# ----------------------------------------------------------------------------
def _w64(W):
    return {k: np.asarray(v, F64) for k, v in W.items()}


def layer_prefill_skip(X, pos, W, shape, m_attn, m_ffn, g_attn=None, g_ffn=None,
                       mode="exact", force_last=True, ffn_criterion="ltp"):
    """One decoder layer with token skipping.  m_attn == N / m_ffn == N is the
    dense block (TopK of everything).  Returns a dict with the updated X, the
    scores, both index sets and the layer's KV cache entries.

    ffn_criterion: "ltp" selects the FFN's tokens by Eq. 14 (proxy norm times S_mha);
    "pap" by S_mha alone (Eq. 4), the criterion Table 4 compares the proxy network against."""
    rnd = rounding(mode)
    W = _w64(W)
    X = np.array(X, dtype=F64)
    pos = np.asarray(pos)
    N, D = X.shape
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    g1 = np.ones(D) if g_attn is None else np.asarray(g_attn, F64)
    g2 = np.ones(D) if g_ffn is None else np.asarray(g_ffn, F64)
    m_attn = min(N, m_attn)
    m_ffn = min(N, m_ffn)

    # --- PAP + reduced MHA
    A = rmsnorm(X, g1, shape.rms_eps)
    K, q, S_mha = pap_score(A, pos, W["wk"], W["wq"], shape)
    Ta = topk_select(S_mha, m_attn, force_last)
    Ah = A[Ta]
    Qh = rnd(rope((Ah @ W["wq"].T).reshape(m_attn, H, d), pos[Ta], shape.rope_theta))
    Vh = rnd((Ah @ W["wv"].T).reshape(m_attn, Hkv, d))
    Kh = rnd(K[Ta])
    att = rnd(causal_gqa_attention(Qh, Kh, Vh))
    X[Ta] = rnd(X[Ta] + att @ W["wo"].T)

    # --- LTP + reduced FFN (on the updated residual; S_mha from before the update)
    B = rmsnorm(X, g2, shape.rms_eps)
    if ffn_criterion == "pap":
        C, S_ffn = None, S_mha
    else:
        C, S_ffn = ltp_score(B, S_mha, W, rnd)
    Tf = topk_select(S_ffn, m_ffn, force_last)
    X[Tf] = rnd(X[Tf] + ffn(B[Tf], W["w_gate"], W["w_up"], W["w_down"], rnd))

    return {"X": X, "S_mha": S_mha, "idx_attn": Ta, "C": C, "S_ffn": S_ffn, "idx_ffn": Tf,
            "K": Kh, "V": Vh, "cache_pos": pos[Ta].copy(), "K_all": K, "q": q}


def attention_block_rows(X, pos, W, shape, Ta, K_all, sample, mode="exact"):
    """Eq. 2 for the attention block on a sample of the active rows: returns the updated
    hidden rows X[Ta[sample]] + F_MHA(...) W_O given the active set Ta (ascending) and the
    post-RoPE keys K_all [N,Hkv,d] of every candidate.  V is projected for all active rows
    (every later active row attends to it), Q only for the sampled rows."""
    rnd = rounding(mode)
    W = _w64(W)
    X = np.asarray(X)
    pos = np.asarray(pos)
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    Ta = np.asarray(Ta)
    sample = np.asarray(sample)
    ones = np.ones(X.shape[1])
    Aa = rmsnorm(X[Ta], ones, shape.rms_eps)
    Vh = rnd((Aa @ W["wv"].T).reshape(len(Ta), Hkv, d))
    Kh = rnd(np.asarray(K_all, F64)[Ta])
    Qs = rnd(rope((Aa[sample] @ W["wq"].T).reshape(len(sample), H, d), pos[Ta[sample]], shape.rope_theta))
    att = rnd(causal_gqa_attention_rows(Qs, sample, Kh, Vh))
    return rnd(np.asarray(X[Ta[sample]], F64) + att @ W["wo"].T), Kh, Vh


def ffn_block_rows(X, W, shape, rows, mode="exact"):
    """Eq. 2 + Eq. 6 for the FFN block on the given rows of the (post-attention) residual X."""
    rnd = rounding(mode)
    W = _w64(W)
    xr = np.asarray(X[np.asarray(rows)], F64)
    B = rmsnorm(xr, np.ones(xr.shape[1]), shape.rms_eps)
    return rnd(xr + ffn(B, W["w_gate"], W["w_up"], W["w_down"], rnd))


def layer_dense(X, pos, W, shape, g_attn=None, g_ffn=None, mode="exact"):
    """Standard pre-norm decoder layer: X += MHA(X); X += FFN(X)."""
    rnd = rounding(mode)
    W = _w64(W)
    X = np.array(X, dtype=F64)
    N, D = X.shape
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    g1 = np.ones(D) if g_attn is None else np.asarray(g_attn, F64)
    g2 = np.ones(D) if g_ffn is None else np.asarray(g_ffn, F64)
    A = rmsnorm(X, g1, shape.rms_eps)
    Q = rnd(rope((A @ W["wq"].T).reshape(N, H, d), pos, shape.rope_theta))
    K = rnd(rope((A @ W["wk"].T).reshape(N, Hkv, d), pos, shape.rope_theta))
    V = rnd((A @ W["wv"].T).reshape(N, Hkv, d))
    att = rnd(causal_gqa_attention(Q, K, V))
    X = rnd(X + att @ W["wo"].T)
    B = rmsnorm(X, g2, shape.rms_eps)
    X = rnd(X + ffn(B, W["w_gate"], W["w_up"], W["w_down"], rnd))
    return {"X": X, "K": K, "V": V, "cache_pos": np.asarray(pos).copy()}


# ----------------------------------------------------------------------------
# Eq. 16 / Algorithm 1 stage end
# ----------------------------------------------------------------------------
def msdp_compact(X, pos, orig, S_mha, n_next, force_last=True):
    """Keep the TopK(S_mha, min(N, n_next)) candidates, in token order."""
    N = X.shape[0]
    T = topk_select(S_mha, min(N, n_next), force_last)
    return X[T].copy(), np.asarray(pos)[T].copy(), np.asarray(orig)[T].copy(), T


# ----------------------------------------------------------------------------
# MSDP budgets (host logic)
# ----------------------------------------------------------------------------
def msdp_schedule(n_layers, n_prompt, stage_first_layer, stage_tokens, m_attn_fixed, m_ffn_fixed,
                  skip_from=0):
    """Per-layer plan: candidates N, active counts M^l = min(|T^l|, M_fixed) and the
    size pruned to after the layer (None if the layer is not a stage end).
    `stage_tokens[s]` is N_s; `m_*_fixed` is one budget or one per stage."""
    ns = len(stage_first_layer)
    ma_f = list(m_attn_fixed) if hasattr(m_attn_fixed, "__len__") else [m_attn_fixed] * ns
    mf_f = list(m_ffn_fixed) if hasattr(m_ffn_fixed, "__len__") else [m_ffn_fixed] * ns
    plan = []
    N = n_prompt
    for l in range(n_layers):
        s = max(i for i in range(ns) if stage_first_layer[i] <= l)
        if l == stage_first_layer[s]:
            N = min(N, stage_tokens[s])
        skip = l >= skip_from
        last_of_stage = (s + 1 < ns) and (l + 1 == stage_first_layer[s + 1])
        prune_to = min(N, stage_tokens[s + 1]) if last_of_stage else None
        plan.append({"layer": l, "stage": s, "N": N, "skip": skip,
                     "m_attn": min(N, ma_f[s]) if skip else N,
                     "m_ffn": min(N, mf_f[s]) if skip else N,
                     "prune_to": prune_to})
        if prune_to is not None:
            N = prune_to
    return plan


def paper_llama_schedule(n_prompt):
    """The paper's LLaMA setting (Implementation Details): skipping from layer 10,
    stage boundaries after layers 13/18/23/28, budgets 9/7/4/2 Ki tokens, candidates
    cut to budget - 1 Ki at each stage end; layers are 0-indexed and the layers after
    the last boundary keep the last stage's budget and its pruned candidate set."""
    Ki = 1024
    budgets = [9 * Ki, 7 * Ki, 4 * Ki, 2 * Ki]
    ends = [13, 18, 23, 28]
    plan = []
    N = n_prompt
    for l in range(32):
        if l < 10:
            plan.append({"layer": l, "stage": -1, "N": N, "skip": False, "m_attn": N, "m_ffn": N,
                         "prune_to": None})
            continue
        s = next((i for i, e in enumerate(ends) if l <= e), 4)
        if s < 4:
            m = min(N, budgets[s])
            prune_to = min(N, budgets[s] - Ki) if l == ends[s] else None
        else:
            m = min(N, budgets[3])   # trailing layers keep the last stage's budget
            prune_to = None
        plan.append({"layer": l, "stage": s, "N": N, "skip": True, "m_attn": m, "m_ffn": m,
                     "prune_to": prune_to})
        if prune_to is not None:
            N = prune_to
    return plan


def kv_cache_token_layers(plan):
    """Number of cached (token, layer) pairs after prefill: sum of m_attn over layers."""
    return sum(p["m_attn"] for p in plan)


def proxy_macs_per_projection(D, d_low, r):
    """Multiply-accumulates per token for one low-rank projection x U V
    (or x W' when r is None: no factorisation)."""
    if r is None:
        return D * d_low
    return r * (D + d_low)


# ----------------------------------------------------------------------------
# offline construction of the low-rank proxy FFN (Section 3.3: saliency, channel
# importance, channel selection, rank-r factorisation)
# ----------------------------------------------------------------------------
def proxy_saliency(Xc, W, shape):
    """z(x) = |silu(x W_gate) * (x W_up)| for every calibration token (rows of Xc are the hidden
    states preceding the FFN block; they are normalised like the FFN's input).  [n_cal, Dff]."""
    B = rmsnorm(np.asarray(Xc, F64), np.ones(Xc.shape[1]), shape.rms_eps)
    return np.abs(silu(B @ np.asarray(W["w_gate"], F64).T) * (B @ np.asarray(W["w_up"], F64).T))


def proxy_channel_importance(z, rho):
    """I_j = mean of the top rho-fraction of channel j's saliency values over the calibration set;
    the count is max(1, floor(rho * |G|))."""
    n = z.shape[0]
    k = max(1, int(math.floor(rho * n)))
    top = -np.sort(-np.asarray(z, F64), axis=0)[:k]
    return top.mean(axis=0)


def proxy_select_channels(importance, d_low):
    """C = TopK(I, D_low), ascending channel indices, ties to the lower index."""
    return topk_select(importance, d_low, force_last=False)


def proxy_factor(Wp, r):
    """Rank-r factorisation W' ~ U V of a [D, D_low] matrix by truncated SVD: U [D, r] has orthonormal
    columns, V = diag(sigma_r) V_r^T [r, D_low].  Returns (U, V, all singular values)."""
    Uf, sg, Vt = np.linalg.svd(np.asarray(Wp, F64), full_matrices=False)
    return Uf[:, :r], sg[:r, None] * Vt[:r], sg


def proxy_build(Xc, W, shape, rho=0.2, channels=None):
    """The whole construction for one layer.  Returns the importance vector, the selected channels and the six
    factors in the library's storage layout: ug/uu [r, D] = U^T, vg/vu [D_low, r] = V^T, vd [r, D_low] = V_down,
    ud [D, r] = U_down, plus the singular values of the three reduced matrices."""
    z = proxy_saliency(Xc, W, shape)
    imp = proxy_channel_importance(z, rho)
    C = proxy_select_channels(imp, shape.ltp_dlow) if channels is None else np.asarray(channels)
    r = shape.ltp_rank
    out = {"importance": imp, "channels": C, "sigma": {}}
    # the paper writes the projections as [D, Dff] matrices; w_gate / w_up are stored [Dff, D], w_down [D, Dff]
    for name, Wp in (("g", np.asarray(W["w_gate"], F64)[C].T), ("u", np.asarray(W["w_up"], F64)[C].T),
                     ("d", np.asarray(W["w_down"], F64)[:, C])):
        U, V, sg = proxy_factor(Wp, r)
        out["sigma"][name] = sg
        if name == "d":
            out["vd"], out["ud"] = V, U
        else:
            out["u" + name], out["v" + name] = U.T, V.T
    return out


# ----------------------------------------------------------------------------
# whole prefill (Algorithm 1) and decode
# ----------------------------------------------------------------------------
def model_prefill(X, layers, shape, plan, mode="exact", force_last=True):
    """Algorithm 1 in the prefill phase.  `layers[l]` is the weight dict of layer l.
    Returns final hidden states (pruned), their positions and original indices,
    the per-layer caches and per-layer traces."""
    rnd = rounding(mode)
    X = np.array(X, dtype=F64)
    pos = np.arange(X.shape[0], dtype=np.int64)
    orig = pos.copy()
    caches, trace = [], []
    for p, W in zip(plan, layers):
        N = X.shape[0]
        assert N == p["N"], (N, p)
        if p["skip"]:
            r = layer_prefill_skip(X, pos, W, shape, p["m_attn"], p["m_ffn"], mode=mode,
                                   force_last=force_last)
        else:
            r = layer_dense(X, pos, W, shape, mode=mode)
        X = r["X"]
        caches.append({"K": r["K"], "V": r["V"], "pos": r["cache_pos"]})
        t = {k: r[k] for k in ("S_mha", "idx_attn", "S_ffn", "idx_ffn") if k in r}
        if p["prune_to"] is not None:
            X, pos, orig, T = msdp_compact(X, pos, orig, r["S_mha"], p["prune_to"], force_last)
            t["idx_prune"] = T
        trace.append(t)
    return {"X": X, "pos": pos, "orig": orig, "caches": caches, "trace": trace}


def first_token(x_last, g_final, lm_head, eps):
    """Final RMSNorm of one row, LM head, argmax (lowest index on ties)."""
    a = rmsnorm(np.asarray(x_last, F64)[None, :], g_final, eps)[0]
    logits = np.asarray(lm_head, F64) @ a
    return logits, int(np.argmax(logits))


def decode_layer(x, pos_new, W, shape, cache, mode="exact"):
    """Dense layer for one new token against cache ∪ itself; appends to the cache."""
    rnd = rounding(mode)
    W = _w64(W)
    x = np.asarray(x, F64).copy()
    D = x.shape[0]
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    G = H // Hkv
    ones = np.ones(D)
    a = rmsnorm(x[None, :], ones, shape.rms_eps)
    p1 = np.array([pos_new])
    q = rnd(rope((a @ W["wq"].T).reshape(1, H, d), p1, shape.rope_theta))[0]
    k = rnd(rope((a @ W["wk"].T).reshape(1, Hkv, d), p1, shape.rope_theta))
    v = rnd((a @ W["wv"].T).reshape(1, Hkv, d))
    Kc = np.concatenate([cache["K"], k], axis=0)
    Vc = np.concatenate([cache["V"], v], axis=0)
    cache["K"], cache["V"] = Kc, Vc
    cache["pos"] = np.concatenate([cache["pos"], p1])
    att = np.zeros((H, d), F64)
    for h in range(H):
        z = Kc[:, h // G, :] @ q[h] / math.sqrt(d)
        z = z - z.max()
        e = np.exp(z)
        att[h] = (e / e.sum()) @ Vc[:, h // G, :]
    att = rnd(att.reshape(-1))
    x = rnd(x + W["wo"] @ att)
    b = rmsnorm(x[None, :], ones, shape.rms_eps)
    x = rnd(x + ffn(b, W["w_gate"], W["w_up"], W["w_down"], rnd)[0])
    return x


def decode_step(x_embed, pos_new, layers, shape, caches, g_final, lm_head, mode="exact"):
    """One auto-regressive step (Algorithm 1 outside the prefill phase: no skipping)."""
    x = np.asarray(x_embed, F64)
    for W, c in zip(layers, caches):
        x = decode_layer(x, pos_new, W, shape, c, mode)
    logits, tok = first_token(x, g_final, lm_head, shape.rms_eps)
    return x, logits, tok
