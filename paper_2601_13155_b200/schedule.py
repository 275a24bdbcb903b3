"""Host-side MSDP schedule (Section 3.4 of the SPTS paper): per-layer active budgets
M^l = min(|T^l|, M_fixed) and the candidate count each stage end prunes to (Eq. 16)."""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple


def stage_plan(n_layers: int, n_prompt: int, stage_first_layer: Sequence[int], stage_tokens: Sequence[int],
               m_attn_fixed, m_ffn_fixed, skip_from: int = 0) -> List[Tuple[int, int, int]]:
    """Returns [(m_attn, m_ffn, prune_to)] per layer; prune_to == 0 when the layer does not end a stage.

    stage_tokens[s] is the candidate count N_s of stage s; the budgets are a single value or one per stage.
    Layers before `skip_from` run densely."""
    ns = len(stage_first_layer)
    ma = list(m_attn_fixed) if hasattr(m_attn_fixed, "__len__") else [m_attn_fixed] * ns
    mf = list(m_ffn_fixed) if hasattr(m_ffn_fixed, "__len__") else [m_ffn_fixed] * ns
    cur = n_prompt
    out = []
    for l in range(n_layers):
        s = max(i for i in range(ns) if stage_first_layer[i] <= l)
        if l == stage_first_layer[s]:
            cur = min(cur, stage_tokens[s])
        ends = s + 1 < ns and l + 1 == stage_first_layer[s + 1]
        nxt = min(cur, stage_tokens[s + 1]) if ends else 0
        if l >= skip_from:
            out.append((min(cur, ma[s]), min(cur, mf[s]), nxt))
        else:
            out.append((cur, cur, nxt))
        if ends:
            cur = nxt
    return out


def workload_plan(w, keep_attn=None, keep_ffn=None, dense: bool = False):
    """Plan for a synth.Workload: budgets are ceil(keep * prompt length), clipped per stage."""
    n = w.n_tokens
    if dense:
        return [(n, n, 0)] * w.shape.n_layers
    ka = w.keep_attn if keep_attn is None else keep_attn
    kf = w.keep_ffn if keep_ffn is None else keep_ffn
    return stage_plan(w.shape.n_layers, n, w.stage_first_layer, w.stage_tokens, math.ceil(ka * n), math.ceil(kf * n))


def cache_capacities(plan, extra: int = 0):
    return [p[0] + extra for p in plan]


def paper_llama_plan(n_prompt: int, n_layers: int = 32, ltp: bool = True, msdp: bool = True):
    """The paper's LLaMA-3.1-8B setting (Section 4.1): layers 0-9 dense, skipping from layer 10, stage ends after
    layers 13 / 18 / 23 / 28 with active budgets of 9 / 7 / 4 / 2 Ki tokens, each stage end pruning the candidates
    to its budget minus 1 Ki; the layers after the last boundary keep the last budget (0-indexed layers; the
    reading that reproduces the KV-cache sizes of Table 3).
    ltp=False leaves the FFN dense (the "PAP only" row of the paper's component ablation, Table 2);
    msdp=False keeps every token a candidate in every layer (budgets unchanged, no pruning)."""
    ki = 1024
    budgets = (9 * ki, 7 * ki, 4 * ki, 2 * ki)
    ends = (13, 18, 23, 28)
    cur = n_prompt
    out = []
    for l in range(n_layers):
        if l < 10:
            out.append((cur, cur, 0))
            continue
        s = next((i for i, e in enumerate(ends) if l <= e), len(ends) - 1)
        m = min(cur, budgets[s])
        nxt = 0
        if msdp and l in ends:
            nxt = min(cur, budgets[ends.index(l)] - ki)
        out.append((m, m if ltp else cur, nxt if nxt < cur else 0))
        if nxt and nxt < cur:
            cur = nxt
    return out


def kv_token_layers(plan) -> int:
    """Cached (token, layer) pairs after prefill: every layer caches its m_attn active rows."""
    return sum(p[0] for p in plan)
