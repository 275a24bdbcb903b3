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
