"""Host-side MSDP schedule (Section 3.4 of the SPTS paper): per-layer active budgets
M^l = min(|T^l|, M_fixed) and the candidate count each stage end prunes to (Eq. 16)."""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple


def _msdp_plan(n_layers: int, n_prompt: int, skip_from: int, stages) -> List[Tuple[int, int, int]]:
    """spts_msdp_plan (the budget rule lives in the library, on the host side of the C boundary):
    stages = [(last_layer, m_attn_fixed, m_ffn_fixed, n_next)]."""
    import ctypes as C
    from . import binding
    lib = binding.load_library()
    st = (binding.MsdpStageC * len(stages))(*[binding.MsdpStageC(*[int(v) for v in t]) for t in stages])
    out = (binding.LayerPlanC * n_layers)()
    code = lib.spts_msdp_plan(n_layers, n_prompt, skip_from, st, len(stages), out, None, None)
    if code != 0:
        raise binding.SptsError(code, "spts_msdp_plan")
    return [(int(p.m_attn), int(p.m_ffn), int(p.prune_to)) for p in out]


def stage_plan(n_layers: int, n_prompt: int, stage_first_layer: Sequence[int], stage_tokens: Sequence[int],
               m_attn_fixed, m_ffn_fixed, skip_from: int = 0) -> List[Tuple[int, int, int]]:
    """Returns [(m_attn, m_ffn, prune_to)] per layer; prune_to == 0 when the layer does not end a stage.

    stage_tokens[s] is the candidate count N_s of stage s (N_0 is the prompt length); the budgets are a single value
    or one per stage.  Layers before `skip_from` run densely."""
    ns = len(stage_first_layer)
    ma = list(m_attn_fixed) if hasattr(m_attn_fixed, "__len__") else [m_attn_fixed] * ns
    mf = list(m_ffn_fixed) if hasattr(m_ffn_fixed, "__len__") else [m_ffn_fixed] * ns
    stages = [(stage_first_layer[s + 1] - 1 if s + 1 < ns else n_layers - 1, ma[s], mf[s],
               stage_tokens[s + 1] if s + 1 < ns else 0) for s in range(ns)]
    return _msdp_plan(n_layers, min(n_prompt, stage_tokens[0]), skip_from, stages)


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


PAPER_SCHEDULES = {
    # model: (layers, first skip layer, stage-end layers, active budgets in Ki tokens, Ki tokens pruned below the budget)
    "llama": (32, 10, (13, 18, 23, 28), (9, 7, 4, 2), 1),
    "qwen": (28, 9, (12, 16, 20, 24), (13, 10, 7, 4), 2),
    "openpangu": (26, 11, (13, 16, 19, 22), (13, 10, 7, 4), 2),
}


def paper_plan(model: str, n_prompt: int, ltp: bool = True, msdp: bool = True):
    """The schedules of the paper's implementation details (Section 4.1), 0-indexed layers: dense layers before the
    first skip layer, then four stages ending at the given layers with fixed active budgets; each stage end prunes
    the candidates to its budget minus the stated number of Ki tokens; the layers after the last boundary keep the
    last budget (the reading that reproduces the KV-cache sizes of Table 3 for LLaMA).
    ltp=False leaves the FFN dense (the "PAP only" row of the paper's component ablation, Table 2);
    msdp=False keeps every token a candidate in every layer (budgets unchanged, no pruning)."""
    n_layers, skip_from, ends, budgets_ki, prune_ki = PAPER_SCHEDULES[model]
    return scaled_paper_plan(n_layers, n_prompt, skip_from, ends, [b * 1024 for b in budgets_ki], prune_ki * 1024,
                             ltp=ltp, msdp=msdp)


def scaled_paper_plan(n_layers: int, n_prompt: int, skip_from: int, ends: Sequence[int], budgets: Sequence[int],
                      prune_below: int, ltp: bool = True, msdp: bool = True):
    """A schedule of the paper's form with every number given in tokens: dense layers before `skip_from`, stage s
    ends after layer ends[s] with active budget budgets[s] and prunes the candidates to budgets[s] - prune_below;
    the layers after the last boundary keep the last budget."""
    stages = [(e, b, b if ltp else 0, b - prune_below if msdp else 0) for e, b in zip(ends, budgets)]
    return _msdp_plan(n_layers, n_prompt, skip_from, stages)


def paper_llama_plan(n_prompt: int, n_layers: int = 32, ltp: bool = True, msdp: bool = True):
    """paper_plan("llama", ...): skipping from layer 10, stage ends after layers 13 / 18 / 23 / 28, budgets
    9 / 7 / 4 / 2 Ki, candidates pruned to budget - 1 Ki."""
    assert n_layers == 32
    return paper_plan("llama", n_prompt, ltp=ltp, msdp=msdp)


def kv_token_layers(plan) -> int:
    """Cached (token, layer) pairs after prefill: every layer caches its m_attn active rows."""
    return sum(p[0] for p in plan)
