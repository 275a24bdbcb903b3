"""Seeded synthetic inputs for the SPTS prefill path.

This module only draws random numbers and lays them out; it holds none of the
method's arithmetic.  Both the CUDA path and the CPU oracle are fed from here so
that they see the same values.  In bf16 configurations every array is rounded
to bf16 once (round-to-nearest-even) and returned as float32 holding exactly
representable bf16 values; `f32_to_bf16_bits` gives the raw 16-bit patterns for
upload.

Workload recipe (shapes follow LLaMA-3.1-8B; the long prompts stand in for the
LongBench prompts used in the paper's efficiency section, which are not
available offline):
  * weights ~ N(0, 0.02), stored [out_features, in_features] row-major;
  * hidden states ~ N(0, 1); a fraction of rows ("heavy" tokens) scaled by 8,
    placed uniformly at random or in 64-token clusters;
  * positions 0..N-1.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, asdict, replace
from typing import Dict, List, Optional

import numpy as np


@dataclass(frozen=True)
class ModelShape:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_dim: int
    ltp_dlow: int
    ltp_rank: int
    n_layers: int = 1
    vocab: int = 0
    rms_eps: float = 1e-5
    rope_theta: float = 500000.0
    dtype: str = "bf16"  # "bf16" or "fp32"

    def asdict(self):
        return asdict(self)


TINY = ModelShape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn_dim=688,
                  ltp_dlow=128, ltp_rank=16, n_layers=1, vocab=512, dtype="fp32")
LLAMA8B = ModelShape(hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn_dim=14336,
                     ltp_dlow=512, ltp_rank=128, n_layers=32, vocab=128256, dtype="bf16")
# the second model family the paper evaluates (Qwen-2.5-7B): 28 query / 4 KV heads (an odd GQA group of 7),
# dimensions from the public model card, (D_low, r) from the paper's implementation details
QWEN7B = ModelShape(hidden=3584, n_q_heads=28, n_kv_heads=4, head_dim=128, ffn_dim=18944,
                    ltp_dlow=1024, ltp_rank=256, n_layers=28, vocab=152064, rms_eps=1e-6,
                    rope_theta=1000000.0, dtype="bf16")


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> uint16 bf16 patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def quantize(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round to the storage type of the configuration; result is float32."""
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(a))
    return np.ascontiguousarray(a, dtype=np.float32)


LAYER_WEIGHT_SHAPES = {
    # name: (out_features, in_features) as functions of the shape
    "wq": lambda s: (s.n_q_heads * s.head_dim, s.hidden),
    "wk": lambda s: (s.n_kv_heads * s.head_dim, s.hidden),
    "wv": lambda s: (s.n_kv_heads * s.head_dim, s.hidden),
    "wo": lambda s: (s.hidden, s.n_q_heads * s.head_dim),
    "w_gate": lambda s: (s.ffn_dim, s.hidden),
    "w_up": lambda s: (s.ffn_dim, s.hidden),
    "w_down": lambda s: (s.hidden, s.ffn_dim),
    # low-rank proxy: x -> r -> dlow (gate, up), dlow -> r -> hidden (down)
    "ug": lambda s: (s.ltp_rank, s.hidden),
    "vg": lambda s: (s.ltp_dlow, s.ltp_rank),
    "uu": lambda s: (s.ltp_rank, s.hidden),
    "vu": lambda s: (s.ltp_dlow, s.ltp_rank),
    "vd": lambda s: (s.ltp_rank, s.ltp_dlow),
    "ud": lambda s: (s.hidden, s.ltp_rank),
}


def layer_weights(shape: ModelShape, seed: int, layer: int = 0, std: float = 0.02,
                  names: Optional[List[str]] = None) -> Dict[str, np.ndarray]:
    """One decoder layer's weights, each [out, in] float32 (bf16-exact if dtype is bf16)."""
    rng = np.random.default_rng(seed * 100 + layer)
    out = {}
    for name, fn in LAYER_WEIGHT_SHAPES.items():
        shp = fn(shape)
        w = rng.standard_normal(shp, dtype=np.float32)
        if names is not None and name not in names:
            continue
        w *= np.float32(std)
        out[name] = quantize(w, shape.dtype)
    return out


def head_weights(shape: ModelShape, seed: int, std: float = 0.02) -> Dict[str, np.ndarray]:
    """LM head [vocab, hidden] and a separate embedding table [vocab, hidden]."""
    rng = np.random.default_rng(seed * 100 + 99)
    lm = rng.standard_normal((shape.vocab, shape.hidden), dtype=np.float32) * np.float32(std)
    emb = rng.standard_normal((shape.vocab, shape.hidden), dtype=np.float32)
    return {"lm_head": quantize(lm, shape.dtype), "embed": quantize(emb, shape.dtype)}


def hidden_states(shape: ModelShape, n_tokens: int, seed: int, heavy: int = 0,
                  cluster: int = 1, heavy_scale: float = 8.0):
    """X [N, hidden] ~ N(0,1) with `heavy` rows scaled; returns (X, heavy_rows).

    cluster == 1: heavy rows drawn without replacement.
    cluster  > 1: heavy // cluster non-overlapping runs of `cluster` consecutive rows.
    """
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n_tokens, shape.hidden), dtype=np.float32)
    if heavy > 0:
        if cluster <= 1:
            rows = np.sort(rng.choice(n_tokens, size=heavy, replace=False))
        else:
            n_cl = max(1, heavy // cluster)
            slots = n_tokens // cluster
            starts = np.sort(rng.choice(slots, size=n_cl, replace=False)) * cluster
            rows = (starts[:, None] + np.arange(cluster)[None, :]).reshape(-1)
        X[rows] *= np.float32(heavy_scale)
    else:
        rows = np.zeros((0,), dtype=np.int64)
    return quantize(X, shape.dtype), rows.astype(np.int64)


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    n_tokens: int
    seed: int
    heavy: int
    cluster: int
    # per-stage description; one-layer workloads have a single stage
    stage_first_layer: tuple
    stage_tokens: tuple          # candidate count N_s per stage
    keep_attn: float
    keep_ffn: float


def workload(name: str) -> Workload:
    if name == "cfg1":
        return Workload("cfg1", TINY, 512, 1001, 32, 1, (0,), (512,), 0.5, 0.5)
    if name == "cfg2":
        s = replace(LLAMA8B, n_layers=1)
        return Workload("cfg2", s, 8192, 1002, 82, 1, (0,), (8192,), 0.5, 0.4)
    if name == "cfg3":
        n = 32768
        return Workload("cfg3", LLAMA8B, n, 1003, 328, 1, (0, 8, 16, 24),
                        (n, round(0.75 * n), round(0.5 * n), round(0.35 * n)), 0.5, 0.4)
    if name == "qwen2":        # one Qwen-2.5-7B-shaped layer, sized like config 2
        s = replace(QWEN7B, n_layers=1)
        return Workload("qwen2", s, 8192, 1012, 82, 1, (0,), (8192,), 0.5, 0.4)
    if name == "qwen3":        # the 28-layer Qwen-shaped model on a 32768-token prompt, staged like config 3
        n = 32768
        return Workload("qwen3", QWEN7B, n, 1013, 328, 1, (0, 7, 14, 21),
                        (n, round(0.75 * n), round(0.5 * n), round(0.35 * n)), 0.5, 0.4)
    if name == "cfg4":
        n = 131072
        return Workload("cfg4", LLAMA8B, n, 1004, 640, 64, (0, 8, 16, 24),
                        (n, round(0.75 * n), round(0.5 * n), round(0.35 * n)), 0.5, 0.4)
    raise KeyError(name)


def tiny_multilayer(n_layers: int = 4, n_tokens: int = 384, dtype: str = "fp32") -> Workload:
    """A small multi-stage workload the oracle finishes in seconds."""
    s = replace(TINY, n_layers=n_layers, dtype=dtype)
    firsts = tuple(range(0, n_layers, max(1, n_layers // 2)))[:2]
    toks = (n_tokens, (n_tokens * 3) // 4)[: len(firsts)]
    return Workload("tiny_ml", s, n_tokens, 1010, 24, 1, firsts, toks, 0.5, 0.4)


# ----------------------------------------------------------------------------------------------
# full-size workloads: drawn on the device (seeded torch generator) because 7 G parameters take
# too long through numpy; the CPU oracle receives copies of the same tensors.
# ----------------------------------------------------------------------------------------------
def device_layer_weights(shape: ModelShape, seed: int, layer: int, device="cuda:0", std: float = 0.02):
    """Same recipe as layer_weights (N(0, std), [out, in], rounded to the storage type) as torch tensors."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed * 100 + layer)
    dt = torch.bfloat16 if shape.dtype == "bf16" else torch.float32
    out = {}
    for name, fn in LAYER_WEIGHT_SHAPES.items():
        w = torch.randn(fn(shape), generator=g, device=device, dtype=torch.float32) * std
        out[name] = w.to(dt).contiguous()
    return out


def device_head_weights(shape: ModelShape, seed: int, device="cuda:0", std: float = 0.02):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed * 100 + 99)
    dt = torch.bfloat16 if shape.dtype == "bf16" else torch.float32
    lm = (torch.randn((shape.vocab, shape.hidden), generator=g, device=device, dtype=torch.float32) * std).to(dt)
    emb = torch.randn((shape.vocab, shape.hidden), generator=g, device=device, dtype=torch.float32).to(dt)
    return {"lm_head": lm.contiguous(), "embed": emb.contiguous()}


def device_hidden_states(w: "Workload", device="cuda:0", n_tokens: Optional[int] = None):
    """X [N, hidden] ~ N(0,1) on the device with the workload's heavy rows (x8); returns (X, heavy_rows)."""
    import torch
    n = w.n_tokens if n_tokens is None else n_tokens
    g = torch.Generator(device=device)
    g.manual_seed(w.seed)
    X = torch.randn((n, w.shape.hidden), generator=g, device=device, dtype=torch.float32)
    rng = np.random.default_rng(w.seed)
    heavy = max(1, int(round(w.heavy * n / w.n_tokens))) if w.heavy else 0
    if heavy:
        if w.cluster <= 1:
            rows = np.sort(rng.choice(n, size=heavy, replace=False))
        else:
            n_cl = max(1, heavy // w.cluster)
            starts = np.sort(rng.choice(n // w.cluster, size=n_cl, replace=False)) * w.cluster
            rows = (starts[:, None] + np.arange(w.cluster)[None, :]).reshape(-1)
        X[torch.from_numpy(rows).to(device)] *= 8.0
    else:
        rows = np.zeros((0,), np.int64)
    dt = torch.bfloat16 if w.shape.dtype == "bf16" else torch.float32
    return X.to(dt).contiguous(), rows
