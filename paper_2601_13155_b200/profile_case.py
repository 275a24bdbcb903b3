"""Runs a few SPTS layers of a named workload shape once (after one warm-up): a small, self-ending case for profilers.

  python -m paper_2601_13155_b200.profile_case [--tokens 8192] [--dense] [--iters 1]
"""
from __future__ import annotations

import argparse
import math
from dataclasses import replace

import torch

from . import binding, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=8192)
    ap.add_argument("--dense", action="store_true")
    ap.add_argument("--iters", type=int, default=1)
    ap.add_argument("--warmup", type=int, default=1)
    a = ap.parse_args()
    w = synth.workload("cfg2")
    shape = replace(w.shape, n_layers=1)
    dev = "cuda:0"
    n = a.tokens
    t = synth.device_layer_weights(shape, w.seed, 0, dev)
    lw = binding.LayerWeights.__new__(binding.LayerWeights)
    lw.t = t
    lw.c = binding.LayerWeightsC(**{k: t[k].data_ptr() for k in binding.WEIGHT_NAMES})
    X0, _ = synth.device_hidden_states(w, dev, n_tokens=n)
    lib = binding.Spts(shape, max_seq=n)
    cache = binding.KvCache(shape, 1, n)
    pos = torch.arange(n, dtype=torch.int32, device=dev)
    ma, mf = (n, n) if a.dense else (math.ceil(w.keep_attn * n), math.ceil(w.keep_ffn * n))
    for it in range(a.warmup + a.iters):
        X = X0.clone()
        if it == a.warmup:
            lib.profile_begin(-1)
        lib.layer_prefill_skip(lw, X, pos, ma, mf, cache)
    tab = lib.profile_end()
    st = lib.device_status()
    for k, v in sorted(tab.items(), key=lambda kv: -kv[1]["ms"]):
        print(f"{k:12s} {v['ms'] / a.iters:8.3f} ms  {v['flops'] / max(v['ms'], 1e-9) / 1e9:8.1f} TFLOP/s  "
              f"{v['bytes'] / max(v['ms'], 1e-9) / 1e6:8.1f} GB/s")
    print("device status", st)
    if st != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
