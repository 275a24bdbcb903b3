"""Runs a few SPTS layers of a named workload shape once (after one warm-up): a small, self-ending case for profilers.

  python -m paper_2601_13155_b200.profile_case [--tokens 8192] [--dense] [--iters 1]
  python -m paper_2601_13155_b200.profile_case --decode 6 [--layers 4] [--cached 16384]
  python -m paper_2601_13155_b200.profile_case --proxy 8192        (proxy-FFN construction on 8192 calibration tokens)
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
    ap.add_argument("--decode", type=int, default=0, help="run this many decode steps instead of a prefill layer")
    ap.add_argument("--layers", type=int, default=4, help="layers of the decode case")
    ap.add_argument("--cached", type=int, default=16384, help="cached tokens per layer of the decode case")
    ap.add_argument("--proxy", type=int, default=0, help="build one layer's proxy FFN from this many calibration tokens")
    a = ap.parse_args()
    if a.decode:
        return decode_case(a)
    if a.proxy:
        return proxy_case(a)
    w = synth.workload("cfg2")
    shape = replace(w.shape, n_layers=1)
    dev = "cuda:0"
    n = a.tokens
    t = synth.device_layer_weights(shape, w.seed, 0, dev)
    lw = binding.LayerWeights.from_tensors(t)
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


def proxy_case(a):
    """spts_proxy_build of one 8B-shaped layer, timed with CUDA events after one warm-up build."""
    w = synth.workload("cfg2")
    shape = replace(w.shape, n_layers=1)
    dev = "cuda:0"
    t = synth.device_layer_weights(shape, w.seed, 0, dev)
    lw = binding.LayerWeights.from_tensors(t)
    Xc, _ = synth.device_hidden_states(w, dev, n_tokens=a.proxy)
    lib = binding.Spts(shape, max_seq=1024)
    lib.proxy_build(lw, Xc, rho=0.2)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = lib.launch_count()
    e0.record()
    lib.proxy_build(lw, Xc, rho=0.2)
    e1.record()
    torch.cuda.synchronize()
    st = lib.device_status()
    print(f"proxy build: {e0.elapsed_time(e1):.1f} ms, {lib.launch_count() - l0} launches, {a.proxy} calibration tokens, "
          f"(D_low, r) = ({shape.ltp_dlow}, {shape.ltp_rank})")
    print("device status", st)
    if st != 0:
        raise SystemExit(1)


def decode_case(a):
    """A few decode steps of an `a.layers`-layer 8B-shaped model against caches of `a.cached` random rows."""
    shape = replace(synth.LLAMA8B, n_layers=a.layers)
    dev = "cuda:0"
    layers = []
    for l in range(a.layers):
        t = synth.device_layer_weights(shape, 7, l, dev)
        lw = binding.LayerWeights.from_tensors(t)
        layers.append(lw)
    hw = synth.device_head_weights(shape, 7, dev)
    model = binding.Model(layers, hw["lm_head"], hw["embed"])
    lib = binding.Spts(shape, max_seq=1024)
    cache = binding.KvCache(shape, a.layers, a.cached + a.decode + 1)
    for l in range(a.layers):
        cache.k[l].normal_()
        cache.v[l].normal_()
        cache.c[l].len = a.cached
    tok = torch.zeros(1, dtype=torch.int32, device=dev)
    lib.decode_step(model, cache, a.cached, token_in=3, token_out=tok)
    lib.profile_begin(14)
    for i in range(1, a.decode):
        lib.decode_step(model, cache, a.cached + i, token_in=5 + i, token_out=tok)
    tab = lib.profile_end()
    st = lib.device_status()
    for k, v in tab.items():
        print(f"{k:12s} {v['ms'] / max(1, v['calls']):8.3f} ms per step  {v['bytes'] / max(v['ms'], 1e-9) / 1e6:8.1f} GB/s")
    print("device status", st)
    if st != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
