#!/usr/bin/env python
"""Benchmark of the SPTS prefill path on B200.

One step = one whole prefill of the 32-layer LLaMA-3.1-8B-shaped model (random-init weights,
synthetic hidden states with heavy tokens) through Algorithm 1: per layer PAP score, top-k,
reduced attention, LTP score, top-k, reduced FFN; stage-end pruning; first-token head.
The default workload is configuration "cfg3" (32768-token prompt, four MSDP stages); its line also
carries `ctx_128k`, the same measurement on config 4 (131072 tokens, three timed steps), and `generation`, config 5
in short (the cfg3 prompt prefilled at keep 0.5 then 32 greedy decode steps, beside the dense request).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3|cfg4|cfg2|cfg5] [--impl reference]

Prints ONE JSON line (rank 0).  `value` = prompt tokens / second over all replicas with inputs
resident in HBM; `e2e` = the same through host buffers (pinned H2D of the prompt's hidden states,
D2H of the first token) every step; `dense` = the same code with skipping disabled.
`--workload cfg5` instead times whole requests (prefill + greedy decoding against the compressed
caches) over a keep-ratio sweep.  More than one GPU = independent replicas (the path has no
inter-GPU exchange).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np


def captured_traffic(workload, op):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `op` at the workload's first-stage shape, from the
    ncu capture recorded in profiles/traffic.json -- or None when there is no record, or when the kernel's source
    files have changed since the capture (the record carries their SHA-256)."""
    from paper_2601_13155_b200 import ncu_summary
    try:
        return ncu_summary.traffic_for(workload, op)
    except Exception:
        return None


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="spts", choices=["spts", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg2", "cfg3", "cfg4", "cfg5", "paper", "qwen2", "qwen3"])
    ap.add_argument("--no-128k", action="store_true", help="skip the 131072-token measurement added to the cfg3 line")
    ap.add_argument("--decode-steps", type=int, default=256)
    ap.add_argument("--model", default="llama", choices=["llama", "qwen"], help="model family of --workload paper")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (debug)")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--breakdown", action="store_true", help="also print a per-operation table to stderr")
    return ap.parse_args()


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake": 0x80, "sync_boost": 0x10}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.05)

    def start(self):
        if self.nv is not None:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()

    def stop(self):
        self._stop.set()
        if self._t is not None:
            self._t.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------
# CPU oracle leg (bounded sample)
# --------------------------------------------------------------------------------------------
def oracle_sample(w):
    """The oracle as it stands on configuration cfg2 in full: one SPTS layer of the 8B shape on an 8192-token prompt
    (attention keep 0.5, FFN keep 0.4), on the host cores.  `w` only supplies the depth the figure is scaled to.
    Returns (tokens/s scaled to that depth, cores, description, measured seconds)."""
    from oracle import spts_oracle as O
    from paper_2601_13155_b200 import synth
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    w2 = synth.workload("qwen2" if w.shape.hidden == synth.QWEN7B.hidden else "cfg2")
    shape, n = w2.shape, w2.n_tokens
    W = synth.layer_weights(shape, w2.seed, 0)
    X, _ = synth.hidden_states(shape, n, w2.seed, heavy=w2.heavy)
    ma, mf = math.ceil(w2.keep_attn * n), math.ceil(w2.keep_ffn * n)
    t = time.perf_counter()
    O.layer_prefill_skip(X, np.arange(n), W, shape, ma, mf, mode="bf16" if shape.dtype == "bf16" else "exact")
    dt = time.perf_counter() - t
    layers = w.shape.n_layers
    tps = n / (dt * layers)
    desc = (f"measured: config {w2.name} in full -- one SPTS layer of the {shape.hidden}-wide model on its {n}-token prompt "
            f"(keep {w2.keep_attn}/{w2.keep_ffn}), fp64 numpy oracle, {dt:.2f} s on {cores} threads.  Extrapolation: "
            f"tokens/s = {n} / ({dt:.2f} s x {layers} layers); the attention term grows with the square of the prompt "
            f"length, so at 32768 / 131072 tokens the oracle would be slower than this figure")
    return tps, cores, desc, dt


def run_reference(args):
    """--impl reference: the oracle as it stands, timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2601_13155_b200 import synth
    w = synth.workload("cfg3" if args.workload in ("cfg5", "paper") else args.workload)
    vals = []
    for i in range(args.warmup + args.steps):
        tps, cores, desc, dt = oracle_sample(w)
        if i >= args.warmup:
            vals.append((tps, dt))
        if i == 0 and dt * (args.warmup + args.steps) > 240:      # keep the run within minutes
            args.warmup, args.steps = 0, max(1, min(args.steps, int(240 / dt)))
            vals.append((tps, dt))
            if len(vals) >= args.steps:
                break
    tps = float(np.mean([v[0] for v in vals]))
    ms = float(np.mean([v[1] for v in vals])) * 1e3
    line = {"impl": "reference", "metric": "prefill_tokens_per_s", "value": tps, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": len(vals), "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload + " (bounded sample)", "sample": desc},
            "cpu_baseline": {"value": tps, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------
# the SPTS arm
# --------------------------------------------------------------------------------------------
def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    from paper_2601_13155_b200 import binding, schedule, synth, build

    from paper_2601_13155_b200.replicas import Replicas
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = f"cuda:{local}"
    torch.cuda.set_device(dev)
    rep = Replicas(backend="nccl", device=torch.device(dev))
    rank, world = rep.rank, rep.world
    if rank == 0 and not os.path.exists(binding.LIB_PATH):
        build.build()
    rep.barrier()

    if args.workload == "cfg5":
        line = generation_line(args, rep, dev)
    elif args.workload == "paper":
        line = paper_protocol_line(args, rep, dev)
    else:
        line = prefill_line(args, rep, dev, args.workload, args.steps, max(args.warmup, 3), 2, True)
        if args.workload == "cfg3" and not args.no_128k and not args.layers:
            # the same measurement at the longest context (cfg4, 131072 tokens), kernels already warm
            torch.cuda.empty_cache()
            sub = prefill_line(args, rep, dev, "cfg4", 3, 1, 0, False)
            if rank == 0:
                line["ctx_128k"] = {k: sub[k] for k in ("value", "unit", "ms_per_step", "ttft_ms", "steps", "warmup", "config",
                                                        "dense", "roofline", "algorithmic_tflop_per_step",
                                                        "achieved_tflops_whole_step", "breakdown_ms", "per_operation",
                                                        "gpu_launches")}
            # whole requests (config 5 in short): the cfg3 prompt prefilled at keep 0.5, then 32 greedy decode steps
            # against the compressed caches, beside the same request with skipping disabled
            torch.cuda.empty_cache()
            gen = generation_line(args, rep, dev, decode_steps=32, keeps=(0.5,))
            if rank == 0:
                line["generation"] = {"config": gen["config"]["workload"], "decode_steps": 32,
                                      "keep_0.5": gen["keep_sweep"]["0.5"], "dense": gen["dense"],
                                      "decode_roofline": gen["roofline"]}
    if rank == 0:
        print(json.dumps(line))
    rep.close()


def generation_line(args, rep, dev, decode_steps=None, keeps=(1.0, 0.7, 0.5, 0.3)):
    """Workload cfg5: a 32768-token prompt is prefilled (Algorithm 1), then `--decode-steps` tokens are decoded
    greedily against the per-layer compressed caches; repeated for keep ratios 1.0 / 0.7 / 0.5 / 0.3 (attention
    and FFN budgets = ceil(keep * prompt), MSDP stages as in config 3) and once with skipping disabled.
    value = generated + prompt tokens per second of the whole request at keep 0.5."""
    import torch
    from paper_2601_13155_b200 import binding, schedule, synth
    rank, world = rep.rank, rep.world
    w = synth.workload("cfg3")
    shape = w.shape
    L, N, T = shape.n_layers, w.n_tokens, (decode_steps or args.decode_steps)
    lib = binding.Spts(shape, max_seq=N, device=dev)
    layers = [lib.prepare_layer(binding.LayerWeights.from_tensors(synth.device_layer_weights(shape, w.seed, l, dev)))
              for l in range(L)]                    # proxy factors repacked once, outside every timed region
    hw = synth.device_head_weights(shape, w.seed, dev)
    model = binding.Model(layers, hw["lm_head"], hw["embed"])
    X0, _ = synth.device_hidden_states(w, dev)
    cache = binding.KvCache(shape, L, N + T, dev)
    X, Xa = torch.empty_like(X0), torch.empty_like(X0)
    ar = torch.arange(N, dtype=torch.int32, device=dev)
    pos, orig, pa, oa = ar.clone(), ar.clone(), ar.clone(), ar.clone()
    tok = torch.zeros(1, dtype=torch.int32, device=dev)
    logits = torch.empty(shape.vocab, dtype=torch.float32, device=dev)

    def request(plan, steps):
        """One request; returns (prefill ms, decode ms, first-step logits, generated tokens, cached token-layers)."""
        cache.reset()
        X.copy_(X0)
        pos.copy_(ar)
        orig.copy_(ar)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        rep.barrier()
        ev[0].record()
        lib.prefill(model, plan, X, pos, orig, Xa, pa, oa, cache, token_out=tok)
        ev[1].record()
        t_in = int(tok.item())                      # greedy decoding reads every token back
        kv = sum(cache.length(l) for l in range(L))
        toks, first = [t_in], None
        for i in range(steps):
            lib.decode_step(model, cache, N + i, token_in=t_in, logits_out=logits if i == 0 else None, token_out=tok)
            if i == 0:
                first = logits.clone()
            t_in = int(tok.item())
            toks.append(t_in)
        ev[2].record()
        rep.barrier()
        return ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2]), first, toks, kv

    def plan_for(keep):
        return schedule.workload_plan(w, keep_attn=keep, keep_ffn=keep)

    request(plan_for(0.5), 8)                        # warm-up
    request(plan_for(0.5), 8)
    request(schedule.workload_plan(w, dense=True), 8)
    lib.profile_begin(14)
    pd, dd, lg_d, tk_d, kv_d = request(schedule.workload_plan(w, dense=True), T)
    prof_d = lib.profile_end()
    sweep = {}
    for keep in keeps:
        lib.profile_begin(14)
        pm, dm, lg, tk, kv = request(plan_for(keep), T)
        prof = lib.profile_end()["decode"]
        dev_l2 = float((lg - lg_d).norm() / lg_d.norm())
        match = float(sum(a == b for a, b in zip(tk, tk_d)) / len(tk))
        sweep[str(keep)] = {"ttft_ms": pm, "decode_ms_per_token": dm / T, "request_ms": pm + dm,
                            "tokens_per_s": (N + T) * world / ((pm + dm) * 1e-3),
                            "decode_tokens_per_s": T * world / (dm * 1e-3),
                            "decode_kernel_gbs": prof["bytes"] / max(prof["ms"], 1e-9) / 1e6,
                            "kv_token_layers": kv, "kv_vs_dense": kv / kv_d,
                            "first_logits_rel_l2_vs_dense": dev_l2, "token_match_vs_dense": match,
                            "speedup_vs_dense": (pd + dd) / (pm + dm)}
    status = lib.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status}")
    peaks = {}
    pk_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk_path):
        peaks = json.load(open(pk_path))
    peak = peaks.get("hbm_gbs", 6650.0)
    dk = prof_d["decode"]
    ach = dk["bytes"] / max(dk["ms"], 1e-9) / 1e6
    mid = sweep["0.5"] if "0.5" in sweep else next(iter(sweep.values()))
    line = None
    if rank == 0:
        line = {"metric": "e2e_generation_tokens_per_s", "value": mid["tokens_per_s"], "unit": "tokens/s", "n_gpus": world,
                "steps": 1, "warmup": 3, "ms_per_step": mid["request_ms"], "ttft_ms": mid["ttft_ms"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"cfg5: {L}-layer LLaMA-3.1-8B shape, prompt {N} prefilled with SPTS (keep 0.5, MSDP "
                                       f"stages of cfg3), then {T} greedy decode steps, vocab {shape.vocab}",
                           "global_batch": world, "seq_len": N, "parallelism": f"replicas x{world}",
                           "l2": "15 GB of weights streamed per decode step"},
                "dense": {"ttft_ms": pd, "decode_ms_per_token": dd / T, "request_ms": pd + dd,
                          "tokens_per_s": (N + T) * world / ((pd + dd) * 1e-3), "kv_token_layers": kv_d},
                "keep_sweep": sweep,
                "roofline": {"bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                             "traffic": decode_traffic(shape, L, kv_d + L * T / 2.0),
                             "traffic_note": "ncu capture of a 4-layer case, scaled by layers and cached rows (profiles/traffic.json)",
                             "kernel": "decode step (all layers, dense arm)", "launches": dk["calls"],
                             "ms_per_launch": dk["ms"] / dk["calls"],
                             "peak_source": "measured (copy)" if peaks else "fallback"},
                "gpu_launches": int(lib.launch_count())}
    lib.close()
    return line


def decode_traffic(shape, n_layers, cached_rows_all_layers):
    """DRAM bytes of one decode step scaled from the capture of a 4-layer case (profiles/traffic.json, op "decode"):
    the weight-streaming kernels move a fixed number of bytes per layer, the attention kernel a fixed number per
    cached row; both grow in proportion to what a launch processes."""
    from paper_2601_13155_b200 import synth
    rec = captured_traffic("cfg5", "decode")
    if rec is None or shape != synth.LLAMA8B:
        return None
    return n_layers * rec["weight_bytes_per_layer"] + rec["kv_bytes_per_row"] * cached_rows_all_layers


def paper_protocol_line(args, rep, dev):
    """The paper's efficiency protocol on this code: LLaMA schedule of Section 4.1 (dense layers 0-9, stage ends after
    13 / 18 / 23 / 28, budgets 9 / 7 / 4 / 2 Ki), prompt lengths 8K-32K, TTFT of dense, PAP only, PAP + LTP and full SPTS
    (the rows of its component ablation, Table 2).  value = prompt tokens / s of full SPTS at 32K."""
    import torch
    from paper_2601_13155_b200 import binding, schedule, synth
    rank, world = rep.rank, rep.world
    w = synth.workload("cfg3" if args.model == "llama" else "qwen3")
    shape = w.shape
    L, Nmax = shape.n_layers, w.n_tokens
    lib = binding.Spts(shape, max_seq=Nmax, device=dev)
    layers = [lib.prepare_layer(binding.LayerWeights.from_tensors(synth.device_layer_weights(shape, w.seed, l, dev)))
              for l in range(L)]
    hw = synth.device_head_weights(shape, w.seed, dev)
    model = binding.Model(layers, hw["lm_head"], hw["embed"])
    X0, _ = synth.device_hidden_states(w, dev)
    cache = binding.KvCache(shape, L, Nmax, dev)
    X, Xa = torch.empty_like(X0), torch.empty_like(X0)
    ar = torch.arange(Nmax, dtype=torch.int32, device=dev)
    pos, orig, pa, oa = ar.clone(), ar.clone(), ar.clone(), ar.clone()
    tok = torch.zeros(1, dtype=torch.int32, device=dev)

    def ttft(plan, n, steps):
        def one():
            X[:n].copy_(X0[:n])
            pos[:n].copy_(ar[:n])
            orig[:n].copy_(ar[:n])
            lib.prefill(model, plan, X, pos, orig, Xa, pa, oa, cache, token_out=tok, n_tokens=n)
        one()
        rep.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            one()
        e1.record()
        rep.barrier()
        return rep.max_over_ranks(e0.elapsed_time(e1)) / steps

    table = {}
    for n in (8192, 16384, 24576, 32768):
        plans = {"dense": [(n, n, 0)] * L,
                 "pap": schedule.paper_plan(args.model, n, ltp=False, msdp=False),
                 "pap_ltp": schedule.paper_plan(args.model, n, msdp=False),
                 "spts": schedule.paper_plan(args.model, n)}
        ms = {k: ttft(p, n, max(1, args.steps)) for k, p in plans.items()}
        kv = schedule.kv_token_layers(plans["spts"])
        table[str(n)] = {"ttft_ms": ms, "speedup_vs_dense": {k: ms["dense"] / v for k, v in ms.items() if k != "dense"},
                         "kv_saving_pct": 100.0 * (1 - kv / (L * n))}
    if lib.device_status() != 0:
        raise RuntimeError("device status")
    line = None
    if rank == 0:
        full = table["32768"]
        line = {"metric": "prefill_tokens_per_s", "value": 32768 * world / (full["ttft_ms"]["spts"] * 1e-3), "unit": "tokens/s",
                "n_gpus": world, "steps": max(1, args.steps), "warmup": 1, "ms_per_step": full["ttft_ms"]["spts"],
                "ttft_ms": full["ttft_ms"]["spts"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"paper protocol: {L}-layer {'LLaMA-3.1-8B' if args.model == 'llama' else 'Qwen-2.5-7B'} shape, "
                                       f"the paper's schedule for it {schedule.PAPER_SCHEDULES[args.model]} (layers, first skip "
                                       "layer, stage ends, budgets Ki, Ki pruned below the budget), prompts 8K-32K",
                           "global_batch": world, "seq_len": 32768, "parallelism": f"replicas x{world}",
                           "l2": "inputs larger than L2 (14 GB of weights streamed per step)"},
                "lengths": table,
                "paper_context": ({"ttft_speedup_a800": {"pap": [1.08, 1.24, 1.35, 1.44], "pap_ltp": [1.26, 1.70, 1.98, 2.15],
                                                          "spts": [1.35, 1.91, 2.26, 2.46]},
                                   "kv_saving_pct": [29.7, 48.4, 55.2, 58.6],
                                   "note": "Table 2 / Table 3 of the paper: one A800 80 GB, trained LLaMA-3.1-8B-Instruct, LongBench "
                                           "prompts, HF Transformers + FlashAttention-2; context only"} if args.model == "llama" else
                                  {"note": "the paper gives no per-length TTFT table for Qwen-2.5-7B (average ratio 1.36x at its "
                                           "accuracy operating point, Table 1, A800); context only"}),
                "gpu_launches": int(lib.launch_count())}
    lib.close()
    return line


def per_operation(table, tensor_ops, peaks, wname=None):
    """Every operation of one instrumented prefill against the roofline that bounds it: algorithmic FLOPs (tensor-core
    operations) or bytes (the rest) over the CUDA-event time summed over the layers, as a fraction of the measured peak
    (sustained cuBLAS bf16 TFLOP/s, copy GB/s)."""
    out = {}
    tf_peak = peaks.get("bf16_tflops_sustained", 1400.0)
    bw_peak = peaks.get("hbm_gbs", 6650.0)
    for k, v in sorted(table.items(), key=lambda kv: -kv[1]["ms"]):
        sec = max(v["ms"], 1e-9) * 1e-3
        if k in tensor_ops:
            ach = v["flops"] / sec / 1e12
            out[k] = {"ms": round(v["ms"], 3), "calls": v["calls"], "bound": "tensor", "achieved_tflops": round(ach, 1),
                      "frac_of_measured_peak": round(ach / tf_peak, 3)}
        else:
            ach = v["bytes"] / sec / 1e9
            out[k] = {"ms": round(v["ms"], 3), "calls": v["calls"], "bound": "hbm", "achieved_gbs": round(ach, 1),
                      "frac_of_measured_peak": round(ach / bw_peak, 3)}
        rec = captured_traffic(wname, k)         # DRAM bytes of one launch at the first-stage shape (ncu capture)
        if rec is not None:
            out[k]["dram_traffic_stage0_launch"] = rec["dram_bytes_per_launch"]
    return out


def prefill_line(args, rep, dev, wname, steps, warmup, dense_warmup, with_cpu):
    """Times `steps` whole prefills of workload `wname` (after `warmup`), the same through host buffers, and the
    dense arm; returns the JSON line as a dict (rank 0) or None."""
    import torch
    from paper_2601_13155_b200 import binding, schedule, synth
    rank, world = rep.rank, rep.world
    local = int(os.environ.get("LOCAL_RANK", "0"))
    w = synth.workload(wname)
    shape = w.shape
    if args.layers:
        from dataclasses import replace
        shape = replace(shape, n_layers=args.layers)
        w = replace(w, shape=shape, stage_first_layer=tuple(f for f in w.stage_first_layer if f < args.layers),
                    stage_tokens=w.stage_tokens[:len([f for f in w.stage_first_layer if f < args.layers])])
    L, N = shape.n_layers, w.n_tokens
    plan = schedule.workload_plan(w)
    plan_dense = schedule.workload_plan(w, dense=True)

    # weights and inputs (seeded, drawn on the device)
    lib = binding.Spts(shape, max_seq=N, device=dev)
    layers = [lib.prepare_layer(binding.LayerWeights.from_tensors(synth.device_layer_weights(shape, w.seed, l, dev)))
              for l in range(L)]                    # proxy factors repacked once, outside every timed region
    hw = synth.device_head_weights(shape, w.seed, dev)
    model = binding.Model(layers, hw["lm_head"], hw["embed"])
    X0, _ = synth.device_hidden_states(w, dev)
    X0_host = torch.empty(X0.shape, dtype=X0.dtype, pin_memory=True)
    X0_host.copy_(X0)
    cache = binding.KvCache(shape, L, [N] * L if not args.no_dense else schedule.cache_capacities(plan), dev)
    X = torch.empty_like(X0)
    Xa = torch.empty_like(X0)
    ar = torch.arange(N, dtype=torch.int32, device=dev)
    pos, orig, pa, oa = ar.clone(), ar.clone(), ar.clone(), ar.clone()
    tok = torch.zeros(1, dtype=torch.int32, device=dev)
    tok_host = torch.zeros(1, dtype=torch.int32, pin_memory=True)

    def step(pl, from_host=False):
        if from_host:
            X.copy_(X0_host, non_blocking=True)
        else:
            X.copy_(X0)
        pos.copy_(ar)
        orig.copy_(ar)
        lib.prefill(model, pl, X, pos, orig, Xa, pa, oa, cache, token_out=tok)
        if from_host:
            tok_host.copy_(tok, non_blocking=True)

    barrier = rep.barrier

    def timed(pl, steps, from_host=False, profile_op=0):
        barrier()
        if profile_op:
            lib.profile_begin(profile_op)
        l0 = lib.launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step(pl, from_host)
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        prof = lib.profile_end() if profile_op else {}
        return rep.max_over_ranks(ms), lib.launch_count() - l0, prof

    for _ in range(warmup):
        step(plan)
    status = lib.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after warm-up")

    # which operation dominates?  one untimed, fully instrumented pass
    lib.profile_begin(-1)
    step(plan)
    table = lib.profile_end()
    dom = max(table.items(), key=lambda kv: kv[1]["ms"])[0]
    dom_id = {v: k for k, v in binding.OP_NAMES.items()}[dom]

    clocks = ClockSampler(local)
    clocks.start()
    ms, launches, prof = timed(plan, steps, profile_op=dom_id)
    clk = clocks.stop()
    ms_step = ms / steps
    value = N * world / (ms_step * 1e-3)

    ms_e2e, _, _ = timed(plan, steps, from_host=True)
    e2e = N * world / (ms_e2e / steps * 1e-3)
    # the host-to-device copy on its own (the same pinned buffer, the same stream), to show its share of an e2e step
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(3):
        X.copy_(X0_host, non_blocking=True)
    c1.record()
    torch.cuda.synchronize()
    h2d_ms = c0.elapsed_time(c1) / 3

    dense = None
    if not args.no_dense:
        for _ in range(dense_warmup):
            step(plan_dense)
        ms_d, _, _ = timed(plan_dense, max(1, steps))
        ms_d /= max(1, steps)
        dense = {"value": N * world / (ms_d * 1e-3), "unit": "tokens/s", "ms_per_step": ms_d,
                 "ttft_ms": ms_d, "speedup_spts_vs_dense": ms_d / ms_step}
    status = lib.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status}")

    # roofline of the dominant kernel, from the events recorded inside the timed region
    peaks = {}
    pk_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk_path):
        peaks = json.load(open(pk_path))
    d = prof[dom]
    tensor_ops = {"kproj_pap", "qv_proj", "attention", "o_proj", "ltp", "gate_up", "down"}
    per_launch_ms = d["ms"] / d["calls"]
    if dom in tensor_ops:
        peak = peaks.get("bf16_tflops_sustained", 1400.0)
        achieved = d["flops"] / d["calls"] / (per_launch_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": None, "kernel": dom, "launches": d["calls"], "ms_per_launch": per_launch_ms,
                "peak_source": "measured (sustained cuBLAS bf16)" if peaks else "fallback"}
    else:
        peak = peaks.get("hbm_gbs", 6650.0)
        achieved = d["bytes"] / d["calls"] / (per_launch_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None, "kernel": dom, "launches": d["calls"], "ms_per_launch": per_launch_ms,
                "peak_source": "measured (copy)" if peaks else "fallback"}

    # DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the stage-0 launch shape, from the ncu
    # capture recorded in profiles/traffic.json; null once the kernel's sources differ from the captured ones
    rec = captured_traffic(wname, dom)
    if rec is not None:
        roof["traffic"] = rec["dram_bytes_per_launch"]
        roof["traffic_note"] = (f"ncu capture of one launch at this workload's first-stage shape ({rec['shape']}), kernel sources "
                                f"unchanged since (sha256 {rec['source_sha256'][:12]}, captured at commit {rec['commit_at_capture']})")
    total_flops = sum(v["flops"] for v in table.values())
    line = None
    if rank == 0:
        line = {
            "metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_step, "ttft_ms": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if shape.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": f"{w.name}: {L}-layer {'Qwen-2.5-7B' if shape.hidden == 3584 else 'LLaMA-3.1-8B'} shape, prompt {N}, MSDP stages at layers "
                                   f"{list(w.stage_first_layer)} with {list(w.stage_tokens)} candidates, keep "
                                   f"{w.keep_attn}/{w.keep_ffn}, LTP (D_low, r) = ({shape.ltp_dlow}, {shape.ltp_rank})",
                       "global_batch": world, "seq_len": N, "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2 (14 GB of weights streamed per step)"},
            "e2e": {"value": e2e, "unit": "tokens/s", "h2d_bytes_per_step": int(X0_host.numel() * X0_host.element_size()),
                    "d2h_bytes_per_step": 4, "ms_per_step": ms_e2e / steps, "h2d_ms_alone": h2d_ms},
            "gpu_launches": int(launches),
            "clocks": clk,
            "roofline": roof,
            "dense": dense,
            "algorithmic_tflop_per_step": total_flops / 1e12,
            "achieved_tflops_whole_step": total_flops / 1e12 / (ms_step * 1e-3),
            "breakdown_ms": {k: round(v["ms"], 3) for k, v in sorted(table.items(), key=lambda kv: -kv[1]["ms"])},
            "per_operation": per_operation(table, tensor_ops, peaks, wname),
        }
        if args.breakdown:
            for k, v in sorted(table.items(), key=lambda kv: -kv[1]["ms"]):
                tf = v["flops"] / max(v["ms"], 1e-9) / 1e9
                gb = v["bytes"] / max(v["ms"], 1e-9) / 1e6
                sys.stderr.write(f"{k:12s} {v['ms']:9.3f} ms  {v['calls']:4d} calls  {tf:8.1f} TFLOP/s  {gb:8.1f} GB/s\n")
        if with_cpu:
            tps_cpu, cores, desc, _ = oracle_sample(w)
            line["cpu_baseline"] = {"value": tps_cpu, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": desc}
    lib.close()
    del lib, cache, model, layers, hw, X, Xa, X0, X0_host
    return line


if __name__ == "__main__":
    main()
