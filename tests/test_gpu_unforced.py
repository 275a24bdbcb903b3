"""Unforced end-to-end comparisons with the oracle, and a multi-layer plan that mixes dense layers, skip stages,
a clipped budget and the trailing segment.

"Unforced" = the oracle runs the whole layer (or the whole prefill) from the same input as the library and nothing
of the library's own intermediate state is handed to it: the FFN selection T_f is then compared against the
oracle's own post-attention residual, which the block-wise tests do not do.

* Configuration cfg1 (the tiny fp32 layer) in fp32 verification mode: every output element within 1e-4 of the output RMS, both index sets
  by the 1e-3 band rule (no one-ulp allowance exists in fp32).
* Configuration cfg2 (one 8B-shaped bf16 layer, 8192 tokens): the oracle runs the layer in full; the test reports
  and bounds the T_f symmetric difference (with and without the band) and the one-bf16-ulp disagreements of the
  output, and checks every row on which both sides took the same decisions.
* A mixed plan in the paper's form (Section 4.1: dense shallow layers, stages with fixed budgets, candidates pruned
  below the budget at each stage end, trailing layers on the last candidate set), scaled down: the per-layer chain
  against the oracle block by block, spts_prefill bit-identical to the chain; in fp32 mode additionally the whole
  prefill unforced against the oracle's Algorithm 1."""
import math
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import spts_oracle as O
from paper_2601_13155_b200 import synth, schedule
from parity_utils import (check_index_set, check_layer_blocks, check_output, dev, host, i32, up, zero_down,
                          index_set_report)

pytestmark = pytest.mark.gpu

SMALL_BF16 = replace(synth.LLAMA8B, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn_dim=1024,
                     ltp_dlow=128, ltp_rank=32, n_layers=1, vocab=1024)


def _unforced_layer(shape, W, X, pos, ma, mf, lw, lib):
    from paper_2601_13155_b200 import binding
    N = X.shape[0]
    Xd = up(X, shape.dtype)
    cache = binding.KvCache(shape, 1, ma)
    S = torch.empty(N, dtype=torch.float32, device=dev())
    ia = torch.empty(ma, dtype=torch.int32, device=dev())
    jf = torch.empty(mf, dtype=torch.int32, device=dev())
    lib.layer_prefill_skip(lw, Xd, i32(pos), ma, mf, cache, S_out=S, idx_attn_out=ia, idx_ffn_out=jf)
    assert lib.device_status() == 0
    want = O.layer_prefill_skip(X, pos, W, shape, ma, mf, mode="bf16" if shape.dtype == "bf16" else "exact")
    return Xd, cache, host(S), ia.cpu().numpy().astype(np.int64), jf.cpu().numpy().astype(np.int64), want


def test_config1_fp32_layer_unforced():
    """Configuration cfg1 (the tiny fp32 layer) end to end in fp32 mode: X, S_mha, T_a, T_f and the cache against the oracle's whole layer."""
    from paper_2601_13155_b200 import binding
    w = synth.workload("cfg1")
    shape = w.shape
    N = w.n_tokens
    ma, mf = math.ceil(w.keep_attn * N), math.ceil(w.keep_ffn * N)
    W = synth.layer_weights(shape, w.seed, 0)
    X, _ = synth.hidden_states(shape, N, w.seed, heavy=w.heavy)
    pos = np.arange(N, dtype=np.int32)
    lib = binding.Spts(shape, max_seq=N)
    lw = binding.LayerWeights(W, shape.dtype)
    Xd, cache, S, ia, jf, want = _unforced_layer(shape, W, X, pos, ma, mf, lw, lib)
    assert np.abs(S - want["S_mha"]).max() <= 1e-4 * want["S_mha"].max()
    swaps_a = check_index_set(ia, want["S_mha"], ma)
    swaps_f = check_index_set(jf, want["S_ffn"], mf)
    print(f"[parity] cfg1 fp32 unforced: T_a swaps {swaps_a}, T_f swaps {swaps_f}")
    # every row both sides treated alike must agree to 1e-4 of the output RMS; with no swap that is every row
    same = np.setdiff1d(np.arange(N), np.concatenate([np.setxor1d(ia, want["idx_attn"]), np.setxor1d(jf, want["idx_ffn"])]))
    assert len(same) >= N - 2 * (swaps_a + swaps_f)
    check_output(host(Xd)[same], want["X"][same], "fp32", what="X")
    if swaps_a == 0:
        check_output(host(cache.k[0][:ma]), want["K"], "fp32", what="cache K")
        check_output(host(cache.v[0][:ma]), want["V"], "fp32", what="cache V")
        assert np.array_equal(cache.pos[0][:ma].cpu().numpy(), want["cache_pos"])
    lib.close()


# Bounds asserted for the unforced 8B-shaped layer (the measured values are printed by the test).
CFG2_MAX_TF_DIFF_OUTSIDE_BAND = 8       # tokens of T_f (of 3277) on which GPU and oracle may disagree beyond the band (measured: 0)
CFG2_MAX_FRACTION_BEYOND_TOL = 1e-3     # elements of the layer output beyond 2e-2 of the RMS (measured: 1.5e-4)
CFG2_MAX_ERROR = 5e-2                   # largest error relative to the RMS, single rounding steps of large entries aside (measured: 3.9e-2)


def test_config2_bf16_layer_unforced_reports_selection_and_flip_counts():
    """Configuration cfg2 with the oracle run in full from the same input.  T_a must obey the band rule outright.  For
    T_f the oracle's LTP score is computed on the oracle's own post-attention residual: where the library's bf16
    residual differs from it by one ulp in elements of a row, that row's proxy norm moves a little, so tokens next to
    the k-th score can change sides; their number is reported and bounded (measured: 3 tokens of 3277, all inside the
    1e-3 band), and every such token must lie close to the k-th score (within 2 %)."""
    from paper_2601_13155_b200 import binding
    w = synth.workload("cfg2")
    shape = w.shape
    N = w.n_tokens
    ma, mf = math.ceil(w.keep_attn * N), math.ceil(w.keep_ffn * N)
    W = synth.layer_weights(shape, w.seed, 0)
    X, _ = synth.hidden_states(shape, N, w.seed, heavy=w.heavy)
    pos = np.arange(N, dtype=np.int32)
    lib = binding.Spts(shape, max_seq=N)
    lw = binding.LayerWeights(W, shape.dtype)
    Xd, cache, S, ia, jf, want = _unforced_layer(shape, W, X, pos, ma, mf, lw, lib)
    assert np.abs(S - want["S_mha"]).max() <= 2e-4 * want["S_mha"].max()
    swaps_a = check_index_set(ia, want["S_mha"], ma)
    rep = index_set_report(jf, want["S_ffn"], mf)
    print(f"[parity] cfg2 bf16 unforced: T_a boundary swaps {swaps_a}; T_f symmetric difference {rep['diff']} tokens "
          f"({rep['outside_band']} outside the 1e-3 band, farthest {rep['max_rel_dist']:.2e} from the k-th score)")
    assert rep["outside_band"] <= CFG2_MAX_TF_DIFF_OUTSIDE_BAND
    assert rep["max_rel_dist"] <= 2e-2
    # outputs: rows on which both sides took the same two decisions
    same = np.setdiff1d(np.arange(N), np.concatenate([np.setxor1d(ia, want["idx_attn"]), np.setxor1d(jf, want["idx_ffn"])]))
    # Unforced, the FFN block of the two sides starts from post-attention residuals that differ by one bf16 ulp in
    # several hundred elements of a row (the attention update is small against the row, so a relative difference of
    # 1e-3 in it crosses a rounding boundary in ~10 % of the elements).  Each such difference is far below the
    # tolerance (2^-7 against an RMS of 2), but the random-init FFN amplifies the row's perturbation: its output is
    # ~10 per element for a normalised input of ~1, so a 0.4 % perturbation of the input moves the output by ~0.04,
    # i.e. ~2e-2 of the RMS.  The whole-layer bound therefore holds for all but a small fraction of the elements,
    # and the rest stays within twice the bound; both are measured and bounded here.
    got, ref = host(Xd)[same], want["X"][same]
    rms = np.sqrt(np.mean(ref ** 2))
    err = np.abs(got - ref)
    over = err > 2e-2 * rms
    rows_over = np.unique(np.nonzero(over)[0])
    print(f"[parity] cfg2 bf16 unforced: X worst error {err.max() / rms:.3e} of RMS; {int(over.sum())} of {err.size} elements "
          f"({over.mean():.2e}) beyond 2e-2 of the RMS, in {len(rows_over)} of {len(same)} compared rows, first rows "
          f"{[int(same[r]) for r in rows_over[:12]]}")
    assert over.mean() <= CFG2_MAX_FRACTION_BEYOND_TOL
    # beyond the second bound only rounding steps of large entries may remain (the x8 rows hold values up to ~30,
    # where one bf16 step is 0.125 = 6e-2 of the RMS; the residual is rounded twice on the way)
    from parity_utils import bf16_ulp
    step = bf16_ulp(np.maximum(np.maximum(np.abs(got), np.abs(ref)), np.abs(X[same])))
    beyond = (err > CFG2_MAX_ERROR * rms) & (err > 2.002 * step)       # one step per storage rounding (two of them)
    print(f"[parity] cfg2 bf16 unforced: {int((err > CFG2_MAX_ERROR * rms).sum())} elements beyond {CFG2_MAX_ERROR} of the RMS, "
          f"all within two rounding steps of their magnitude: {not beyond.any()}")
    assert not beyond.any(), f"{int(beyond.sum())} elements beyond {CFG2_MAX_ERROR} of the RMS and beyond two rounding steps"
    if swaps_a == 0:
        check_output(host(cache.k[0][:ma]), want["K"], "bf16", what="cache K")
        check_output(host(cache.v[0][:ma]), want["V"], "bf16", what="cache V")
    lib.close()


def _oracle_plan(plan, n_prompt, skip_from):
    cur, out = n_prompt, []
    for l, (ma, mf, prune) in enumerate(plan):
        out.append({"layer": l, "N": cur, "skip": l >= skip_from, "m_attn": ma, "m_ffn": mf, "prune_to": prune or None})
        cur = prune or cur
    return out


@pytest.mark.parametrize("dtype,ref", [("fp32", None), ("bf16", False), ("bf16", True)])
def test_mixed_plan_dense_skip_prune_trailing(dtype, ref):
    """Eight layers in the form of the paper's LLaMA setting, scaled down: layers 0-1 dense, stage ends after layers
    3, 5 and 6 with budgets 320 / 300 / 120, every stage end prunes to its budget - 64, layer 7 trails.  On 512 tokens
    that gives 320 of 512 active, a prune to 256, a budget (300) clipped by the 256 candidates, a prune to 236, 120 of
    236 active, a prune to 56 and a dense trailing layer on 56 -- every transition spts_prefill carries state across
    (dense -> skip, skip -> prune -> clipped, prune -> skip, prune -> trailing)."""
    from paper_2601_13155_b200 import binding
    base = SMALL_BF16 if dtype == "bf16" else synth.TINY
    L, N, skip_from = 8, 512, 2
    shape = replace(base, n_layers=L, vocab=1000)
    plan = schedule.scaled_paper_plan(L, N, skip_from, (3, 5, 6), (320, 300, 120), 64)
    assert plan == [(512, 512, 0), (512, 512, 0), (320, 320, 0), (320, 320, 256), (256, 256, 0), (256, 256, 236),
                    (120, 120, 56), (56, 56, 0)]
    lib = binding.Spts(shape, max_seq=N)
    if ref is not None:
        lib.set_reference_kernels(ref)
    layers = [synth.layer_weights(shape, 2020, l, std=0.03) for l in range(L)]
    hw = synth.head_weights(shape, 2020)
    X, _ = synth.hidden_states(shape, N, 2020, heavy=32)
    lws = [binding.LayerWeights(wl, dtype) for wl in layers]
    lmid = [binding.LayerWeights(zero_down(wl), dtype) for wl in layers]
    model = binding.Model(lws, up(hw["lm_head"], dtype), up(hw["embed"], dtype))
    caps = [p[0] for p in plan]

    # ---- per-layer chain, each layer against the oracle block by block on the library's own layer input
    cache = binding.KvCache(shape, L, caps)
    Xd, pos, orig = up(X, dtype), i32(np.arange(N)), i32(np.arange(N))
    for l, (ma, mf, prune) in enumerate(plan):
        S = check_layer_blocks(lib, shape, layers[l], lws[l], lmid[l], Xd, pos, ma, mf, cache, layer=l)["S"]
        if prune:
            Xn = torch.empty(prune, shape.hidden, dtype=lib.dtype, device=dev())
            pn, on, keep = (torch.empty(prune, dtype=torch.int32, device=dev()) for _ in range(3))
            lib.msdp_compact(Xd, pos, orig, S, prune, Xn, pn, on, keep)
            assert np.array_equal(keep.cpu().numpy(), O.topk_select(host(S).astype(np.float32), prune, True))
            Xd, pos, orig = Xn, pn, on
    assert lib.device_status() == 0

    # ---- one spts_prefill call: bit-identical to the chain (hidden states, survivors, every layer's cache)
    cache2 = binding.KvCache(shape, L, caps)
    X2, Xa = up(X, dtype), torch.empty(N, shape.hidden, dtype=lib.dtype, device=dev())
    p2, o2 = i32(np.arange(N)), i32(np.arange(N))
    pa, oa = torch.empty_like(p2), torch.empty_like(o2)
    tok = torch.zeros(1, dtype=torch.int32, device=dev())
    nf, in_alt = lib.prefill(model, plan, X2, p2, o2, Xa, pa, oa, cache2, token_out=tok)
    assert lib.device_status() == 0
    assert nf == 56 and in_alt                                   # three compactions: the result sits in the alternate buffer
    assert torch.equal(Xa[:nf], Xd) and torch.equal(oa[:nf], orig) and torch.equal(pa[:nf], pos)
    for l in range(L):
        n = cache.length(l)
        assert n == plan[l][0] and cache2.length(l) == n
        assert torch.equal(cache2.k[l][:n], cache.k[l][:n]) and torch.equal(cache2.v[l][:n], cache.v[l][:n])
        assert torch.equal(cache2.pos[l][:n], cache.pos[l][:n])

    # ---- fp32 mode: the whole prefill unforced against the oracle's Algorithm 1 (no rounding carve-out applies)
    if dtype == "fp32":
        want = O.model_prefill(X, layers, shape, _oracle_plan(plan, N, skip_from), mode="exact")
        assert np.array_equal(oa[:nf].cpu().numpy(), want["orig"]), "survivor sets differ"
        check_output(host(Xa[:nf]), want["X"], "fp32", scale=float(L), what="final X after 8 layers")
        for l in range(L):
            assert np.array_equal(cache2.pos[l][:plan[l][0]].cpu().numpy(), want["caches"][l]["pos"]), f"layer {l}: cached tokens"
    lib.close()
