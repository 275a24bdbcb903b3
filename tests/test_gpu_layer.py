"""GPU parity of the probes, the skip layer, the whole prefill and the decode step against the oracle.

Tolerances: bf16 storage -> max-abs error <= 2e-2 of the output RMS; fp32 verification mode -> 1e-4.
Index sets must equal the oracle's except for tokens within 1e-3 (relative) of the k-th score."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import spts_oracle as O
from paper_2601_13155_b200 import synth, schedule
from parity_utils import TOL, check_index_set, check_layer_blocks, check_output, dev, host, i32, rel_rms_err, up, zero_down

pytestmark = pytest.mark.gpu

SMALL_BF16 = replace(synth.LLAMA8B, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn_dim=1024,
                     ltp_dlow=128, ltp_rank=32, n_layers=1, vocab=1024)


# an odd GQA group (3 query heads per KV head): the attention kernel pairs two query tiles of one head; per-head decode attention
ODD_GROUP_BF16 = replace(synth.LLAMA8B, hidden=384, n_q_heads=6, n_kv_heads=2, head_dim=128, ffn_dim=768,
                         ltp_dlow=128, ltp_rank=32, n_layers=1, vocab=1024)


# a GQA group of 16 query heads per KV head: more than the eight probe logits the K-projection epilogue keeps in registers
WIDE_GROUP_BF16 = replace(synth.LLAMA8B, hidden=512, n_q_heads=16, n_kv_heads=1, head_dim=128, ffn_dim=1024,
                          ltp_dlow=128, ltp_rank=32, n_layers=1, vocab=1024)


def _mk(shape, max_seq, reference=None):
    from paper_2601_13155_b200 import binding
    lib = binding.Spts(shape, max_seq=max_seq)
    if reference is not None:
        lib.set_reference_kernels(reference)
    return lib


def _layer_case(shape, n, seed, heavy, std=0.02):
    from paper_2601_13155_b200 import binding
    W = synth.layer_weights(shape, seed, 0, std=std)
    X, _ = synth.hidden_states(shape, n, seed, heavy=heavy)
    return W, X, binding.LayerWeights(W, shape.dtype)


def _modes():
    # (shape, N, m_attn, m_ffn, reference kernels)
    return [
        pytest.param(synth.TINY, 512, 256, 256, None, id="cfg1-fp32"),
        pytest.param(synth.TINY, 389, 100, 57, None, id="tiny-fp32-ragged"),
        pytest.param(replace(synth.TINY, dtype="bf16"), 512, 256, 256, True, id="cfg1-bf16-refkernels"),
        pytest.param(SMALL_BF16, 777, 300, 211, True, id="small8b-bf16-refkernels"),
        pytest.param(SMALL_BF16, 777, 300, 211, False, id="small8b-bf16-tensorcore"),
        pytest.param(SMALL_BF16, 1024, 1024, 1024, False, id="small8b-bf16-tensorcore-dense"),
        pytest.param(SMALL_BF16, 640, 640, 200, False, id="small8b-bf16-tensorcore-attn-dense"),
        pytest.param(ODD_GROUP_BF16, 515, 259, 130, False, id="oddgroup-bf16-tensorcore"),
        pytest.param(WIDE_GROUP_BF16, 333, 150, 101, False, id="group16-bf16-tensorcore"),
    ]


@pytest.mark.parametrize("shape,N,ma,mf,ref", _modes())
def test_probes_match_oracle(shape, N, ma, mf, ref):
    lib = _mk(shape, 2048, ref)
    W, X, Wd = _layer_case(shape, N, 1001, 32, std=0.05)
    pos = (np.arange(N) * 2 + 5).astype(np.int32)
    tol = TOL[shape.dtype]
    Xd = up(X, shape.dtype)
    Kd = torch.empty(N, shape.n_kv_heads, shape.head_dim, dtype=lib.dtype, device=dev())
    S = lib.pap_score(Wd, Xd, i32(pos), K_out=Kd)
    A = O.rmsnorm(X, np.ones(shape.hidden), shape.rms_eps)
    Ko, qo, So = O.pap_score(A, pos, W["wk"].astype(np.float64), W["wq"].astype(np.float64), shape)
    check_output(host(Kd), O.rounding("bf16" if shape.dtype == "bf16" else "exact")(Ko), shape.dtype)
    assert np.abs(host(S) - So).max() <= 2e-4 * So.max()
    assert abs(host(S).sum() - 1.0) < 1e-4
    # LTP on the same rows
    Cd = torch.empty(N, dtype=torch.float32, device=dev())
    Sf = lib.ltp_score(Wd, Xd, S, C_out=Cd)
    Co, Sfo = O.ltp_score(A, So, {k: v.astype(np.float64) for k, v in W.items()}, O.rounding("bf16" if shape.dtype == "bf16" else "exact"))
    ctol = 2e-3 if shape.dtype == "bf16" else 1e-4
    assert np.abs(host(Cd) - Co).max() <= ctol * Co.max()
    assert np.abs(host(Sf) - Sfo).max() <= ctol * Sfo.max()
    assert lib.device_status() == 0
    lib.close()


@pytest.mark.parametrize("shape,ref", [(SMALL_BF16, False), (SMALL_BF16, True), (synth.TINY, None),
                                       (replace(SMALL_BF16, ltp_rank=48), False)])
def test_prepared_layer_gives_the_same_bits(shape, ref):
    """spts_prepare_layer moves the repacking of the proxy factors out of the calls; scores and layer outputs must
    not change by a bit.  (The rank-48 shape takes the route without the Gram matrix in tensor-core mode.)"""
    from paper_2601_13155_b200 import binding
    lib = _mk(shape, 1024, ref)
    N, ma, mf = 700, 300, 222
    W, X, Wd = _layer_case(shape, N, 909, 16, std=0.05)
    Wp = lib.prepare_layer(binding.LayerWeights(W, shape.dtype))
    assert Wp.c.prepared and not Wd.c.prepared
    pos = i32(np.arange(N))
    outs = []
    for lw in (Wd, Wp):
        Xd = up(X, shape.dtype)
        S = lib.pap_score(lw, Xd, pos)
        Cd = torch.empty(N, dtype=torch.float32, device=dev())
        Sf = lib.ltp_score(lw, Xd, S, C_out=Cd)
        jf = torch.empty(mf, dtype=torch.int32, device=dev())
        lib.layer_prefill_skip(lw, Xd, pos, ma, mf, binding.KvCache(shape, 1, N), idx_ffn_out=jf)
        outs.append((Cd, Sf, jf, Xd))
    assert lib.device_status() == 0
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    lib.close()


@pytest.mark.parametrize("shape,N,ma,mf,ref", _modes())
def test_layer_matches_oracle(shape, N, ma, mf, ref):
    from paper_2601_13155_b200 import binding
    lib = _mk(shape, 2048, ref)
    W, X, Wd = _layer_case(shape, N, 1001, 32)
    Wmid = binding.LayerWeights(zero_down(W), shape.dtype)
    pos = np.arange(N, dtype=np.int32)
    Xd = up(X, shape.dtype)
    cache = binding.KvCache(shape, 1, N)
    check_layer_blocks(lib, shape, W, Wd, Wmid, Xd, i32(pos), ma, mf, cache)
    lib.close()


@pytest.mark.parametrize("dtype,ref", [("fp32", None), ("bf16", True), ("bf16", False)])
def test_keep_all_equals_dense_and_is_deterministic(dtype, ref):
    from paper_2601_13155_b200 import binding
    shape = SMALL_BF16 if dtype == "bf16" else synth.TINY
    lib = _mk(shape, 1024, ref)
    N = 300
    W, X, Wd = _layer_case(shape, N, 5, 8)
    pos = i32(np.arange(N))
    outs = []
    for _ in range(2):
        Xd = up(X, shape.dtype)
        cache = binding.KvCache(shape, 1, N)
        lib.layer_prefill_skip(Wd, Xd, pos, N, N, cache)
        outs.append(Xd)
    assert torch.equal(outs[0], outs[1])
    want = O.layer_dense(X, np.arange(N), W, shape, mode="bf16" if dtype == "bf16" else "exact")
    check_output(host(outs[0]), want["X"], dtype)
    assert lib.device_status() == 0
    lib.close()


@pytest.mark.parametrize("dtype,ref", [("fp32", None), ("bf16", True), ("bf16", False), ("bf16-oddgroup", False)])
def test_prefill_and_decode_match_oracle(dtype, ref):
    """Algorithm 1 over four layers in two stages, then two decode steps.

    Layers are compared one by one with forced inputs: the oracle receives the GPU's input to
    each layer, so the per-layer tolerance and the 1e-3 index band apply (chained differences
    -- a boundary token swapped in an earlier layer -- would otherwise compound).  The single
    spts_prefill call must then reproduce the per-layer chain bit for bit."""
    from paper_2601_13155_b200 import binding
    base = {"bf16": SMALL_BF16, "fp32": synth.TINY, "bf16-oddgroup": ODD_GROUP_BF16}[dtype]
    dtype = base.dtype
    L = 4
    shape = replace(base, n_layers=L, vocab=1000)
    lib = _mk(shape, 1024, ref)
    N = 384
    layers = [synth.layer_weights(shape, 1010, l, std=0.03) for l in range(L)]
    hw = synth.head_weights(shape, 1010)
    X, _ = synth.hidden_states(shape, N, 1010, heavy=24)
    plan = schedule.stage_plan(L, N, (0, 2), (N, 288), 192, 150)
    assert [p["m_attn"] for p in O.msdp_schedule(L, N, (0, 2), (N, 288), 192, 150)] == [p[0] for p in plan]
    mode = "bf16" if dtype == "bf16" else "exact"
    lws = [binding.LayerWeights(w, dtype) for w in layers]
    model = binding.Model(lws, up(hw["lm_head"], dtype), up(hw["embed"], dtype))
    caps = [p[0] + 4 for p in plan]

    # ---- per-layer chain on the GPU, oracle with forced inputs
    cache = binding.KvCache(shape, L, caps)
    Xd, pos, orig = up(X, dtype), i32(np.arange(N)), i32(np.arange(N))
    lmid = [binding.LayerWeights(zero_down(w), dtype) for w in layers]
    for l, (ma, mf, prune) in enumerate(plan):
        S = check_layer_blocks(lib, shape, layers[l], lws[l], lmid[l], Xd, pos, ma, mf, cache, layer=l)["S"]
        if prune:
            Xn = torch.empty(prune, shape.hidden, dtype=lib.dtype, device=dev())
            pn, on = torch.empty(prune, dtype=torch.int32, device=dev()), torch.empty(prune, dtype=torch.int32, device=dev())
            keep = torch.empty(prune, dtype=torch.int32, device=dev())
            lib.msdp_compact(Xd, pos, orig, S, prune, Xn, pn, on, keep)
            T = O.topk_select(host(S).astype(np.float32), prune, True)      # exact given the GPU's scores
            assert np.array_equal(keep.cpu().numpy(), T)
            assert torch.equal(Xn, Xd[keep.long()]) and torch.equal(pn, pos[keep.long()])
            Xd, pos, orig = Xn, pn, on
    assert lib.device_status() == 0

    # ---- the single-call prefill reproduces the chain bit for bit
    cache2 = binding.KvCache(shape, L, caps)
    X2, Xa = up(X, dtype), torch.empty(N, shape.hidden, dtype=lib.dtype, device=dev())
    p2, o2 = i32(np.arange(N)), i32(np.arange(N))
    pa, oa = torch.empty_like(p2), torch.empty_like(o2)
    tok = torch.zeros(1, dtype=torch.int32, device=dev())
    nf, in_alt = lib.prefill(model, plan, X2, p2, o2, Xa, pa, oa, cache2, token_out=tok)
    assert lib.device_status() == 0
    assert nf == 288 and in_alt
    assert torch.equal(Xa[:nf], Xd) and torch.equal(oa[:nf], orig) and torch.equal(pa[:nf], pos)
    for l in range(L):
        n = cache.length(l)
        assert cache2.length(l) == n
        assert torch.equal(cache2.k[l][:n], cache.k[l][:n]) and torch.equal(cache2.v[l][:n], cache.v[l][:n])
        assert torch.equal(cache2.pos[l][:n], cache.pos[l][:n])
    lg, tk = O.first_token(host(Xd)[-1], np.ones(shape.hidden), hw["lm_head"], shape.rms_eps)
    top2 = np.sort(lg)[-2:]
    if top2[1] - top2[0] > 1e-3 * np.abs(lg).max():
        assert int(tok.item()) == tk

    # ---- two decode steps against the compressed caches; the oracle starts from the GPU's caches
    ocaches = [{"K": host(cache2.k[l][:cache2.length(l)]), "V": host(cache2.v[l][:cache2.length(l)]),
                "pos": cache2.pos[l][:cache2.length(l)].cpu().numpy()} for l in range(L)]
    emb = hw["embed"]
    for step, token in enumerate((17, 523)):
        xo = torch.empty(shape.hidden, dtype=lib.dtype, device=dev())
        lgd = torch.empty(shape.vocab, dtype=torch.float32, device=dev())
        lib.decode_step(model, cache2, N + step, token_in=token, x_out=xo, logits_out=lgd, token_out=tok)
        x, lg, tk = O.decode_step(emb[token], N + step, layers, shape, ocaches, np.ones(shape.hidden),
                                  hw["lm_head"], mode=mode)
        check_output(host(xo), x, dtype, scale=2, what="decode hidden state")
        lg_err = rel_rms_err(host(lgd), lg)
        print(f"[parity] decode step {step}: logits max-abs error {lg_err:.3e} of their RMS")
        assert lg_err <= 2 * TOL[dtype]
        assert all(cache2.length(l) == len(ocaches[l]["pos"]) for l in range(L))
        assert int(tok.item()) == int(np.argmax(host(lgd)))
    assert lib.device_status() == 0
    lib.close()


def _attention_inputs(shape, m, kind, seed):
    """Q [m,H,d], K, V [m,Hkv,d] as the attention step sees them, rounded to the storage type.
    kind "normal": logits ~ N(0, 1).  "peaky": logits ~ N(0, 12^2), rows nearly one-hot, the row maximum moves by tens
    of octaves from one key block to the next in either direction.  "ramp": the logit of key j grows by about half a
    unit per key, so every row's running maximum rises by ~90 octaves per 128-key block and its mass sits on the
    last few keys before the diagonal."""
    rng = np.random.default_rng(seed)
    H, Hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    Q = rng.standard_normal((m, H, d))
    K = rng.standard_normal((m, Hkv, d))
    V = rng.standard_normal((m, Hkv, d))
    if kind == "peaky":
        Q *= 12.0
    elif kind == "ramp":
        u = rng.standard_normal(d)
        u /= np.linalg.norm(u)
        Q = Q + 8.0 * u
        K = K + (np.arange(m)[:, None, None] * (0.5 * np.sqrt(d) / 8.0)) * u
    return tuple(synth.quantize(a.astype(np.float32), shape.dtype) for a in (Q, K, V))


@pytest.mark.parametrize("kind", ["normal", "peaky", "ramp"])
@pytest.mark.parametrize("shape,m,ref", [
    pytest.param(SMALL_BF16, 1101, False, id="pair-kernel-even-group"),
    pytest.param(ODD_GROUP_BF16, 600, False, id="pair-kernel-odd-group"),
    pytest.param(WIDE_GROUP_BF16, 385, False, id="pair-kernel-group16"),
    pytest.param(SMALL_BF16, 129, False, id="pair-kernel-one-past-a-tile"),
    pytest.param(SMALL_BF16, 1, False, id="pair-kernel-single-row"),
    pytest.param(SMALL_BF16, 300, True, id="plain-kernels-bf16"),
    pytest.param(synth.TINY, 389, None, id="plain-kernels-fp32"),
])
def test_reduced_attention_matches_oracle(shape, m, ref, kind):
    """spts_reduced_attention (Algorithm 1's F_MHA(Q^, K^, V^) on the active rows) on operands of the test's choosing
    against the oracle's causal GQA attention on the very same Q, K, V.  The tensor-core kernel keeps its running
    row maximum lazily (O is rescaled only when the maximum has grown by more than 2^8); the "peaky" and "ramp"
    operands make that happen at almost every key block, in the regime where a wrong rescale would show."""
    lib = _mk(shape, 2048, ref)
    Q, K, V = _attention_inputs(shape, m, kind, 4000 + m)
    got = lib.reduced_attention(up(Q, shape.dtype), up(K, shape.dtype), up(V, shape.dtype))
    assert lib.device_status() == 0
    want = O.causal_gqa_attention(Q.astype(np.float64), K.astype(np.float64), V.astype(np.float64))
    if kind != "normal" and m >= 130:
        # the cases are only worth their name if a row's logits really spread by more than the 2^8 threshold
        z = (K[:, 0].astype(np.float64) @ Q[-1, 0].astype(np.float64)) / np.sqrt(shape.head_dim)
        assert z.max() - np.sort(z)[-130] > 8.0 * np.log(2.0)
    # Rows of an attention output are independent averages: row 0 is V[0] itself, row 1000 the mean of a thousand
    # values, thirty times smaller.  The tolerance is therefore taken relative to each row's own RMS.  fp32 mode on
    # the ramp: logits reach ~200, i.e. raw dot products of ~1500 whose fp32 spacing (1.2e-4) times 1/sqrt(d) already
    # moves a probability by ~1e-5 per rounding, so that case gets three times the fp32 bound.
    check_output(host(got), O.rounding("bf16" if shape.dtype == "bf16" else "exact")(want), shape.dtype, per_row=True,
                 scale=3.0 if (shape.dtype == "fp32" and kind == "ramp") else 1.0, what=f"attention {kind}")
    assert lib.check_guards() == 0
    lib.close()


@pytest.mark.parametrize("N,ma,mf", [(1, 1, 1), (2, 1, 2), (3, 2, 1), (17, 5, 17), (129, 128, 1), (257, 129, 130)])
@pytest.mark.parametrize("ref", [True, False])
def test_tiny_and_ragged_sequences(N, ma, mf, ref):
    """Degenerate sizes on the bf16 kernels (tensor-core and plain): a single token, budgets of one row, sizes one
    past a tile edge.  Same block-wise comparison with the oracle as the larger cases."""
    from paper_2601_13155_b200 import binding
    shape = SMALL_BF16
    lib = _mk(shape, 512, ref)
    W, X, Wd = _layer_case(shape, N, 77 + N, min(N, 3))
    Wmid = binding.LayerWeights(zero_down(W), shape.dtype)
    pos = (np.arange(N) * 3 + 1).astype(np.int32)
    Xd = up(X, shape.dtype)
    cache = binding.KvCache(shape, 1, N)
    check_layer_blocks(lib, shape, W, Wd, Wmid, Xd, i32(pos), ma, mf, cache)
    lib.close()


@pytest.mark.parametrize("shape,N,ref", [
    pytest.param(synth.TINY, 389, None, id="tiny-fp32"),
    pytest.param(SMALL_BF16, 777, False, id="small8b-bf16-tensorcore"),
    pytest.param(ODD_GROUP_BF16, 300, False, id="oddgroup-bf16-tensorcore"),
    pytest.param(SMALL_BF16, 40, True, id="small8b-bf16-refkernels-short"),
])
@pytest.mark.parametrize("window", [4, 64])
def test_window_probe_matches_oracle(shape, N, ref, window):
    """The probe score averaged over the last `window` queries (SPTS_PAP_WINDOW; the paper's query-length ablation):
    every query over its causal range, K and the queries as stored.  Also through the layer call: its S_out is the
    windowed score and its attention set the top-k of it."""
    from paper_2601_13155_b200 import binding
    lib = _mk(shape, 1024, ref)
    lib.set_pap_window(window)
    W, X, Wd = _layer_case(shape, N, 1003, 16, std=0.05)
    pos = (np.arange(N) * 2 + 5).astype(np.int32)
    Xd = up(X, shape.dtype)
    S = lib.pap_score(Wd, Xd, i32(pos))
    A = O.rmsnorm(X, np.ones(shape.hidden), shape.rms_eps)
    rnd = O.rounding("bf16" if shape.dtype == "bf16" else "exact")
    _, So = O.pap_score_window(A, pos, W["wk"].astype(np.float64), W["wq"].astype(np.float64), shape, window, rnd)
    assert np.abs(host(S) - So).max() <= 2e-4 * So.max()
    assert abs(host(S).sum() - 1.0) < 1e-4
    ma = max(1, N // 3)
    S2 = torch.empty(N, dtype=torch.float32, device=dev())
    ia = torch.empty(ma, dtype=torch.int32, device=dev())
    lib.layer_prefill_skip(Wd, Xd, i32(pos), ma, N, binding.KvCache(shape, 1, N), S_out=S2, idx_attn_out=ia)
    assert torch.equal(S2, S)
    check_index_set(ia.cpu().numpy(), So, ma)
    assert lib.device_status() == 0
    lib.close()


def test_decode_steps_are_reproducible_bit_for_bit():
    """The decode kernels of a step overlap (programmatic dependent launches): two runs from the same caches must still
    give identical logits and tokens, step after step."""
    from paper_2601_13155_b200 import binding
    L = 3
    shape = replace(SMALL_BF16, n_layers=L, vocab=2000)
    lib = _mk(shape, 1024, False)
    layers = [synth.layer_weights(shape, 1020, l, std=0.03) for l in range(L)]
    hw = synth.head_weights(shape, 1020)
    lws = [binding.LayerWeights(w, "bf16") for w in layers]
    model = binding.Model(lws, up(hw["lm_head"], "bf16"), up(hw["embed"], "bf16"))
    n0, steps = 700, 12
    rng = np.random.default_rng(8)
    k0 = [up(rng.standard_normal((n0, shape.n_kv_heads, shape.head_dim)).astype(np.float32), "bf16") for _ in range(L)]
    v0 = [up(rng.standard_normal((n0, shape.n_kv_heads, shape.head_dim)).astype(np.float32), "bf16") for _ in range(L)]
    runs = []
    for _ in range(2):
        cache = binding.KvCache(shape, L, n0 + steps)
        for l in range(L):
            cache.k[l][:n0].copy_(k0[l])
            cache.v[l][:n0].copy_(v0[l])
            cache.c[l].len = n0
        tok = torch.zeros(1, dtype=torch.int32, device=dev())
        out, t_in = [], 11
        for i in range(steps):
            lg = torch.empty(shape.vocab, dtype=torch.float32, device=dev())
            lib.decode_step(model, cache, n0 + i, token_in=t_in, logits_out=lg, token_out=tok)
            t_in = int(tok.item())
            out.append((lg.clone(), t_in))
        runs.append(out)
    for (a, ta), (b, tb) in zip(*runs):
        assert ta == tb and torch.equal(a, b)
    assert lib.device_status() == 0
    lib.close()


DECODE_HEAD_LAYOUTS = {
    # name: (query heads, KV heads, head dim) -- the GQA group decides how the query heads fill the 16 fragment rows
    "group4_d128": (8, 2, 128),        # the 8B layout: rows 0..3 of one block
    "group7_d128": (7, 1, 128),        # an odd group (the Qwen layout)
    "group12_d128": (12, 1, 128),      # both halves of the fragment carry heads
    "group20_d64": (20, 1, 64),        # two blocks per KV head (16 + 4 query heads), head dim 64
    "group1_d64": (4, 4, 64),          # no grouping
}


@pytest.mark.parametrize("layout", sorted(DECODE_HEAD_LAYOUTS))
@pytest.mark.parametrize("n0", [5, 2077])
def test_decode_attention_over_long_caches(layout, n0):
    """Decode against synthetic caches long enough for many slices per head (2077 rows: 16 ragged slices, each
    shared by four warps in 16-row groups with a masked tail) and against a 5-row cache, for head layouts that fill
    the tensor-core fragments differently.  Two steps, so the second reads the row the first appended."""
    from paper_2601_13155_b200 import binding
    H, Hkv, hd = DECODE_HEAD_LAYOUTS[layout]
    shape = replace(synth.LLAMA8B, hidden=256, n_q_heads=H, n_kv_heads=Hkv, head_dim=hd, ffn_dim=512,
                    ltp_dlow=128, ltp_rank=32, n_layers=1, vocab=1000)
    lib = _mk(shape, 1024, hd != 128)           # the prefill tensor-core kernels want head dim 128; decode has no such limit
    # a large W_o and no FFN update (W_down = 0): the step's output is dominated by the attention result
    W = zero_down(synth.layer_weights(shape, 1030, 0, std=0.05))
    W["wo"] = synth.quantize(W["wo"] * np.float32(8.0), "bf16")
    hw = synth.head_weights(shape, 1030)
    model = binding.Model([binding.LayerWeights(W, "bf16")], up(hw["lm_head"], "bf16"), up(hw["embed"], "bf16"))
    rng = np.random.default_rng(n0)
    k0 = up((3.0 * rng.standard_normal((n0, Hkv, hd))).astype(np.float32), "bf16")
    v0 = up(rng.standard_normal((n0, Hkv, hd)).astype(np.float32), "bf16")
    cache = binding.KvCache(shape, 1, n0 + 2)
    cache.k[0][:n0].copy_(k0)
    cache.v[0][:n0].copy_(v0)
    cache.pos[0][:n0].copy_(i32(np.arange(n0)))
    cache.c[0].len = n0
    oc = [{"K": host(k0), "V": host(v0), "pos": np.arange(n0)}]
    tok = torch.zeros(1, dtype=torch.int32, device=dev())
    for step, token in enumerate((3, 998)):
        xo = torch.empty(shape.hidden, dtype=lib.dtype, device=dev())
        lg = torch.empty(shape.vocab, dtype=torch.float32, device=dev())
        lib.decode_step(model, cache, n0 + step, token_in=token, x_out=xo, logits_out=lg, token_out=tok)
        x, lgo, _ = O.decode_step(hw["embed"][token], n0 + step, [W], shape, oc, np.ones(shape.hidden), hw["lm_head"],
                                  mode="bf16")
        check_output(host(xo), x, "bf16", scale=2)
        assert rel_rms_err(host(lg), lgo) <= 2 * TOL["bf16"]
        check_output(host(cache.k[0][n0 + step]), oc[0]["K"][n0 + step], "bf16")
    assert cache.length(0) == n0 + 2 and lib.device_status() == 0
    lib.close()


@pytest.mark.parametrize("dtype,ref", [("fp32", None), ("bf16", False)])
def test_ffn_selection_by_the_attention_score_alone(dtype, ref):
    """The setting of the paper's proxy-network ablation (Table 4): attention dense, 40 % of the tokens skipped in the
    FFN block, selected by S_mha (Eq. 4) alone.  T_f must be exactly TopK of the library's own S_mha, the update must
    match the oracle run with the same criterion, and switching the option off must bring Eq. 14 back."""
    shape = SMALL_BF16 if dtype == "bf16" else synth.TINY
    N, mf = 640, 384
    lib = _mk(shape, 1024, ref)
    W, X, lw = _layer_case(shape, N, 1041, heavy=16, std=0.03)
    from paper_2601_13155_b200 import binding
    pos = i32(np.arange(N) * 3 + 1)
    out = {}
    for on in (True, False):
        lib.set_ffn_score_pap_only(on)
        Xd = up(X, shape.dtype)
        S = torch.empty(N, dtype=torch.float32, device=dev())
        jf = torch.empty(mf, dtype=torch.int32, device=dev())
        lib.layer_prefill_skip(lw, Xd, pos, N, mf, binding.KvCache(shape, 1, N), S_out=S, idx_ffn_out=jf)
        assert lib.device_status() == 0
        out[on] = (host(Xd), host(S).astype(np.float32), jf.cpu().numpy())
    xg, Sg, jg = out[True]
    assert np.array_equal(jg, O.topk_select(Sg, mf, True))
    mode = "bf16" if shape.dtype == "bf16" else "exact"
    want = O.layer_prefill_skip(X, np.arange(N) * 3 + 1, W, shape, N, mf, mode=mode, ffn_criterion="pap")
    assert np.abs(Sg - want["S_mha"]).max() <= 2e-4 * want["S_mha"].max()
    check_index_set(jg, want["S_mha"], mf)
    same = np.setdiff1d(np.arange(N), np.setxor1d(jg, want["idx_ffn"]))
    check_output(xg[same], want["X"][same], shape.dtype)
    # with the option off the proxy decides again: a different set on these inputs
    assert not np.array_equal(out[False][2], jg)
    lib.close()


@pytest.mark.parametrize("dtype,ref", [("fp32", None), ("bf16", False), ("bf16", True), ("bf16-oddgroup", False),
                                       ("bf16-group16", False)])
def test_packed_batch_equals_one_call_per_sequence(dtype, ref):
    """spts_layer_prefill_skip_batch on four ragged prompts (one of them dense in the FFN, one dense in attention, one a
    single token) against spts_layer_prefill_skip on each prompt alone: hidden states, scores, both index lists and the
    caches must agree bit for bit -- the packed FFN GEMMs compute every row exactly as the per-sequence ones do -- and
    the single-sequence call is what the oracle comparisons above cover."""
    from paper_2601_13155_b200 import binding
    shape = {"bf16": SMALL_BF16, "fp32": synth.TINY, "bf16-oddgroup": ODD_GROUP_BF16, "bf16-group16": WIDE_GROUP_BF16}[dtype]
    lens = [300, 1, 517, 130]
    ma = [150, 1, 517, 70]
    mf = [120, 1, 200, 130]
    start = np.concatenate([[0], np.cumsum(lens)])
    total = int(start[-1])
    lib = _mk(shape, 1024, ref)
    W, X, lw = _layer_case(shape, total, 1051, heavy=20, std=0.03)
    pos_h = np.concatenate([np.arange(n) * 2 + 5 * b for b, n in enumerate(lens)]).astype(np.int32)
    pos = i32(pos_h)
    # one call per sequence
    Xs = up(X, shape.dtype)
    Ss = torch.zeros(total, dtype=torch.float32, device=dev())
    single = binding.KvCache(shape, len(lens), [m + 1 for m in ma])
    ia_s, jf_s = [], []
    for b, n in enumerate(lens):
        s0 = int(start[b])
        ia = torch.empty(ma[b], dtype=torch.int32, device=dev())
        jf = torch.empty(mf[b], dtype=torch.int32, device=dev())
        lib.layer_prefill_skip(lw, Xs[s0:s0 + n], pos[s0:s0 + n], ma[b], mf[b], single, layer=b, S_out=Ss[s0:s0 + n],
                               idx_attn_out=ia, idx_ffn_out=jf)
        ia_s.append(ia)
        jf_s.append(jf)
    # the packed call
    Xb = up(X, shape.dtype)
    Sb = torch.zeros(total, dtype=torch.float32, device=dev())
    packed = binding.KvCache(shape, len(lens), [m + 1 for m in ma])
    ia_b = torch.empty(sum(ma), dtype=torch.int32, device=dev())
    jf_b = torch.empty(sum(mf), dtype=torch.int32, device=dev())
    lib.layer_prefill_skip_batch(lw, Xb, pos, start, ma, mf, packed, S_out=Sb, idx_attn_out=ia_b, idx_ffn_out=jf_b)
    assert lib.device_status() == 0
    assert torch.equal(Xb, Xs)
    assert torch.equal(ia_b, torch.cat(ia_s)) and torch.equal(jf_b, torch.cat(jf_s))
    for b, n in enumerate(lens):
        s0 = int(start[b])
        if ma[b] < n or mf[b] < n:
            assert torch.equal(Sb[s0:s0 + n], Ss[s0:s0 + n])
        assert packed.length(b) == ma[b] == single.length(b)
        assert torch.equal(packed.k[b][:ma[b]], single.k[b][:ma[b]])
        assert torch.equal(packed.v[b][:ma[b]], single.v[b][:ma[b]])
        assert torch.equal(packed.pos[b][:ma[b]], single.pos[b][:ma[b]])
    # and without the optional outputs
    Xc = up(X, shape.dtype)
    lib.layer_prefill_skip_batch(lw, Xc, pos, start, ma, mf, binding.KvCache(shape, len(lens), [m + 1 for m in ma]))
    assert torch.equal(Xc, Xs)
    # host-side argument checks: a budget above the sequence length, a start list that does not begin at 0
    with pytest.raises(binding.SptsError):
        lib.layer_prefill_skip_batch(lw, Xc, pos, start, [150, 2, 517, 70], mf, packed)
    with pytest.raises(binding.SptsError):
        lib.layer_prefill_skip_batch(lw, Xc, pos, start + 1, ma, mf, packed)
    assert lib.device_status() == 0
    lib.close()
