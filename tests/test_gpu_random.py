"""Seeded random cases through the C-ABI on small model shapes: layer calls against the oracle block by block, packed
batches against one call per prompt (bit for bit), decode steps against the oracle from synthetic caches.  The shapes,
sequence lengths, budgets and positions are drawn from a fixed seed, so the cases are the same on every run; they are
there to reach combinations the hand-picked cases leave out (budgets of 1, prompts of 1-3 tokens, lengths just
around tile edges, an odd GQA group, a single KV head)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import spts_oracle as O
from paper_2601_13155_b200 import synth
from parity_utils import check_layer_blocks, check_output, dev, host, i32, up, zero_down

pytestmark = pytest.mark.gpu

SMALL = replace(synth.LLAMA8B, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn_dim=1024, ltp_dlow=128,
                ltp_rank=32, n_layers=1, vocab=1024)
ODD = replace(synth.LLAMA8B, hidden=384, n_q_heads=6, n_kv_heads=2, head_dim=128, ffn_dim=768, ltp_dlow=128,
              ltp_rank=32, n_layers=1, vocab=1024)
ONE_KV = replace(synth.LLAMA8B, hidden=896, n_q_heads=7, n_kv_heads=1, head_dim=128, ffn_dim=1280, ltp_dlow=256,
                 ltp_rank=64, n_layers=1, vocab=1024)
SHAPES = [SMALL, ODD, ONE_KV, synth.TINY]
EDGE_LENGTHS = [1, 2, 3, 17, 127, 128, 129, 255, 256, 257, 300, 511, 640, 777, 1000]


def _lib(shape, rng):
    from paper_2601_13155_b200 import binding
    lib = binding.Spts(shape, max_seq=1024)
    if shape.dtype == "bf16":
        lib.set_reference_kernels(bool(rng.integers(0, 2)) if shape is SMALL else False)
    return lib


@pytest.mark.parametrize("seed", range(12))
def test_random_layer_cases(seed):
    from paper_2601_13155_b200 import binding
    rng = np.random.default_rng(5000 + seed)
    for _ in range(3):
        shape = SHAPES[rng.integers(0, len(SHAPES))]
        lib = _lib(shape, rng)
        N = int(rng.choice(EDGE_LENGTHS + [int(rng.integers(1, 1024))]))
        ma = N if rng.random() < 0.2 else int(rng.integers(1, N + 1))
        mf = N if rng.random() < 0.2 else int(rng.integers(1, N + 1))
        ws = int(rng.integers(1, 10 ** 6))
        W = synth.layer_weights(shape, ws, 0, std=0.03)
        X, _ = synth.hidden_states(shape, N, ws, heavy=min(N, 8))
        lw, lmid = binding.LayerWeights(W, shape.dtype), binding.LayerWeights(zero_down(W), shape.dtype)
        pos = i32(np.sort(rng.choice(4 * N + 8, size=N, replace=False)))      # increasing, with gaps
        check_layer_blocks(lib, shape, W, lw, lmid, up(X, shape.dtype), pos, ma, mf, binding.KvCache(shape, 1, N))
        assert lib.device_status() == 0
        lib.close()


@pytest.mark.parametrize("seed", range(8))
def test_random_packed_batches(seed):
    from paper_2601_13155_b200 import binding
    rng = np.random.default_rng(6000 + seed)
    shape = SHAPES[rng.integers(0, len(SHAPES))]
    lib = _lib(shape, rng)
    nseq = int(rng.integers(1, 7))
    lens = [int(rng.integers(1, 1024 // nseq + 1)) for _ in range(nseq)]
    ma = [int(rng.integers(1, n + 1)) for n in lens]
    mf = [n if rng.random() < 0.25 else int(rng.integers(1, n + 1)) for n in lens]
    start = np.concatenate([[0], np.cumsum(lens)])
    total = int(start[-1])
    W = synth.layer_weights(shape, 77 + seed, 0, std=0.03)
    X, _ = synth.hidden_states(shape, total, 77 + seed, heavy=min(total, 8))
    lw = binding.LayerWeights(W, shape.dtype)
    pos = i32(np.concatenate([np.arange(n) * 2 + b for b, n in enumerate(lens)]))
    Xs, Xb = up(X, shape.dtype), up(X, shape.dtype)
    c1 = binding.KvCache(shape, nseq, [m + 1 for m in ma])
    c2 = binding.KvCache(shape, nseq, [m + 1 for m in ma])
    for b, n in enumerate(lens):
        s0 = int(start[b])
        lib.layer_prefill_skip(lw, Xs[s0:s0 + n], pos[s0:s0 + n], ma[b], mf[b], c1, layer=b)
    lib.layer_prefill_skip_batch(lw, Xb, pos, start, ma, mf, c2)
    assert lib.device_status() == 0
    assert torch.equal(Xs, Xb)
    for b in range(nseq):
        assert c2.length(b) == ma[b]
        assert torch.equal(c1.k[b][:ma[b]], c2.k[b][:ma[b]]) and torch.equal(c1.v[b][:ma[b]], c2.v[b][:ma[b]])
        assert torch.equal(c1.pos[b][:ma[b]], c2.pos[b][:ma[b]])
    lib.close()


@pytest.mark.parametrize("seed", range(10))
def test_random_decode_cases(seed):
    from paper_2601_13155_b200 import binding
    rng = np.random.default_rng(7000 + seed)
    shape = [SMALL, ODD, ONE_KV][rng.integers(0, 3)]
    n0 = int(rng.choice([1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 255, 256, 257, 1000, 2077,
                         int(rng.integers(1, 6000))]))
    lib = binding.Spts(shape, max_seq=1024)
    W = zero_down(synth.layer_weights(shape, 900 + seed, 0, std=0.05))
    W["wo"] = synth.quantize(W["wo"] * np.float32(8.0), "bf16")       # the step's output is dominated by attention
    hw = synth.head_weights(shape, 900 + seed)
    model = binding.Model([binding.LayerWeights(W, "bf16")], up(hw["lm_head"], "bf16"), up(hw["embed"], "bf16"))
    k0 = up((3.0 * rng.standard_normal((n0, shape.n_kv_heads, shape.head_dim))).astype(np.float32), "bf16")
    v0 = up(rng.standard_normal((n0, shape.n_kv_heads, shape.head_dim)).astype(np.float32), "bf16")
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
        x, _, _ = O.decode_step(hw["embed"][token], n0 + step, [W], shape, oc, np.ones(shape.hidden), hw["lm_head"],
                                mode="bf16")
        check_output(host(xo), x, "bf16", scale=2)
        assert int(tok.item()) == int(np.argmax(host(lg)))
    assert lib.device_status() == 0 and cache.length(0) == n0 + 2
    lib.close()
