"""Stand-ins for a memory checker and for fault injection, none of which faults, traps or hangs the GPU:
guard bands behind every workspace slice and around caller outputs, the device-side index-list check, and the
give-up path of the bounded barrier waits run on barriers nobody arrives on with a 1 ms limit."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2601_13155_b200 import synth
from parity_utils import Guarded, dev, i32, up

pytestmark = pytest.mark.gpu

SMALL_BF16 = replace(synth.LLAMA8B, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn_dim=1024,
                     ltp_dlow=128, ltp_rank=32, n_layers=2, vocab=1024)


@pytest.mark.parametrize("shape,ref", [(SMALL_BF16, False), (SMALL_BF16, True), (replace(synth.TINY, n_layers=2), None)])
def test_guard_bands_survive_every_call(shape, ref):
    """Ragged sizes one past the tile edges through every entry point that uses the workspace; afterwards every band
    behind a workspace slice and around the caller's outputs still holds its pattern."""
    from paper_2601_13155_b200 import binding, schedule
    N = 641
    lib = binding.Spts(shape, max_seq=N)
    if ref is not None:
        lib.set_reference_kernels(ref)
    assert lib.check_guards() == 0
    layers = [synth.layer_weights(shape, 303, l) for l in range(2)]
    lws = [binding.LayerWeights(w, shape.dtype) for w in layers]
    hw = synth.head_weights(shape, 303)
    model = binding.Model(lws, up(hw["lm_head"], shape.dtype), up(hw["embed"], shape.dtype))
    X, _ = synth.hidden_states(shape, N, 303, heavy=8)
    gX, gXa = Guarded((N, shape.hidden), lib.dtype), Guarded((N, shape.hidden), lib.dtype)
    gX.t.copy_(up(X, shape.dtype))
    gp, go, gpa, goa = (Guarded((N,), torch.int32) for _ in range(4))
    gp.t.copy_(i32(np.arange(N)))
    go.t.copy_(i32(np.arange(N)))
    gS, gC, gSf = (Guarded((N,), torch.float32) for _ in range(3))
    gK = Guarded((N, shape.n_kv_heads, shape.head_dim), lib.dtype)
    lib.pap_score(lws[0], gX.t, gp.t, K_out=gK.t, S_out=gS.t)
    lib.ltp_score(lws[0], gX.t, gS.t, C_out=gC.t, S_out=gSf.t)
    gi = Guarded((257,), torch.int32)
    lib.topk_select(gSf.t, 257, flags=1, idx_out=gi.t)
    plan = schedule.stage_plan(2, N, (0, 1), (N, 385), 321, 257)
    cache = binding.KvCache(shape, 2, [p[0] + 2 for p in plan])
    gtok = Guarded((1,), torch.int32)
    lib.set_debug_checks(True)
    nf, in_alt = lib.prefill(model, plan, gX.t, gp.t, go.t, gXa.t, gpa.t, goa.t, cache, token_out=gtok.t)
    gx1, glg = Guarded((shape.hidden,), lib.dtype), Guarded((shape.vocab,), torch.float32)
    lib.decode_step(model, cache, N, token_in=5, x_out=gx1.t, logits_out=glg.t, token_out=gtok.t)
    assert lib.device_status() == 0
    assert nf == 385 and in_alt
    for g in (gX, gXa, gp, go, gpa, goa, gS, gC, gSf, gK, gi, gtok, gx1, glg):
        assert g.intact()
    assert lib.check_guards() == 0
    lib.close()


def test_device_index_check_flags_bad_lists_only():
    from paper_2601_13155_b200 import binding
    lib = binding.Spts(synth.TINY, max_seq=4096)
    good = i32(np.arange(0, 3000, 3))
    lib.debug_check_index_list(good, 3000)
    assert lib.device_status() == 0
    for bad, N in ((np.array([0, 5, 5, 9]), 10),          # a repeated entry
                   (np.array([0, 7, 6, 9]), 10),          # not ascending
                   (np.array([0, 5, 6, 10]), 10),         # beyond the candidate count
                   (np.array([-1, 5, 6, 9]), 10)):        # negative
        lib.debug_check_index_list(i32(bad), N)
        assert lib.device_status() == 8                   # SPTS_ERR_INDEX, and the word is cleared by the read
        assert lib.device_status() == 0
    # with the option on, the library's own selections are checked and pass
    lib.set_debug_checks(True)
    s = torch.rand(3000, device=dev())
    lib.topk_select(s, 1234, flags=1)
    assert lib.device_status() == 0
    lib.close()


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """Two roles wait on barriers nothing ever arrives on, with the limit cut to 1 ms: the first gives up on the
    clock, the second because of the first's flag, the CTA records SPTS_ERR_TIMEOUT and exits; the next call on the
    same context works."""
    import time
    from paper_2601_13155_b200 import binding
    lib = binding.Spts(SMALL_BF16, max_seq=1024)
    t0 = time.time()
    lib.selftest_wait_timeout(1000)
    assert lib.device_status() == 5                       # SPTS_ERR_TIMEOUT
    assert time.time() - t0 < 1.0                         # ended by the 1 ms limit, not by the kernels' 2 s one
    assert lib.device_status() == 0
    s = torch.rand(2000, device=dev())
    idx = lib.topk_select(s, 100)
    assert lib.device_status() == 0
    assert torch.equal(idx.long().sort().values, torch.topk(s, 100).indices.sort().values)
    with pytest.raises(binding.SptsError):
        lib.selftest_wait_timeout(0)
    lib.close()
