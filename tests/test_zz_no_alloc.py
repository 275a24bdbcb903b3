"""spts_topk_select_static: the top-k entry point for callers that cannot allocate device memory (hosts with a
frozen memory plan, plugins that only receive input/output buffers).  Its scratch is a fixed array inside the
library, so it needs neither a context nor a workspace.  Checked here through the C-ABI against the ordinary
entry point, bit for bit (index lists are integers), on calls in a row that share the array.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(77)
    e = np.exp(rng.standard_normal(100000) * 2).astype(np.float32)
    return [
        (rng.standard_normal(5000).astype(np.float32), 1234, 0),
        (rng.integers(0, 4, 40000).astype(np.float32), 13000, 1),       # heavy ties; last element forced in
        ((e / e.sum()).astype(np.float32), 50000, 1),                    # softmax-like scores
        (rng.standard_normal(513).astype(np.float32), 512, 0),
        (rng.standard_normal(64).astype(np.float32), 64, 0),             # k == N: identity list
        (rng.standard_normal(3).astype(np.float32), 1, 1),
    ]


def test_static_topk_equals_workspace_topk_on_calls_in_a_row():
    from paper_2601_13155_b200 import binding, synth
    dev = torch.device("cuda:0")
    lib = binding.Spts(synth.TINY, max_seq=1 << 17)
    for rep in range(2):                       # the second round runs on whatever the first left in the array
        for s, k, flags in _cases():
            d = torch.from_numpy(s).to(dev)
            out = torch.full((k,), -1, dtype=torch.int32, device=dev)
            binding.topk_select_static(d, k, flags, idx_out=out)
            want = lib.topk_select(d, k, flags=flags)
            assert torch.equal(out, want), (rep, len(s), k, flags)
    # two calls back to back on one stream with nothing in between
    (s1, k1, f1), (s2, k2, f2) = _cases()[1], _cases()[2]
    d1, d2 = torch.from_numpy(s1).to(dev), torch.from_numpy(s2).to(dev)
    o1 = torch.empty(k1, dtype=torch.int32, device=dev)
    o2 = torch.empty(k2, dtype=torch.int32, device=dev)
    binding.topk_select_static(d1, k1, f1, idx_out=o1)
    binding.topk_select_static(d2, k2, f2, idx_out=o2)
    assert torch.equal(o1, lib.topk_select(d1, k1, flags=f1))
    assert torch.equal(o2, lib.topk_select(d2, k2, flags=f2))
    assert lib.device_status() == 0
    lib.close()


def test_static_topk_rejects_bad_sizes_before_launching():
    from paper_2601_13155_b200 import binding
    d = torch.zeros(8, device="cuda:0")
    o = torch.zeros(8, dtype=torch.int32, device="cuda:0")
    lib = binding.load_library()
    st = torch.cuda.current_stream().cuda_stream
    assert lib.spts_topk_select_static(d.data_ptr(), binding.TOPK_STATIC_MAX_N + 1, 4, 0, o.data_ptr(), st) == 2   # SHAPE
    for n, k in ((8, 0), (8, 9), (0, 1)):
        assert lib.spts_topk_select_static(d.data_ptr(), n, k, 0, o.data_ptr(), st) == 1                           # INVALID_ARG
    assert lib.spts_topk_select_static(None, 8, 4, 0, o.data_ptr(), st) == 1
    torch.cuda.synchronize()
    assert torch.count_nonzero(o).item() == 0
