"""GPU parity of spts_topk_select and spts_msdp_compact against the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import spts_oracle as O
from paper_2601_13155_b200 import synth
from parity_utils import dev, i32, up

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2601_13155_b200 import binding
    s = binding.Spts(synth.TINY, max_seq=1 << 18)
    yield s
    s.close()


def _scores_cases():
    rng = np.random.default_rng(21)
    out = []
    for n in (1, 2, 3, 17, 64, 513, 2048, 2049, 5000, 40000):
        out.append(rng.standard_normal(n).astype(np.float32))
        out.append(rng.integers(0, 5, n).astype(np.float32))            # heavy ties
        out.append(np.full(n, 0.25, np.float32))                        # all equal
    out.append(np.array([0.0, -0.0, 0.0, -0.0, 1.0, -1.0, -0.0], np.float32))
    z = rng.standard_normal(3000).astype(np.float32) * 1e-40            # denormals
    out.append(z)
    e = np.exp(rng.standard_normal(131072) * 2).astype(np.float32)
    out.append((e / e.sum()).astype(np.float32))                        # softmax-like, full length
    return out


@pytest.mark.parametrize("force_last", [0, 1])
def test_topk_matches_oracle(lib, force_last):
    for s in _scores_cases():
        n = len(s)
        ks = sorted({1, 2, n // 3, n // 2, n - 1, n} - {0})
        d = torch.from_numpy(s).to(dev())
        for k in ks:
            if k > n:
                continue
            got = lib.topk_select(d, k, flags=force_last).cpu().numpy()
            want = O.topk_select(s, k, bool(force_last))
            assert np.array_equal(got, want), (n, k, force_last)
    assert lib.device_status() == 0


def test_topk_nan_ranks_last_and_is_reported(lib):
    s = np.array([np.nan, 1.0, 0.5, np.nan, 2.0, -3.0], np.float32)
    got = lib.topk_select(torch.from_numpy(s).to(dev()), 4).cpu().numpy()
    assert got.tolist() == O.topk_select(s, 4).tolist() == [1, 2, 4, 5]
    assert lib.device_status() == 6          # SPTS_ERR_NONFINITE, then cleared
    assert lib.device_status() == 0


def test_topk_rejects_bad_arguments(lib):
    from paper_2601_13155_b200.binding import SptsError
    d = torch.zeros(8, device=dev())
    for k in (0, 9, -1):
        with pytest.raises(SptsError):
            lib.topk_select(d, k)


def test_topk_is_deterministic(lib):
    rng = np.random.default_rng(3)
    s = torch.from_numpy(rng.integers(0, 50, 100000).astype(np.float32)).to(dev())
    a = lib.topk_select(s, 33333).clone()
    for _ in range(3):
        assert torch.equal(a, lib.topk_select(s, 33333))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_compact_matches_oracle(dtype):
    from dataclasses import replace
    from paper_2601_13155_b200 import binding
    shape = replace(synth.TINY, dtype=dtype)
    lib = binding.Spts(shape, max_seq=8192)
    lib.set_reference_kernels(True)
    rng = np.random.default_rng(5)
    for n, keep in ((1, 1), (37, 11), (513, 512), (4099, 1500), (4099, 4099), (4099, 9000)):
        X, _ = synth.hidden_states(shape, n, 77)
        pos = np.cumsum(rng.integers(1, 4, n)).astype(np.int32)
        orig = (np.arange(n) * 2 + 1).astype(np.int32)
        S = rng.random(n).astype(np.float32)
        kk = min(n, keep)
        Xo = torch.empty(kk, shape.hidden, dtype=lib.dtype, device=dev())
        po = torch.empty(kk, dtype=torch.int32, device=dev())
        oo = torch.empty(kk, dtype=torch.int32, device=dev())
        io = torch.empty(kk, dtype=torch.int32, device=dev())
        Xd = up(X, dtype)
        lib.msdp_compact(Xd, i32(pos), i32(orig), torch.from_numpy(S).to(dev()), keep, Xo, po, oo, io)
        wX, wp, wo, wT = O.msdp_compact(X, pos, orig, S, keep)
        assert np.array_equal(io.cpu().numpy(), wT)
        assert torch.equal(Xo, Xd[torch.from_numpy(wT).to(dev())])          # rows bit-identical
        assert np.array_equal(Xo.float().cpu().numpy().astype(np.float64), wX.astype(np.float64))
        assert np.array_equal(po.cpu().numpy(), wp) and np.array_equal(oo.cpu().numpy(), wo)
        assert np.all(np.diff(po.cpu().numpy()) > 0) if kk > 1 else True
    assert lib.device_status() == 0
    lib.close()


def test_host_detectable_errors_are_returned_before_any_launch():
    """Bad shapes, undersized caches and misaligned pointers come back as status codes (nothing is launched, the
    buffers stay untouched, the device status stays clean)."""
    from paper_2601_13155_b200 import binding
    from paper_2601_13155_b200.binding import SptsError
    shape = synth.TINY
    lib = binding.Spts(shape, max_seq=256)
    W = synth.layer_weights(shape, 3, 0)
    Wd = binding.LayerWeights(W, shape.dtype)
    N = 128
    X, _ = synth.hidden_states(shape, N, 3)
    Xd = up(X, shape.dtype)
    X0 = Xd.clone()
    pos = i32(np.arange(N))
    launches = lib.launch_count()

    def code(fn):
        with pytest.raises(SptsError) as e:
            fn()
        return e.value.code

    small = binding.KvCache(shape, 1, 16)
    assert code(lambda: lib.layer_prefill_skip(Wd, Xd, pos, 64, 64, small)) == 3            # WORKSPACE: cache too small
    ok = binding.KvCache(shape, 1, N)
    assert code(lambda: lib.layer_prefill_skip(Wd, Xd, pos, 0, 64, ok)) == 1                # INVALID_ARG: m_attn < 1
    assert code(lambda: lib.layer_prefill_skip(Wd, Xd, pos, N + 1, 64, ok)) == 1            # INVALID_ARG: m_attn > N
    big = up(synth.hidden_states(shape, 300, 4)[0], shape.dtype)
    assert code(lambda: lib.pap_score(Wd, big, i32(np.arange(300)))) == 2                    # SHAPE: N > max_seq
    odd = torch.empty(N * shape.hidden + 1, dtype=lib.dtype, device=dev())[1:].view(N, shape.hidden)
    assert code(lambda: lib.pap_score(Wd, odd, pos)) == 1                                    # INVALID_ARG: misaligned X
    S = torch.zeros(N, device=dev())
    Xo = torch.empty(N, shape.hidden, dtype=lib.dtype, device=dev())
    assert code(lambda: lib.msdp_compact(Xd, pos, pos.clone(), S, 64, Xd, pos.clone(), pos.clone())) == 1   # aliasing
    with pytest.raises(SptsError):
        binding.Spts(replace_shape(shape, head_dim=96), max_seq=64)                           # unsupported shape
    assert lib.launch_count() == launches
    assert torch.equal(Xd, X0)
    assert lib.device_status() == 0
    lib.close()


def replace_shape(shape, **kw):
    from dataclasses import replace
    return replace(shape, **kw)
