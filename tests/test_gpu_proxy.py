"""GPU parity of the offline proxy-FFN construction (Section 3.3) against the CPU oracle: channel importance,
selected channels, singular values and the rank-r products U V of the three reduced projections.

Singular vectors are only unique up to sign, so the factors are compared through what is unique: the product
U V (the best rank-r approximation) and the singular values; the selected channel set must equal the oracle's
outside a 1e-3 relative band at the D_low-th importance."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import spts_oracle as O
from paper_2601_13155_b200 import synth
from parity_utils import check_index_set, dev, host, up

pytestmark = pytest.mark.gpu

SMALL_BF16 = replace(synth.LLAMA8B, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn_dim=1024,
                     ltp_dlow=128, ltp_rank=32, n_layers=1, vocab=1024)


def _case(shape, n_cal, seed, rho, ref=None):
    from paper_2601_13155_b200 import binding
    lib = binding.Spts(shape, max_seq=1024)
    if ref is not None:
        lib.set_reference_kernels(ref)
    W = synth.layer_weights(shape, seed, 0, std=0.05)
    # give the channels different scales so that importance is not flat
    rng = np.random.default_rng(seed)
    scale = np.exp(rng.standard_normal(shape.ffn_dim) * 0.5).astype(np.float32)
    W["w_gate"] = synth.quantize(W["w_gate"] * scale[:, None], shape.dtype)
    Xc, _ = synth.hidden_states(shape, n_cal, seed + 1, heavy=5)
    Wd = binding.LayerWeights(W, shape.dtype)
    got = lib.proxy_build(Wd, up(Xc, shape.dtype), rho=rho, want_sigma=True)
    assert lib.device_status() == 0
    return lib, W, Wd, Xc, got


@pytest.mark.parametrize("shape,n_cal,rho,ref", [
    pytest.param(synth.TINY, 300, 0.2, None, id="tiny-fp32"),
    pytest.param(synth.TINY, 41, 1.0, None, id="tiny-fp32-all-samples"),
    pytest.param(SMALL_BF16, 777, 0.2, False, id="small8b-bf16-tensorcore"),
    pytest.param(SMALL_BF16, 300, 0.05, True, id="small8b-bf16-refkernels"),
])
def test_proxy_build_matches_oracle(shape, n_cal, rho, ref):
    lib, W, Wd, Xc, got = _case(shape, n_cal, 90, rho, ref)
    fp32 = shape.dtype == "fp32"
    z = O.proxy_saliency(Xc, W, shape)
    imp = O.proxy_channel_importance(z, rho)
    assert np.abs(host(got["importance"]) - imp).max() <= 1e-4 * imp.max()
    C = got["channels"].cpu().numpy().astype(np.int64)
    check_index_set(C, imp, shape.ltp_dlow, force_last=False)
    want = O.proxy_build(Xc, W, shape, rho=rho, channels=C)          # factors of the GPU's (validated) channel set
    sg = host(got["sigma"])
    r = shape.ltp_rank
    tol = 2e-4 if fp32 else 1e-2                                      # bf16 factors carry 2^-9 per element
    for row, name, ukey, vkey in ((0, "g", "ug", "vg"), (1, "u", "uu", "vu"), (2, "d", "ud", "vd")):
        s_o = want["sigma"][name]
        assert np.abs(sg[row] - s_o).max() <= 2e-4 * s_o[0], name
        if name == "d":
            prod_g = host(got["ud"]) @ host(got["vd"])
            prod_o = want["ud"] @ want["vd"]
            Wp = np.asarray(W["w_down"], np.float64)[:, C]
        else:
            prod_g = host(got[ukey]).T @ host(got[vkey]).T
            prod_o = want[ukey].T @ want[vkey].T
            Wp = np.asarray(W["w_gate" if name == "g" else "w_up"], np.float64)[C].T
        assert np.linalg.norm(prod_g - prod_o) <= tol * np.linalg.norm(Wp), name
        if fp32:                                                      # Eckart-Young on the GPU's own factors
            err = np.linalg.norm(Wp - prod_g) ** 2
            assert abs(err - np.sum(s_o[r:] ** 2)) <= 1e-3 * np.sum(s_o ** 2), name
    lib.close()


def test_full_rank_proxy_built_on_gpu_reproduces_the_ffn_norm():
    """All channels kept and r = min(D, Dff): the proxy built by spts_proxy_build is the FFN itself, so the LTP
    transformation score C_n equals ||F_FFN(x_n)||_2 (Eq. 6 against Eq. 12-13)."""
    from paper_2601_13155_b200 import binding
    shape = replace(synth.TINY, ltp_dlow=synth.TINY.ffn_dim, ltp_rank=min(synth.TINY.hidden, synth.TINY.ffn_dim))
    lib, W, Wd, Xc, got = _case(shape, 64, 91, 0.2)
    assert got["channels"].cpu().numpy().tolist() == list(range(shape.ffn_dim))
    Wp = dict(W)
    for k in ("ug", "vg", "uu", "vu", "vd", "ud"):
        Wp[k] = host(got[k]).astype(np.float32)
    Wpd = binding.LayerWeights(Wp, shape.dtype)
    X, _ = synth.hidden_states(shape, 97, 5, heavy=4)
    Xd = up(X, shape.dtype)
    S = torch.full((97,), 1.0 / 97, dtype=torch.float32, device=dev())
    Cd = torch.empty(97, dtype=torch.float32, device=dev())
    lib.ltp_score(Wpd, Xd, S, C_out=Cd)
    B = O.rmsnorm(X, np.ones(shape.hidden), shape.rms_eps)
    want = np.linalg.norm(O.ffn(B, W["w_gate"].astype(np.float64), W["w_up"].astype(np.float64),
                                W["w_down"].astype(np.float64)), axis=1)
    assert np.abs(host(Cd) - want).max() <= 2e-3 * want.max()
    assert lib.device_status() == 0
    lib.close()
