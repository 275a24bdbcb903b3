"""Helpers shared by the GPU parity tests: upload inputs, compare with the oracle."""
import numpy as np
import torch

from oracle import spts_oracle as O


def dev():
    return torch.device("cuda:0")


def up(a, dtype):
    from paper_2601_13155_b200 import binding
    return binding.to_device(a, dtype)


def i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev())


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_rms_err(got, want):
    """max-abs error relative to the RMS of the expected output."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    rms = np.sqrt(np.mean(want ** 2))
    return float(np.abs(got - want).max() / max(rms, 1e-30))


def check_index_set(got_idx, oracle_scores, k, force_last=True, band=1e-3):
    """Selected sets must match the oracle's exactly, except for tokens whose oracle score lies
    within `band` (relative) of the k-th largest score.  Returns the number of boundary swaps."""
    got = np.asarray(got_idx, np.int64)
    assert got.shape[0] == k
    assert np.all(np.diff(got) > 0), "indices must be strictly ascending"
    want = O.topk_select(oracle_scores, k, force_last)
    if np.array_equal(got, want):
        return 0
    s = np.asarray(oracle_scores, np.float64)
    kth = np.sort(s[want])[0] if not force_last else np.sort(s[want[want != len(s) - 1]])[0] if k > 1 else s[-1]
    diff = np.setxor1d(got, want)
    bad = [int(i) for i in diff if abs(s[i] - kth) > band * abs(kth)]
    assert not bad, f"{len(bad)} selected indices differ outside the boundary band: {bad[:8]}"
    return len(diff) // 2


TOL = {"bf16": 2e-2, "fp32": 1e-4}


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x| (8 significant bits)."""
    x = np.abs(np.asarray(x, np.float64))
    e = np.floor(np.log2(np.maximum(x, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def check_output(got, want, dtype, scale=1.0):
    """Layer outputs: max-abs error <= tol * RMS(want).  In bf16 storage a single element whose
    fp32-accumulated value and fp64 value fall on different sides of a rounding boundary differs by
    one bf16 ulp, which for the large entries of heavy rows exceeds tol * RMS on its own; such
    elements are allowed one ulp and must be rare (< 0.1 % of the elements)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    tol = TOL[dtype] * scale
    rms = max(np.sqrt(np.mean(want ** 2)), 1e-30)
    err = np.abs(got - want)
    over = err > tol * rms
    if dtype == "fp32":
        assert not over.any(), f"max-abs error {err.max() / rms:.3e} of RMS exceeds {tol:.1e}"
        return float(err.max() / rms)
    flips = over & (err <= 1.001 * bf16_ulp(want))
    bad = over & ~flips
    assert not bad.any(), f"max-abs error {err[bad].max() / rms:.3e} of RMS exceeds {tol:.1e} (beyond one bf16 ulp)"
    assert flips.sum() <= max(1, 1e-3 * want.size), f"{int(flips.sum())} one-ulp disagreements"
    return float(err[~over].max() / rms) if (~over).any() else 0.0
