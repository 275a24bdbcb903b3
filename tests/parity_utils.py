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
