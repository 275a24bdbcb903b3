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


class Guarded:
    """A device buffer with a band of a known pattern on either side, standing in for a memory checker: a kernel that
    writes just outside a caller's output buffer spoils a band, and `intact()` sees it."""
    BAND = 1024

    def __init__(self, shape, dtype):
        self.n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((self.n + 2 * self.BAND,), 0xA5, dtype=torch.uint8, device=dev())
        self.t = self.raw[self.BAND:self.BAND + self.n].view(dtype).view(*shape)

    def intact(self):
        b = self.BAND
        return bool((self.raw[:b] == 0xA5).all().item()) and bool((self.raw[b + self.n:] == 0xA5).all().item())


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


def index_set_report(got_idx, oracle_scores, k, force_last=True, band=1e-3):
    """Measures, without asserting, how a selected set differs from the oracle's: `diff` = tokens of the oracle's set
    that are missing (= tokens selected instead), `outside_band` = how many of the differing tokens (both sides) have
    an oracle score farther than `band` (relative) from the k-th score, `max_rel_dist` = the farthest of them."""
    got = np.asarray(got_idx, np.int64)
    assert got.shape[0] == k and np.all(np.diff(got) > 0)
    s = np.asarray(oracle_scores, np.float64)
    want = O.topk_select(s, k, force_last)
    body = want[want != len(s) - 1] if force_last and k > 1 else want
    kth = np.sort(s[body])[0]
    diff = np.setxor1d(got, want)
    dist = np.abs(s[diff] - kth) / abs(kth) if len(diff) else np.zeros(0)
    return {"diff": len(diff) // 2, "outside_band": int((dist > band).sum()),
            "max_rel_dist": float(dist.max()) if len(diff) else 0.0}


TOL = {"bf16": 2e-2, "fp32": 1e-4}


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x| (8 significant bits)."""
    x = np.abs(np.asarray(x, np.float64))
    e = np.floor(np.log2(np.maximum(x, 2.0 ** -126)))
    return 2.0 ** (e - 7)


class OutputStats(dict):
    """What check_output measured: max_rel (largest error outside the tolerated one-ulp cases, relative to the RMS),
    worst_rel (largest error of all), flips (elements beyond the tolerance that are exactly a one-ulp disagreement),
    flip_rows (the rows they sit in, at most 16 listed), elements."""


REPORT = []          # one entry per check_output call of the running test; printed by the conftest hook


def check_output(got, want, dtype, scale=1.0, what="output", ulps=1, per_row=False, ref_mag=None):
    """Layer outputs: max-abs error <= tol * RMS(want).  In bf16 storage a single element whose
    fp32-accumulated value and fp64 value fall on different sides of a rounding boundary differs by
    one bf16 ulp, which for the large entries of heavy rows exceeds tol * RMS on its own; such
    elements are allowed one ulp and must be rare (< 0.1 % of the elements).  `ulps` = 2 is for comparisons that span
    two storage roundings of the same element with nothing forced in between (the residual after the attention block
    and again after the FFN block): each rounding can fall on the other side once; `ref_mag` (same shape) then gives a
    magnitude the element had on the way (its input value), so that the ulp is taken at the largest binade it passed
    through.  `per_row`: the tolerance is relative to each row's own RMS instead of the RMS of the whole output (rows
    of an attention output are independent averages whose sizes differ by orders of magnitude).  Returns OutputStats (the number and
    the rows of the tolerated one-ulp cases among them) and appends them to REPORT, which every GPU test prints."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    tol = TOL[dtype] * scale
    if per_row:
        rms = np.maximum(np.sqrt(np.mean(want ** 2, axis=-1, keepdims=True)), 1e-30)
    else:
        rms = max(np.sqrt(np.mean(want ** 2)), 1e-30)
    err = np.abs(got - want)
    over = err > tol * rms
    mag = np.maximum(np.abs(want), np.abs(got)) if ulps > 1 else np.abs(want)
    if ref_mag is not None:
        mag = np.maximum(mag, np.abs(np.asarray(ref_mag, np.float64)))
    rel = err / rms
    stats = OutputStats(what=what, elements=int(want.size), tol=tol, worst_rel=float(rel.max()) if err.size else 0.0,
                        flips=0, flip_rows=[], max_rel=0.0)
    if dtype == "fp32":
        assert not over.any(), f"max-abs error {rel.max():.3e} of RMS exceeds {tol:.1e}"
        stats["max_rel"] = stats["worst_rel"]
        REPORT.append(stats)
        return stats
    flips = over & (err <= 1.001 * ulps * bf16_ulp(mag))
    bad = over & ~flips
    assert not bad.any(), f"max-abs error {rel[bad].max():.3e} of RMS exceeds {tol:.1e} (beyond {ulps} bf16 ulp)"
    assert flips.sum() <= max(1, 1e-3 * want.size), f"{int(flips.sum())} one-ulp disagreements"
    stats["flips"] = int(flips.sum())
    stats["flips_beyond_one_ulp"] = int((flips & (err > 1.001 * bf16_ulp(want))).sum())
    rel = np.where(over, 0.0, rel)
    if stats["flips"]:
        rows = np.unique(np.nonzero(flips)[0]) if flips.ndim > 1 else np.nonzero(flips)[0]
        stats["flip_rows"] = [int(r) for r in rows[:16]]
        stats["n_flip_rows"] = int(len(rows))
    stats["max_rel"] = float(rel.max()) if rel.size else 0.0
    REPORT.append(stats)
    return stats


def zero_down(W):
    """Same layer with W_down = 0: the FFN block becomes a no-op, exposing the residual after attention."""
    Wz = dict(W)
    Wz["w_down"] = np.zeros_like(W["w_down"])
    return Wz


def check_layer_blocks(lib, shape, W, lw, lw_mid, Xd, pos_t, ma, mf, cache, layer=0):
    """Runs spts_layer_prefill_skip on Xd (in place) and checks it against the oracle block by block.

    The attention block is compared on the layer's input.  The FFN block's decision (T_f) and
    update are compared on the GPU's own post-attention residual (obtained by a second run with
    W_down = 0), because a single one-ulp bf16 disagreement in that residual moves the LTP score of
    its token by more than the 1e-3 band.  Returns the outputs of the real run."""
    import torch
    from paper_2601_13155_b200 import binding
    dtype = shape.dtype
    mode = "bf16" if dtype == "bf16" else "exact"
    n = Xd.shape[0]
    x_in, pos_in = host(Xd), pos_t.cpu().numpy()
    X0 = Xd.clone()
    # GPU: attention block only
    Xmid = Xd.clone()
    scratch = binding.KvCache(shape, 1, n)
    lib.layer_prefill_skip(lw_mid, Xmid, pos_t, ma, n, scratch)
    # GPU: the real layer
    gS, gia, gjf = Guarded((n,), torch.float32), Guarded((ma,), torch.int32), Guarded((mf,), torch.int32)
    S, ia, jf = gS.t, gia.t, gjf.t
    lib.set_debug_checks(True)           # index lists checked on the device as well (range, strictly ascending)
    lib.layer_prefill_skip(lw, Xd, pos_t, ma, mf, cache, layer=layer, S_out=S, idx_attn_out=ia, idx_ffn_out=jf)
    lib.set_debug_checks(False)
    assert lib.device_status() == 0
    assert gS.intact() and gia.intact() and gjf.intact(), "a kernel wrote outside a caller's output buffer"
    assert lib.check_guards() == 0, "a kernel wrote past the end of its workspace slice"
    ia_h, jf_h = ia.cpu().numpy(), jf.cpu().numpy()
    # oracle: attention block from the layer input
    wa = O.layer_prefill_skip(x_in, pos_in, zero_down(W), shape, ma, n, mode=mode)
    assert np.abs(host(S) - wa["S_mha"]).max() <= 2e-4 * wa["S_mha"].max()
    swaps_a = check_index_set(ia_h, wa["S_mha"], ma)
    same = np.setdiff1d(np.arange(n), np.setxor1d(ia_h, wa["idx_attn"]))
    check_output(host(Xmid)[same], wa["X"][same], dtype)
    assert cache.length(layer) == ma
    assert np.array_equal(cache.pos[layer][:ma].cpu().numpy(), pos_in[ia_h])
    if swaps_a == 0:
        check_output(host(cache.k[layer][:ma]), wa["K"], dtype)
        check_output(host(cache.v[layer][:ma]), wa["V"], dtype)
    # oracle: FFN block from the GPU's post-attention residual and the oracle's S_mha
    rnd = O.rounding(mode)
    W64 = {k: np.asarray(v, np.float64) for k, v in W.items()}
    xm = host(Xmid)
    B = O.rmsnorm(xm, np.ones(shape.hidden), shape.rms_eps)
    Cw, Sf = O.ltp_score(B, wa["S_mha"], W64, rnd)
    swaps_f = check_index_set(jf_h, Sf, mf)
    Tf = O.topk_select(Sf, mf, True)
    xo = xm.copy()
    xo[Tf] = rnd(xo[Tf] + O.ffn(B[Tf], W64["w_gate"], W64["w_up"], W64["w_down"], rnd))
    samef = np.setdiff1d(np.arange(n), np.setxor1d(jf_h, Tf))
    check_output(host(Xd)[samef], xo[samef], dtype)
    # Eq. 2: rows outside both sets are bit-identical to the input
    rest = np.setdiff1d(np.arange(n), np.union1d(ia_h, jf_h))
    if len(rest):
        r = torch.from_numpy(rest).to(dev())
        assert torch.equal(Xd[r], X0[r])
    return {"S": S, "idx_attn": ia, "idx_ffn": jf, "swaps": swaps_a + swaps_f}
