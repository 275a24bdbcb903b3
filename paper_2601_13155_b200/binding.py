"""ctypes binding of libspts.so (the C boundary declared in include/spts.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch is used for device memory and streams.  There is no CPU fallback: importing this
module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SPTS_LIBRARY") or os.path.join(_PKG, "libspts.so")     # SPTS_LIBRARY: another build of the library

SPTS_BF16, SPTS_FP32 = 0, 1
FORCE_LAST = 1
OPT_REFERENCE_KERNELS = 2
OPT_PAP_WINDOW = 8
OPT_FFN_SCORE_PAP_ONLY = 16
OPT_DEBUG_CHECKS = 32

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "WORKSPACE", 4: "CUDA", 5: "TIMEOUT",
                6: "NONFINITE", 7: "UNSUPPORTED", 8: "INDEX"}


class SptsError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: SPTS_ERR_{STATUS_NAMES.get(code, code)}")
        self.code = code


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn_dim",
                                          "ltp_dlow", "ltp_rank", "n_layers", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("dtype", C.c_int32)]


WEIGHT_NAMES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "ug", "vg", "uu", "vu", "vd", "ud")


class LayerWeightsC(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES] + [("prepared", C.c_void_p)]


class KvLayerC(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("pos", C.c_void_p), ("len", C.c_int32),
                ("capacity", C.c_int32)]


class LayerPlanC(C.Structure):
    _fields_ = [("m_attn", C.c_int32), ("m_ffn", C.c_int32), ("prune_to", C.c_int32)]


class MsdpStageC(C.Structure):
    _fields_ = [("last_layer", C.c_int32), ("m_attn_fixed", C.c_int32), ("m_ffn_fixed", C.c_int32),
                ("n_next", C.c_int32)]


class ModelWeightsC(C.Structure):
    _fields_ = [("layers", C.POINTER(LayerWeightsC)), ("lm_head", C.c_void_p), ("embed", C.c_void_p)]


EXPORTS = ("spts_workspace_bytes", "spts_create", "spts_destroy", "spts_set_option",
           "spts_last_device_status", "spts_launch_count", "spts_fold_norm_gain", "spts_pap_score",
           "spts_ltp_score", "spts_topk_select", "spts_layer_prefill_skip", "spts_msdp_compact",
           "spts_first_token", "spts_prefill", "spts_decode_step", "spts_profile_begin", "spts_profile_end",
           "spts_topk_select_static", "spts_proxy_scratch_bytes", "spts_proxy_build",
           "spts_layer_prefill_skip_batch", "spts_msdp_plan", "spts_check_guards", "spts_selftest_wait_timeout",
           "spts_debug_check_index_list", "spts_reduced_attention", "spts_prepared_bytes", "spts_prepare_layer")

OP_NAMES = {1: "prep", 2: "kproj_pap", 3: "pap_softmax", 4: "topk", 5: "kv_gather", 6: "qv_proj", 7: "attention",
            8: "o_proj", 9: "ltp", 10: "gate_up", 11: "down", 12: "compact", 13: "head", 14: "decode"}
OP_COUNT = 16


def load_library() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_13155_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, u32 = C.c_void_p, C.c_int, C.c_uint32
    lib.spts_workspace_bytes.restype = C.c_size_t
    lib.spts_workspace_bytes.argtypes = [C.POINTER(ModelDesc), i32]
    lib.spts_create.argtypes = [C.POINTER(ModelDesc), i32, vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.spts_destroy.argtypes = [vp]
    lib.spts_destroy.restype = None
    lib.spts_set_option.argtypes = [vp, u32, i32]
    lib.spts_last_device_status.argtypes = [vp]
    lib.spts_launch_count.argtypes = [vp]
    lib.spts_launch_count.restype = C.c_int64
    lib.spts_fold_norm_gain.argtypes = [vp, vp, vp, i32, i32]
    lib.spts_pap_score.argtypes = [vp, C.POINTER(LayerWeightsC), vp, vp, i32, vp, vp]
    lib.spts_ltp_score.argtypes = [vp, C.POINTER(LayerWeightsC), vp, vp, i32, vp, vp]
    lib.spts_topk_select.argtypes = [vp, vp, i32, i32, u32, vp]
    lib.spts_topk_select_static.argtypes = [vp, i32, i32, u32, vp, vp]
    lib.spts_proxy_scratch_bytes.restype = C.c_size_t
    lib.spts_proxy_scratch_bytes.argtypes = [C.POINTER(ModelDesc), i32]
    lib.spts_proxy_build.argtypes = [vp, C.POINTER(LayerWeightsC), vp, i32, C.c_double, vp, C.c_size_t, vp, vp,
                                     vp, vp, vp, vp, vp, vp, vp]
    lib.spts_layer_prefill_skip.argtypes = [vp, C.POINTER(LayerWeightsC), vp, vp, i32, i32, i32, u32,
                                            C.POINTER(KvLayerC), vp, vp, vp]
    lib.spts_layer_prefill_skip_batch.argtypes = [vp, C.POINTER(LayerWeightsC), vp, vp, i32, C.POINTER(C.c_int32),
                                                  C.POINTER(C.c_int32), C.POINTER(C.c_int32), u32,
                                                  C.POINTER(KvLayerC), vp, vp, vp]
    lib.spts_msdp_compact.argtypes = [vp, vp, vp, vp, vp, i32, i32, u32, vp, vp, vp, vp]
    lib.spts_msdp_plan.argtypes = [i32, i32, i32, C.POINTER(MsdpStageC), i32, C.POINTER(LayerPlanC),
                                   C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    lib.spts_check_guards.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.spts_selftest_wait_timeout.argtypes = [vp, u32]
    lib.spts_debug_check_index_list.argtypes = [vp, vp, i32, i32]
    lib.spts_reduced_attention.argtypes = [vp, vp, vp, vp, i32, vp]
    lib.spts_prepared_bytes.restype = C.c_size_t
    lib.spts_prepared_bytes.argtypes = [C.POINTER(ModelDesc)]
    lib.spts_prepare_layer.argtypes = [vp, C.POINTER(LayerWeightsC), vp, C.c_size_t]
    lib.spts_first_token.argtypes = [vp, vp, vp, vp, vp]
    lib.spts_prefill.argtypes = [vp, C.POINTER(ModelWeightsC), C.POINTER(LayerPlanC), vp, vp, vp, vp, vp, vp,
                                 i32, u32, C.POINTER(KvLayerC), C.POINTER(C.c_int32), C.POINTER(C.c_int32), vp]
    lib.spts_decode_step.argtypes = [vp, C.POINTER(ModelWeightsC), C.POINTER(KvLayerC), vp, C.c_int32,
                                     C.c_int32, vp, vp, vp]
    lib.spts_profile_begin.argtypes = [vp, i32]
    lib.spts_profile_end.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int64), C.POINTER(C.c_double),
                                     C.POINTER(C.c_double)]
    for n in EXPORTS:
        if n not in ("spts_workspace_bytes", "spts_destroy", "spts_launch_count", "spts_proxy_scratch_bytes",
                     "spts_prepared_bytes"):
            getattr(lib, n).restype = C.c_int
    return lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def torch_dtype(dtype: str):
    return torch.bfloat16 if dtype == "bf16" else torch.float32


def to_device(a: np.ndarray, dtype: str, device="cuda:0") -> torch.Tensor:
    """Uploads a float32 array (already rounded to the storage type) as a device tensor."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return t.to(torch_dtype(dtype)).contiguous()


TOPK_STATIC_MAX_N = 8388608
_static_lib = None


def topk_select_static(scores: torch.Tensor, k: int, flags: int = 0, idx_out: Optional[torch.Tensor] = None,
                       stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """spts_topk_select_static: top-k without a context or a workspace, for callers that cannot allocate
    device memory (the scratch is a fixed array inside the library).  The index buffer is the caller's:
    pass `idx_out` [k] int32 to keep this call itself free of allocations."""
    global _static_lib
    if _static_lib is None:
        _static_lib = load_library()
    N = scores.shape[0]
    if idx_out is None:
        idx_out = torch.empty(max(k, 1), dtype=torch.int32, device=scores.device)
    st = stream if stream is not None else torch.cuda.current_stream(scores.device)
    with torch.cuda.device(scores.device):
        code = _static_lib.spts_topk_select_static(_ptr(scores), N, k, flags, _ptr(idx_out), C.c_void_p(st.cuda_stream))
    if code != 0:
        raise SptsError(code, "spts_topk_select_static")
    return idx_out


class LayerWeights:
    """Device copies of one layer's matrices plus the C struct that points at them."""

    def __init__(self, arrays: Dict[str, np.ndarray], dtype: str, device="cuda:0"):
        self.t = {n: to_device(arrays[n], dtype, device) for n in WEIGHT_NAMES}
        self.c = LayerWeightsC(**{n: self.t[n].data_ptr() for n in WEIGHT_NAMES})
        self.prepared = None

    @classmethod
    def from_tensors(cls, tensors: Dict[str, torch.Tensor]) -> "LayerWeights":
        """Wraps device tensors that already hold the matrices in the storage type (no copy)."""
        w = cls.__new__(cls)
        w.t = tensors
        w.c = LayerWeightsC(**{n: tensors[n].data_ptr() for n in WEIGHT_NAMES})
        w.prepared = None
        return w


class KvCache:
    """Per-layer caches [capacity, Hkv, d] (K after RoPE), original positions and lengths."""

    def __init__(self, shape, n_layers: int, capacity, device="cuda:0"):
        caps = list(capacity) if hasattr(capacity, "__len__") else [capacity] * n_layers
        dt = torch_dtype(shape.dtype)
        self.k = [torch.zeros(c, shape.n_kv_heads, shape.head_dim, dtype=dt, device=device) for c in caps]
        self.v = [torch.zeros(c, shape.n_kv_heads, shape.head_dim, dtype=dt, device=device) for c in caps]
        self.pos = [torch.zeros(c, dtype=torch.int32, device=device) for c in caps]
        self.c = (KvLayerC * n_layers)()
        for l in range(n_layers):
            self.c[l] = KvLayerC(self.k[l].data_ptr(), self.v[l].data_ptr(), self.pos[l].data_ptr(), 0, caps[l])

    def length(self, l: int) -> int:
        return int(self.c[l].len)

    def reset(self):
        for e in self.c:
            e.len = 0


class Spts:
    """One library context bound to a device and a stream."""

    def __init__(self, shape, max_seq: int, device="cuda:0", stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("the SPTS library needs a CUDA device (no CPU fallback)")
        self.lib = load_library()
        self.shape = shape
        self.device = torch.device(device)
        self.dtype = torch_dtype(shape.dtype)
        self.desc = ModelDesc(shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn_dim,
                              shape.ltp_dlow, shape.ltp_rank, shape.n_layers, shape.vocab, shape.rms_eps,
                              shape.rope_theta, SPTS_BF16 if shape.dtype == "bf16" else SPTS_FP32)
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        nbytes = self.lib.spts_workspace_bytes(C.byref(self.desc), max_seq)
        if nbytes == 0:
            raise SptsError(2, "spts_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.max_seq = max_seq
        h = C.c_void_p()
        self._check(self.lib.spts_create(C.byref(self.desc), max_seq, _ptr(self.workspace), nbytes,
                                         C.c_void_p(self.stream.cuda_stream), C.byref(h)), "spts_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.spts_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, code: int, where: str):
        if code != 0:
            raise SptsError(code, where)

    # ------------------------------------------------------------------ options / status
    def set_reference_kernels(self, on: bool):
        self._check(self.lib.spts_set_option(self.h, OPT_REFERENCE_KERNELS, 1 if on else 0), "spts_set_option")

    def set_pap_window(self, window: int):
        self._check(self.lib.spts_set_option(self.h, OPT_PAP_WINDOW, int(window)), "spts_set_option")

    def set_ffn_score_pap_only(self, on: bool):
        """T_f = TopK(S_mha, m_ffn): the FFN criterion without the proxy network (Table 4's baseline row)."""
        self._check(self.lib.spts_set_option(self.h, OPT_FFN_SCORE_PAP_ONLY, 1 if on else 0), "spts_set_option")

    def set_debug_checks(self, on: bool):
        """Every selected index list is checked on the device (range, strictly ascending); SPTS_ERR_INDEX otherwise."""
        self._check(self.lib.spts_set_option(self.h, OPT_DEBUG_CHECKS, 1 if on else 0), "spts_set_option")

    def check_guards(self) -> int:
        """Number of guard bands between the workspace slices that no longer hold their pattern (0 = intact)."""
        n = C.c_int32(-1)
        self._check(self.lib.spts_check_guards(self.h, C.byref(n)), "spts_check_guards")
        return int(n.value)

    def debug_check_index_list(self, idx, N: int):
        self._check(self.lib.spts_debug_check_index_list(self.h, _ptr(idx), idx.shape[0], N), "spts_debug_check_index_list")

    def selftest_wait_timeout(self, limit_us: int = 1000):
        self._check(self.lib.spts_selftest_wait_timeout(self.h, int(limit_us)), "spts_selftest_wait_timeout")

    def device_status(self) -> int:
        return int(self.lib.spts_last_device_status(self.h))

    def launch_count(self) -> int:
        return int(self.lib.spts_launch_count(self.h))

    def fold_norm_gain(self, W: torch.Tensor, g: torch.Tensor):
        self._check(self.lib.spts_fold_norm_gain(self.h, _ptr(W), _ptr(g), W.shape[0], W.shape[1]),
                    "spts_fold_norm_gain")

    def profile_begin(self, op: int = -1):
        self._check(self.lib.spts_profile_begin(self.h, op), "spts_profile_begin")

    def profile_end(self):
        """Returns {op name: {"ms", "calls", "flops", "bytes"}} for the operations timed since profile_begin."""
        ms = (C.c_float * OP_COUNT)()
        calls = (C.c_int64 * OP_COUNT)()
        fl = (C.c_double * OP_COUNT)()
        by = (C.c_double * OP_COUNT)()
        self._check(self.lib.spts_profile_end(self.h, ms, calls, fl, by), "spts_profile_end")
        return {OP_NAMES[i]: {"ms": float(ms[i]), "calls": int(calls[i]), "flops": float(fl[i]), "bytes": float(by[i])}
                for i in OP_NAMES if calls[i] > 0}

    # ------------------------------------------------------------------ the six calls
    def pap_score(self, w: LayerWeights, X, pos, K_out=None, S_out=None):
        N = X.shape[0]
        if S_out is None:
            S_out = torch.empty(N, dtype=torch.float32, device=self.device)
        self._check(self.lib.spts_pap_score(self.h, C.byref(w.c), _ptr(X), _ptr(pos), N, _ptr(K_out), _ptr(S_out)),
                    "spts_pap_score")
        return S_out

    def ltp_score(self, w: LayerWeights, X, S_mha, C_out=None, S_out=None):
        N = X.shape[0]
        if S_out is None:
            S_out = torch.empty(N, dtype=torch.float32, device=self.device)
        self._check(self.lib.spts_ltp_score(self.h, C.byref(w.c), _ptr(X), _ptr(S_mha), N, _ptr(C_out), _ptr(S_out)),
                    "spts_ltp_score")
        return S_out

    def topk_select(self, scores, k: int, flags: int = 0, idx_out=None):
        N = scores.shape[0]
        if idx_out is None:
            idx_out = torch.empty(max(k, 1), dtype=torch.int32, device=self.device)
        self._check(self.lib.spts_topk_select(self.h, _ptr(scores), N, k, flags, _ptr(idx_out)), "spts_topk_select")
        return idx_out

    def layer_prefill_skip(self, w: LayerWeights, X, pos, m_attn: int, m_ffn: int, cache: KvCache, layer: int = 0,
                           flags: int = FORCE_LAST, S_out=None, idx_attn_out=None, idx_ffn_out=None):
        N = X.shape[0]
        self._check(self.lib.spts_layer_prefill_skip(self.h, C.byref(w.c), _ptr(X), _ptr(pos), N, m_attn, m_ffn,
                                                     flags, C.byref(cache.c[layer]), _ptr(S_out),
                                                     _ptr(idx_attn_out), _ptr(idx_ffn_out)),
                    "spts_layer_prefill_skip")

    def prepare_layer(self, w: "LayerWeights"):
        """spts_prepare_layer: repacks the layer's proxy factors once into a buffer the weights object then owns;
        later calls with `w` skip the per-call repacking.  Redo after changing ug / uu / vg / vu / ud."""
        nbytes = self.lib.spts_prepared_bytes(C.byref(self.desc))
        buf = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        w.c.prepared = None
        self._check(self.lib.spts_prepare_layer(self.h, C.byref(w.c), _ptr(buf), nbytes), "spts_prepare_layer")
        w.prepared = buf
        w.c.prepared = buf.data_ptr()
        return w

    def reduced_attention(self, Q, K, V, O_out=None):
        """spts_reduced_attention: causal GQA attention among the m rows of Q [m,H,d], K, V [m,Hkv,d] -> [m, H*d]."""
        m = Q.shape[0]
        if O_out is None:
            O_out = torch.empty(m, self.shape.n_q_heads * self.shape.head_dim, dtype=self.dtype, device=self.device)
        self._check(self.lib.spts_reduced_attention(self.h, _ptr(Q), _ptr(K), _ptr(V), m, _ptr(O_out)),
                    "spts_reduced_attention")
        return O_out

    def layer_prefill_skip_batch(self, w: LayerWeights, X, pos, seq_start, m_attn, m_ffn, caches: KvCache,
                                 flags: int = FORCE_LAST, S_out=None, idx_attn_out=None, idx_ffn_out=None):
        """Several prompts packed into X; `caches` holds one entry per sequence (a KvCache built with
        n_layers = number of sequences); seq_start, m_attn, m_ffn are host integer lists."""
        n_seq = len(m_attn)
        arr = lambda v: (C.c_int32 * len(v))(*[int(x) for x in v])
        self._check(self.lib.spts_layer_prefill_skip_batch(self.h, C.byref(w.c), _ptr(X), _ptr(pos), n_seq,
                                                           arr(seq_start), arr(m_attn), arr(m_ffn), flags, caches.c,
                                                           _ptr(S_out), _ptr(idx_attn_out), _ptr(idx_ffn_out)),
                    "spts_layer_prefill_skip_batch")

    def msdp_compact(self, X_in, pos_in, orig_in, S_mha, n_next: int, X_out, pos_out, orig_out, idx_out=None,
                     flags: int = FORCE_LAST):
        N = X_in.shape[0]
        self._check(self.lib.spts_msdp_compact(self.h, _ptr(X_in), _ptr(pos_in), _ptr(orig_in), _ptr(S_mha), N,
                                               n_next, flags, _ptr(X_out), _ptr(pos_out), _ptr(orig_out),
                                               _ptr(idx_out)), "spts_msdp_compact")

    def proxy_build(self, w: LayerWeights, calib, rho: float = 0.2, want_sigma: bool = False):
        """spts_proxy_build: returns {"importance", "channels", "ug", "vg", "uu", "vu", "vd", "ud"[, "sigma"]} as
        device tensors (the factors in the storage type and the layouts LayerWeights uses)."""
        s = self.shape
        n_cal = calib.shape[0]
        nbytes = self.lib.spts_proxy_scratch_bytes(C.byref(self.desc), n_cal)
        if nbytes == 0:
            raise SptsError(2, "spts_proxy_scratch_bytes")
        scratch = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        dt, dv = self.dtype, self.device
        out = {"importance": torch.empty(s.ffn_dim, dtype=torch.float32, device=dv),
               "channels": torch.empty(s.ltp_dlow, dtype=torch.int32, device=dv),
               "ug": torch.empty(s.ltp_rank, s.hidden, dtype=dt, device=dv),
               "vg": torch.empty(s.ltp_dlow, s.ltp_rank, dtype=dt, device=dv),
               "uu": torch.empty(s.ltp_rank, s.hidden, dtype=dt, device=dv),
               "vu": torch.empty(s.ltp_dlow, s.ltp_rank, dtype=dt, device=dv),
               "vd": torch.empty(s.ltp_rank, s.ltp_dlow, dtype=dt, device=dv),
               "ud": torch.empty(s.hidden, s.ltp_rank, dtype=dt, device=dv)}
        if want_sigma:
            out["sigma"] = torch.empty(3, s.ltp_dlow, dtype=torch.float32, device=dv)
        self._check(self.lib.spts_proxy_build(self.h, C.byref(w.c), _ptr(calib), n_cal, float(rho), _ptr(scratch), nbytes,
                                              _ptr(out["importance"]), _ptr(out["channels"]), _ptr(out["ug"]),
                                              _ptr(out["vg"]), _ptr(out["uu"]), _ptr(out["vu"]), _ptr(out["vd"]),
                                              _ptr(out["ud"]), _ptr(out.get("sigma"))), "spts_proxy_build")
        self.stream.synchronize()                                  # scratch is released on return
        return out

    def first_token(self, x_row, lm_head, logits_out=None, token_out=None):
        self._check(self.lib.spts_first_token(self.h, _ptr(x_row), _ptr(lm_head), _ptr(logits_out), _ptr(token_out)),
                    "spts_first_token")

    def prefill(self, model: "Model", plan: Sequence[Sequence[int]], X, pos, orig, X_alt, pos_alt, orig_alt,
                cache: KvCache, token_out=None, flags: int = FORCE_LAST, n_tokens: Optional[int] = None):
        """Algorithm 1 over all layers.  Returns (n_final, result_is_in_alt)."""
        L = self.shape.n_layers
        cplan = (LayerPlanC * L)(*[LayerPlanC(int(a), int(b), int(c or 0)) for a, b, c in plan])
        nf, ia = C.c_int32(0), C.c_int32(0)
        N = X.shape[0] if n_tokens is None else n_tokens
        self._check(self.lib.spts_prefill(self.h, C.byref(model.c), cplan, _ptr(X), _ptr(pos), _ptr(orig),
                                          _ptr(X_alt), _ptr(pos_alt), _ptr(orig_alt), N, flags, cache.c,
                                          C.byref(nf), C.byref(ia), _ptr(token_out)), "spts_prefill")
        return nf.value, bool(ia.value)

    def decode_step(self, model: "Model", cache: KvCache, pos: int, x_in=None, token_in: int = 0, x_out=None,
                    logits_out=None, token_out=None):
        self._check(self.lib.spts_decode_step(self.h, C.byref(model.c), cache.c, _ptr(x_in), token_in, pos,
                                              _ptr(x_out), _ptr(logits_out), _ptr(token_out)), "spts_decode_step")


class Model:
    """All layers' weights plus the LM head / embedding table."""

    def __init__(self, layers: List[LayerWeights], lm_head: Optional[torch.Tensor] = None,
                 embed: Optional[torch.Tensor] = None):
        self.layers = layers
        self.lm_head, self.embed = lm_head, embed
        self._arr = (LayerWeightsC * len(layers))(*[l.c for l in layers])
        self.c = ModelWeightsC(self._arr, lm_head.data_ptr() if lm_head is not None else None,
                               embed.data_ptr() if embed is not None else None)
