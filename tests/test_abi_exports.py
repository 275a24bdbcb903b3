"""The C-ABI library builds, loads without a GPU and exports every symbol include/spts.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2601_13155_b200 import build
    return build.build()


def _declared():
    src = open(os.path.join(ROOT, "include", "spts.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(spts_[a-z0-9_]+)\s*\(", src)))


def test_exports_match_header(lib_path):
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert {"spts_pap_score", "spts_ltp_score", "spts_topk_select", "spts_layer_prefill_skip",
            "spts_msdp_compact", "spts_decode_step"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2601_13155_b200 import binding
    assert set(binding.EXPORTS) == set(names)
    binding.load_library()


def test_workspace_bytes_is_host_arithmetic(lib_path):
    from paper_2601_13155_b200 import binding, synth
    lib = binding.load_library()
    s = synth.LLAMA8B
    d = binding.ModelDesc(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn_dim, s.ltp_dlow, s.ltp_rank,
                          s.n_layers, s.vocab, s.rms_eps, s.rope_theta, 0)
    small = lib.spts_workspace_bytes(ctypes.byref(d), 8192)
    big = lib.spts_workspace_bytes(ctypes.byref(d), 131072)
    assert 0 < small < big < 40 * 2 ** 30
    d.head_dim = 96                      # unsupported shape -> 0
    assert lib.spts_workspace_bytes(ctypes.byref(d), 8192) == 0
    assert lib.spts_workspace_bytes(None, 8192) == 0


def test_host_argument_checks_need_no_gpu(lib_path):
    from paper_2601_13155_b200 import binding
    lib = binding.load_library()
    assert lib.spts_topk_select(None, None, 4, 2, 0, None) == 1        # SPTS_ERR_INVALID_ARG
    assert lib.spts_launch_count(None) == 0
    # a call without a context is refused before anything is touched
    assert lib.spts_layer_prefill_skip_batch(None, None, None, None, 2, None, None, None, 0, None, None, None, None) == 1
    assert lib.spts_set_option(None, 16, 1) == 1
    assert lib.spts_reduced_attention(None, None, None, None, 4, None) == 1
    assert lib.spts_prepare_layer(None, None, None, 0) == 1
    assert lib.spts_check_guards(None, None) == 1
    assert lib.spts_selftest_wait_timeout(None, 1000) == 1
    assert lib.spts_debug_check_index_list(None, None, 4, 8) == 1
    assert lib.spts_prepared_bytes(None) == 0


def test_workspace_at_the_longest_context_stays_below_four_gigabytes(lib_path):
    """The SwiGLU intermediate is held for one chunk of 16384 rows, not per candidate: 131072 candidates of the 8B shape
    need less than 4 GB of workspace, and the prepared proxy factors of a layer a few MB."""
    from paper_2601_13155_b200 import binding, synth
    lib = binding.load_library()
    s = synth.LLAMA8B
    d = binding.ModelDesc(s.hidden, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn_dim, s.ltp_dlow, s.ltp_rank,
                          s.n_layers, s.vocab, s.rms_eps, s.rope_theta, 0)
    assert lib.spts_workspace_bytes(ctypes.byref(d), 131072) < 4 * 10 ** 9
    assert lib.spts_workspace_bytes(ctypes.byref(d), 32768) < 1.5 * 10 ** 9
    assert 2 * 2 ** 20 < lib.spts_prepared_bytes(ctypes.byref(d)) < 4 * 2 ** 20


def test_traffic_records_are_dropped_when_the_kernel_source_changes(tmp_path, monkeypatch):
    """bench.py reports a captured DRAM-traffic figure only while the SHA-256 of the kernel's source files equals the
    one stored with the capture."""
    import json
    from paper_2601_13155_b200 import ncu_summary
    rec = {"workload": "cfg3", "op": "attention", "dram_bytes_per_launch": 1.0, "source_sha256": ncu_summary.source_digest("attention")}
    f = tmp_path / "traffic.json"
    f.write_text(json.dumps({"records": [rec]}))
    monkeypatch.setattr(ncu_summary, "TRAFFIC_JSON", str(f))
    assert ncu_summary.traffic_for("cfg3", "attention")["dram_bytes_per_launch"] == 1.0
    assert ncu_summary.traffic_for("cfg4", "attention") is None and ncu_summary.traffic_for("cfg3", "topk") is None
    rec["source_sha256"] = "0" * 64
    f.write_text(json.dumps({"records": [rec]}))
    assert ncu_summary.traffic_for("cfg3", "attention") is None


def test_product_schedule_matches_budget_rule():
    from paper_2601_13155_b200 import schedule, synth
    w = synth.workload("cfg3")
    plan = schedule.workload_plan(w)
    assert [plan[l] for l in (0, 7, 8, 23, 24, 31)] == [
        (16384, 13108, 0), (16384, 13108, 24576), (16384, 13108, 0), (16384, 13108, 11469),
        (11469, 11469, 0), (11469, 11469, 0)]
    w4 = synth.workload("cfg4")
    p4 = schedule.workload_plan(w4)
    assert p4[0] == (65536, 52429, 0) and p4[31] == (45875, 45875, 0)
    # agrees with the oracle's independent statement of the rule
    from oracle import spts_oracle as O
    import math
    op = O.msdp_schedule(32, w.n_tokens, w.stage_first_layer, w.stage_tokens,
                         math.ceil(w.keep_attn * w.n_tokens), math.ceil(w.keep_ffn * w.n_tokens))
    assert [(p["m_attn"], p["m_ffn"], p["prune_to"] or 0) for p in op] == plan


def test_paper_llama_plan_matches_oracle_and_table3():
    """The product's statement of the paper's LLaMA schedule agrees with the oracle's independent one and
    reproduces the KV-cache sizes the paper prints (Table 3: 2.81 / 4.13 / 5.38 / 6.63 with PAP against
    4 / 8 / 12 / 16 without, i.e. savings of 29.7 / 48.4 / 55.2 / 58.6 %)."""
    from paper_2601_13155_b200 import schedule
    from oracle import spts_oracle as O
    printed = {8192: (2.81, 29.7), 16384: (4.13, 48.4), 24576: (5.38, 55.2), 32768: (6.63, 58.6)}
    for n, (size, saving) in printed.items():
        plan = schedule.paper_llama_plan(n)
        cur, want = n, []
        for q in O.paper_llama_schedule(n):
            pr = q["prune_to"] if q["prune_to"] is not None and q["prune_to"] < cur else 0
            want.append((q["m_attn"], q["m_ffn"], pr))
            cur = pr or cur
        assert plan == want
        kv = schedule.kv_token_layers(plan)
        assert f"{kv / 1024 / 64 + 1e-9:.2f}" == f"{size:.2f}"
        assert abs(100 * (1 - kv / (32 * n)) - saving) < 0.06
    # ablation switches: FFN dense without LTP; no pruning without MSDP
    p = schedule.paper_llama_plan(32768, ltp=False)
    assert p[20] == (4096, 6144, 0)                                  # 6144 candidates left after two prunes
    p = schedule.paper_llama_plan(32768, msdp=False)
    assert all(c == 0 for _, _, c in p) and p[31] == (2048, 2048, 0) and p[12] == (9216, 9216, 0)


def test_msdp_plan_call_counts_and_errors():
    """spts_msdp_plan through the C boundary: the optional outputs (final candidate count, cached token-layer pairs:
    the paper's LLaMA setting at 32 Ki tokens gives the 6.63 of Table 3 in units of 64 Ki pairs) and the host
    errors (null pointers, empty inputs, stages out of order)."""
    import ctypes as C
    from paper_2601_13155_b200 import binding
    lib = binding.load_library()
    Ki = 1024
    st = (binding.MsdpStageC * 4)(*[binding.MsdpStageC(e, b * Ki, b * Ki, (b - 1) * Ki)
                                    for e, b in zip((13, 18, 23, 28), (9, 7, 4, 2))])
    out = (binding.LayerPlanC * 32)()
    nf, kv = C.c_int32(0), C.c_int64(0)
    assert lib.spts_msdp_plan(32, 32 * Ki, 10, st, 4, out, C.byref(nf), C.byref(kv)) == 0
    assert nf.value == 1 * Ki and f"{kv.value / Ki / 64 + 1e-9:.2f}" == "6.63"     # 6.625 exactly
    assert [(out[l].m_attn, out[l].m_ffn, out[l].prune_to) for l in (0, 9, 10, 13, 14, 28, 29, 31)] == [
        (32 * Ki, 32 * Ki, 0), (32 * Ki, 32 * Ki, 0), (9 * Ki, 9 * Ki, 0), (9 * Ki, 9 * Ki, 8 * Ki),
        (7 * Ki, 7 * Ki, 0), (2 * Ki, 2 * Ki, 1 * Ki), (1 * Ki, 1 * Ki, 0), (1 * Ki, 1 * Ki, 0)]
    # a prompt shorter than every budget: nothing is skipped, nothing is pruned
    assert lib.spts_msdp_plan(32, 700, 10, st, 4, out, C.byref(nf), None) == 0
    assert nf.value == 700 and all((out[l].m_attn, out[l].m_ffn, out[l].prune_to) == (700, 700, 0) for l in range(32))
    assert lib.spts_msdp_plan(32, 32 * Ki, 10, None, 4, out, None, None) == 1
    assert lib.spts_msdp_plan(32, 32 * Ki, 10, st, 4, None, None, None) == 1
    assert lib.spts_msdp_plan(0, 32 * Ki, 10, st, 4, out, None, None) == 1
    assert lib.spts_msdp_plan(32, 0, 10, st, 4, out, None, None) == 1
    assert lib.spts_msdp_plan(32, 32 * Ki, 10, st, 0, out, None, None) == 1
    bad = (binding.MsdpStageC * 2)(binding.MsdpStageC(5, 8, 8, 4), binding.MsdpStageC(5, 4, 4, 2))
    assert lib.spts_msdp_plan(8, 100, 0, bad, 2, out, None, None) == 1
