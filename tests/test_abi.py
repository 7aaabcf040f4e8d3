"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every symbol gm.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "gm.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(gm_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_entry_point():
    from paper_2609_16648_b200.build import build
    import paper_2609_16648_b200 as gmb
    path = build()
    L = ctypes.CDLL(path)
    names = _declared()
    assert {"gm_init", "gm_draft", "gm_verify", "gm_accept", "gm_spec_step"} <= set(names)
    for n in names:
        assert hasattr(L, n), n
    assert sorted(gmb.EXPORTS) == names


def test_error_strings_and_null_handling_need_no_gpu():
    import paper_2609_16648_b200 as gmb
    L = gmb.lib()
    assert gmb.gm_strerror(0) == "ok"
    for code in range(-9, 0):
        assert gmb.gm_strerror(code) not in ("ok", "unknown error")
    assert L.gm_last_status(None) == gmb.GM_ERR_INVALID_ARG
    assert L.gm_launch_count(None) == 0
    out = ctypes.c_void_p()
    assert L.gm_init(ctypes.byref(out), None, None, None) == gmb.GM_ERR_INVALID_ARG
    L.gm_destroy(None)
    # every entry point checks its context before anything else: a null context is an argument error, not a crash
    inv = gmb.GM_ERR_INVALID_ARG
    assert L.gm_draft(None, None, 3, 1.0, None, 0, 0, None, None, None) == inv
    assert L.gm_verify(None, None, 3, None, None, None) == inv
    assert L.gm_accept(None, None, 1, 3, 1.0, None, None, None, None, 0, 0, None, None, None, None, None, 0) == inv
    assert L.gm_spec_step(None, None, 3, 1.0, 0, 0, None, None, None) == inv
    assert L.gm_prefill(None, None, None, None, 0, 0, 1.0, None, 0, None, None) == inv
    assert L.gm_set_top_p(None, 0.7) == inv
    assert L.gm_nucleus(None, None, 1, 1.0, 0.7, None, None) == inv
    assert L.gm_capture_hidden(None, None, 0) == inv
    assert L.gm_head_prefill(None, None, None, 0, None, 0, None, 0) == inv
    assert L.gm_reconstruct(None, None, 1, 3, None, None, None, 0, None, None) == inv
    assert L.gm_reconstruct_states(None, None, 1, 3, None, None, None, 0, None, None, None) == inv
    assert L.gm_head_state_grad(None, 1, None, None, None, None, 0) == inv
    assert L.gm_head_ffn_backward(None, 1, None, None, None, None, None, None, 0) == inv
    assert L.gm_attention_backward(None, None, None, None, 1, 1, 0, None, None, None, 1, 1, None, None, None) == inv
    assert L.gm_head_attn_backward(None, None, None, None, 1, None, None, None, 1, 1, None, None, None, None, None, None, None, None, 0) == inv
    assert L.gm_head_update_backward(None, None, 1, 1, None, None, None, 2, None, None, None, 1, None, 2, None, None, None) == inv
    assert L.gm_head_update_step(None, None, 1, 1, 1.0, None, None, None, 2, None, None, 1, None, 2, 1, 1e-4, 0.9, 0.999, 1e-8, 0.01, None) == inv
    assert L.gm_head_input_backward(None, 1, None, None, None, None, None, None, None, 0) == inv
    assert L.gm_adamw_step(None, 1, None, None, None, None, None, 1, 1e-4, 0.9, 0.999, 1e-8, 0.01, 1.0) == inv
    assert L.gm_overlap(None, 1, 3, 1.0, None, None, None, None) == inv
    assert L.gm_dca_loss(None, 1, 3, None, None, None, None) == inv
    assert L.gm_dca_grad(None, 1, 3, 1.0, None, None, None, None, None, None) == inv
    assert L.gm_gemm(None, None, None, None, 1, 8, 64, 0) == inv
    assert L.gm_gemm_swiglu(None, None, None, None, 1, 16, 64) == inv
    assert L.gm_rollout_begin(None, None, None) == inv
    assert L.gm_rollout_step(None, None, None, 3, 1.0, 0, 0) == inv
    assert L.gm_rollout_run(None, None, None, 3, 1.0, 0, 0, 1, 1, None, None) == inv
    assert L.gm_pages_reset(None, None) == inv
    assert L.gm_pages_reserve(None, None, None, 1, None) == inv
    assert L.gm_pages_release(None, None, None) == inv
    assert L.gm_pages_free_count(None, None, None) == inv


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_16648_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text, f
