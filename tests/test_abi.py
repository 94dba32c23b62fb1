"""The C-ABI library loads on a machine without a GPU and exports what include/st.h declares."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "st.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(st_[a-z0-9_]+)\s*\(", text)) - {"st_alloc_fn", "st_free_fn"})


def test_library_exports_every_declared_symbol():
    from paper_2504_12329_b200 import build, binding
    build.build()
    L = binding.lib()
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names


def test_struct_layouts_match_header():
    from paper_2504_12329_b200 import binding
    # sizes implied by the header on LP64: st_config = 14 int32/float + 3 pointers; st_handoff = 3 int32
    assert C.sizeof(binding.StConfig) == 14 * 4 + 3 * 8
    assert C.sizeof(binding.StHandoff) == 12
    assert C.sizeof(binding.StSpecParams) == 4 + 4 + 8 + 8 * 4 + (8 + 4 + 4) + (8 + 4) + 3 * 4 + 8 + 4 + 4 + (8 + 4 + 4) + 8 + (4 + 4)   # ... sample_seed, top_p + tail padding
    # st_spec_result ends with three doubles and three int32 (8-byte aligned tail)
    assert binding.StSpecResult.t_prompt_prefill_s.offset % 8 == 0
    assert C.sizeof(binding.StSpecResult) == binding.StSpecResult.n_decode.offset + 8
    assert binding.st_strerror(0) == "ok" and "KV" in binding.st_strerror(binding.ST_ERR_KV_FULL)


def test_no_device_is_a_loud_error():
    import torch
    from paper_2504_12329_b200 import binding
    if torch.cuda.is_available():
        return
    cfg = binding.StConfig(n_layers=1, hidden=64, n_q_heads=1, n_kv_heads=1, head_dim=64, ffn=64, vocab=16,
                           rope_theta=1e4, rms_eps=1e-6, tie_embeddings=1, qkv_bias=1, max_seqs=1, max_tokens=64, page_size=16)
    h = C.c_void_p()
    rc = binding.lib().st_model_create(C.byref(cfg), 0, 0, None, C.byref(h))
    assert rc == binding.ST_ERR_INTERNAL and not h.value
    assert "no CPU path" in binding.st_strerror(rc)
