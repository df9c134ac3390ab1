"""Host-only checks of the C-ABI boundary: the library builds, loads and exports every symbol the header
declares, and the Python binding declares a signature for each of them (no compute calls: no GPU here)."""
import ctypes
import os
import re

from paper_2607_24434_b200 import build as dx_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "draftexpert.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:dx_status|int32_t|int64_t|const char\*)\s+(\w+)\s*\(", text)
    return sorted(set(names))


def test_header_symbols_exported_and_bound():
    lib_path = dx_build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 25
    for required in ("moe_draft_step", "moe_verify_block", "spec_accept", "expert_cache_prefetch",
                     "expert_cache_stage", "dx_pack_expert", "moe_verify_block_cached", "moe_draft_step_cached",
                     "dx_set_wait_limit", "dx_set_accept_l2_keep", "dx_stage_block", "dx_decoder_step"):
        assert required in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    from paper_2607_24434_b200 import binding
    assert sorted(binding.SIGNATURES) == names
    loaded = binding.load()
    assert loaded.dx_status_string(0) == b"ok"
    assert loaded.dx_status_string(8) == b"unsupported configuration"


def test_desc_struct_layout_matches_header():
    from paper_2607_24434_b200 import binding, synth
    assert ctypes.sizeof(binding.LayerDesc) == 12 * 4
    assert ctypes.sizeof(binding.CacheStats) == 11 * 8
    d = binding._desc(synth.shape_moonlight())
    assert (d.hidden, d.n_experts, d.top_k, d.inter, d.score_fn) == (2048, 64, 6, 1408, 1)
    assert abs(d.routed_scale - 2.446) < 1e-6
    n = ctypes.c_size_t(0)
    assert binding.load().dx_expert_blob_bytes(ctypes.byref(d), 1408, ctypes.byref(n)) == 0
    assert n.value == 17301504          # one bf16 expert of the DeepSeek-V2-Lite shape
    assert binding.load().dx_expert_blob_bytes(ctypes.byref(d), 1407, ctypes.byref(n)) == 8


def test_argument_errors_without_a_device():
    from paper_2607_24434_b200 import binding
    lib = binding.load()
    assert lib.dx_destroy(None) == 1
    assert lib.moe_draft_step(None, None, None, None, None, None) == 1
    assert lib.spec_accept(None, None, 1, None, 1, 256, 1, None, 0, 0, None, None, None, None) == 1
    assert lib.moe_verify_block_cached(None, None, 4, None, 0, None, None, None, None, None, None, None, None, None,
                                       None) == 1
    assert lib.dx_set_wait_limit(None, 100) == 1 and lib.dx_set_launch_overlap(None, 3) == 1
    assert lib.dx_set_accept_l2_keep(None, 1 << 20) == 1
    assert lib.dx_stage_block(None, None, None, 16, None) == 1
    assert lib.dx_decoder_destroy(None) == 1
    assert lib.dx_decoder_step(None, 0, -1, None, None, None, None, None, None, None, None) == 1
