"""The C-ABI library loads without a GPU and exports every symbol include/specvla.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "specvla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specvla_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_header_symbols():
    from paper_2507_22424_b200.build import build
    path = build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"specvla_prefill", "specvla_draft_tree", "specvla_verify_tree",
            "specvla_generate_action"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_declares_every_export():
    from paper_2507_22424_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_host_side_validation_without_gpu():
    from paper_2507_22424_b200 import binding as B
    md = B.ModelDesc(2, 256, 4, 64, 688, 1024, 768, 256, 1e-6, 1e4, 512, 1, 512, 1, 16)
    full = B.lib.specvla_workspace_bytes(ctypes.byref(md))
    md.weight_bits = 8
    assert 0 < B.lib.specvla_workspace_bytes(ctypes.byref(md)) < full      # int8 codes: smaller weight copy
    md.weight_bits = 5
    assert B.lib.specvla_workspace_bytes(ctypes.byref(md)) == 0
    md.weight_bits = 16
    assert B.lib.specvla_workspace_bytes(ctypes.byref(md)) > 0
    md.head_dim = 48
    assert B.lib.specvla_workspace_bytes(ctypes.byref(md)) == 0
    assert B.lib.specvla_strerror(-3) == b"malformed draft tree"
    assert B.lib.specvla_gemm_scratch_bytes(27, 4096, 4096) >= 27 * 4096 * 4
    assert B.lib.specvla_reset(None, 0) == -1
