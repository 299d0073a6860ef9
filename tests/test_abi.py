"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dd_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2607_26475_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "dd_select_topk" in names and "dd_gather_kv_from_host" in names
    assert "dd_sparse_decode_attn" in names and "dd_decode_layer_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/dd.h but not exported"


def test_binding_lists_the_same_entry_points_and_error_strings():
    from paper_2607_26475_b200 import build
    build.build()
    from paper_2607_26475_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    assert binding.lib.dd_strerror(0) == b"ok"
    assert binding.lib.dd_strerror(binding.DD_ERR_NOT_PINNED) == b"host memory is not page-locked"
    # size queries and configuration checks run on the host
    cfg = binding.DDConfig(32, 8, 32, 8, 128, 16, 2048, 128, 0, 2, 2, 0, 0, 0, 0, None, None, None, 0, 0, 0, None, None)
    assert binding.lib.dd_slot_bytes(ctypes.byref(cfg)) == 64 << 20
    assert binding.lib.dd_ring_bytes(ctypes.byref(cfg)) == 128 << 20
    bad = binding.DDConfig(32, 8, 32, 8, 64, 16, 2048, 128, 0, 2, 2, 0, 0, 0, 0, None, None, None, 0, 0, 0, None, None)
    assert binding.lib.dd_slot_bytes(ctypes.byref(bad)) == 0
    h = ctypes.c_void_p()
    assert binding.lib.dd_create(ctypes.byref(bad), ctypes.byref(h)) == binding.DD_ERR_INVALID_ARG
    assert b"head_dim" in binding.lib.dd_last_error_message(None)
