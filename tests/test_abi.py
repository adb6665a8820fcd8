"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2510_18239_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    with open(os.path.join(ROOT, "include", "lime.h")) as f:
        text = f.read()
    return re.findall(r"LIME_API\s+[\w\s\*]+?\b(lime_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    lib_path = build.build()
    assert os.path.exists(lib_path)
    names = declared_symbols()
    assert len(names) >= 12 and "lime_score_candidates" in names and "lime_encode_user" in names
    lib = ctypes.CDLL(lib_path)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_version_string_and_host_side_validation():
    lib = binding.load_library()
    assert b"sm_100a" in lib.lime_version()
    # NULL config / out pointer are rejected before any CUDA call
    assert lib.lime_create(None, None) == 1
    h = ctypes.c_void_p()
    bad = binding.lime_config(d=30, H=2, ell=8, n_layers=1, d_ff=0, dtype=0, phi=0, ln=1, gated_mlp=1)
    assert lib.lime_create(ctypes.byref(bad), ctypes.byref(h)) == 2          # d % 8 != 0
    bad = binding.lime_config(d=32, H=3, ell=8, n_layers=1, d_ff=0, dtype=0, phi=0, ln=1, gated_mlp=1)
    assert lib.lime_create(ctypes.byref(bad), ctypes.byref(h)) == 2          # d % H != 0
    bad = binding.lime_config(d=32, H=2, ell=0, n_layers=1, d_ff=0, dtype=0, phi=0, ln=1, gated_mlp=1)
    assert lib.lime_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    bad = binding.lime_config(d=32, H=2, ell=8, n_layers=17, d_ff=0, dtype=0, phi=0, ln=1, gated_mlp=1)
    assert lib.lime_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    bad = binding.lime_config(d=32, H=2, ell=8, n_layers=1, d_ff=0, dtype=7, phi=0, ln=1, gated_mlp=1)
    assert lib.lime_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    assert lib.lime_destroy(None) == 0
    assert lib.lime_workspace_bytes(None, 1, 1) == 0


def test_struct_layouts_match_header():
    assert ctypes.sizeof(binding.lime_config) == 13 * 4          # 12 fields of the paper's model + cand_heads
    assert ctypes.sizeof(binding.lime_weights) == 8 * (1 + 6 * binding.LIME_MAX_LAYERS + 3)
    assert ctypes.sizeof(binding.lime_ffn) == 4 * 4 + 8 * 8      # n_hidden + 3 widths, 4 weight and 4 bias pointers


def test_ffn_entry_points_validate_on_the_host():
    lib = binding.load_library()
    assert lib.lime_set_head(None, None, None) == 1
    assert lib.lime_set_context_mlp(None, 4, None, None) == 1
    assert lib.lime_contextualize_links(None, None, 1, None, None) == 1
    assert lib.lime_head_workspace_bytes(None, 4) == 0
    assert lib.lime_score_candidates_head(None, None, 1, None, None, None, 1, 1, None, 0, None, None, None, 0, None) == 1
