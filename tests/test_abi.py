"""The C-ABI library builds, loads without a GPU, and exports every symbol that
include/aflex.h declares; the binding lists the same names."""
import ctypes
import os
import re

from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "aflex.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"AFLEX_API[^;(]*?\b(aflex_\w+)\s*\(", text)))


def test_header_declares_the_hot_path_entry_points():
    names = declared_symbols()
    for required in ("aflex_attn_decode", "aflex_ffn_dense", "aflex_ffn_moe", "aflex_layer_step",
                     "aflex_create", "aflex_destroy", "aflex_workspace_bytes"):
        assert required in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = B.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    for name in declared_symbols():
        assert hasattr(lib, name), f"{name} declared in aflex.h but not exported"
    assert sorted(AF.EXPORTS) == declared_symbols()


def test_host_only_calls_work_without_a_gpu():
    lib = AF.load_library()
    assert lib.aflex_version() >= 100
    assert lib.aflex_status_string(0) == b"AFLEX_OK"
    assert lib.aflex_status_string(5) == b"AFLEX_ERR_TIMEOUT"
    # workspace query is pure host arithmetic
    layer = AF.LayerDesc(AF.attn_desc(64, 8, 128), 5120, 25600, 0, 0, None, None, None, None, None)
    small = AF.workspace_bytes(layer, 32, 256)
    big = AF.workspace_bytes(layer, 128, 512)
    assert 0 < small < big < (8 << 30)
    assert lib.aflex_destroy(None) == 0
