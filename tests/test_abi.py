"""The C-ABI library builds, loads and exports every function include/lynx.h declares (no GPU)."""
import ctypes
import os
import re

import paper_2607_01831_b200 as lynx
from paper_2607_01831_b200 import build as lynx_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "lynx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lynx_[a-z0-9_]+)\s*\(", text)))


def test_header_declarations_are_exported():
    path = lynx_build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"lynx_split_quantize", "lynx_anchor_attention", "lynx_merge_verify_attention",
            "lynx_recombine"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in lynx.h but not exported"
    assert sorted(lynx.EXPORTS) == [n for n in names]


def test_host_side_validation_needs_no_gpu():
    L = lynx.load()
    assert L.lynx_version() >= 100
    assert L.lynx_status_string(0) == b"ok"
    # size/NULL checks run before any CUDA call
    assert L.lynx_split_quantize(None, 0, None, 0, 0, None, None, None, None) == 0
    assert L.lynx_split_quantize(None, 8, None, 0, 0, None, None, None, None) == 1
    assert L.lynx_recombine(None, None, None, -1, None, None, None) == 2
    geo = lynx.Geometry(32, 8, 16, 1024, 64)
    assert lynx.workspace_bytes(geo, 1, 1) > 256
    assert lynx.workspace_bytes(geo, 1, 4) > lynx.workspace_bytes(geo, 1, 1)
    assert lynx.workspace_bytes(lynx.Geometry(32, 8, 16, 1024, 64, head_dim=64), 1, 1) == 0
    assert lynx.workspace_bytes(lynx.Geometry(32, 8, 24, 1024, 64), 1, 1) == 0      # block_tokens % 16
    assert lynx.workspace_bytes(lynx.Geometry(32, 8, 16, 1024, 64), 1, 65) == 0     # too many positions
    assert lynx.workspace_bytes(lynx.Geometry(32, 8, 16, 1024, 64), 1, 64) > 0      # the window cap (in slices)
    assert lynx.workspace_bytes(lynx.Geometry(64, 8, 16, 1024, 64), 1, 16) > 0      # 128 columns: two slices
    assert lynx.workspace_bytes(lynx.Geometry(8 * 17, 8, 16, 1024, 64), 1, 1) == 0  # more than 16 q heads per KV head
    assert lynx.workspace_bytes(lynx.Geometry(30, 8, 16, 1024, 64), 1, 1) == 0      # Hq % Hkv
