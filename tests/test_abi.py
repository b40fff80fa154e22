"""The C-ABI library loads on a machine without a GPU, exports every symbol the
header declares, and turns bad arguments into status codes."""
import ctypes as C
import os
import re

import pytest

from paper_2409_15355_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ba.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ba_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = B.load_library()
    names = declared_symbols()
    assert {"ba_segment", "ba_reencode_k", "ba_block_prefill", "ba_final_attend"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_status_strings():
    assert B.status_string(B.BA_OK) == "ok"
    assert "workspace" in B.status_string(B.BA_ERR_WORKSPACE)
    assert "unknown" in B.status_string(99)


def test_size_queries_and_argument_checks():
    cfg = B.ba_config(32, 8, 128, 0, 500000.0, 0.0, 0)
    assert B.ba_workspace_bytes(cfg, 512, 1024) > 512 * 128 * 4
    n = B.ba_segments_bytes(2, 5, 9)
    assert n >= (3 * 9 + 9 * 5) * 4 and n % 16 == 0
    with pytest.raises(B.BaError) as e:
        B.ba_segments_bytes(0, 5, 9)
    assert e.value.status == B.BA_ERR_INVALID_ARG
    for bad in (B.ba_config(32, 8, 96, 0, 1e4, 0.0, 0), B.ba_config(32, 5, 128, 0, 1e4, 0.0, 0)):
        with pytest.raises(B.BaError) as e:
            B.ba_workspace_bytes(bad, 8, 8)
        assert e.value.status == B.BA_ERR_UNSUPPORTED
    lib = B.load_library()
    assert lib.ba_destroy(None) == B.BA_ERR_INVALID_ARG
    assert lib.ba_last_device_status(None) == B.BA_ERR_INVALID_ARG
    assert lib.ba_create(None, C.byref(cfg), 0, 0) == B.BA_ERR_INVALID_ARG


def test_create_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    cfg = B.ba_config(4, 2, 64, 0, 10000.0, 0.0, 0)
    with pytest.raises(B.BaError) as e:
        B.ba_create(cfg, 0, 1 << 20)
    assert e.value.status == B.BA_ERR_CUDA
