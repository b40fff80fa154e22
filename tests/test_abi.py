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


def test_struct_mirrors_match_the_header(tmp_path):
    """The ctypes mirrors of the header's structs have the header's field names, order, offsets and sizes
    (a C program compiled against include/ba.h prints them)."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    mirrors = {"ba_config": B.ba_config, "ba_segments": B.ba_segments, "ba_page_table": B.ba_page_table}
    lines = ["#include <stdio.h>", "#include <stddef.h>", '#include "ba.h"', "int main(void) {"]
    for name, cls in mirrors.items():
        lines.append(f'  printf("{name} size %zu\\n", sizeof({name}));')
        for field, _ in cls._fields_:
            lines.append(f'  printf("{name} {field} %zu\\n", offsetof({name}, {field}));')
    lines += ["  return 0;", "}"]
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([gcc, "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    got = {tuple(line.split()[:2]): int(line.split()[2]) for line in out if line}
    for name, cls in mirrors.items():
        assert got[(name, "size")] == C.sizeof(cls), name
        for field, _ in cls._fields_:
            assert got[(name, field)] == getattr(cls, field).offset, (name, field)
    # no field of the header is missing from a mirror
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "ba.h")).read(), flags=re.S)
    for name, cls in mirrors.items():
        body = re.search(r"typedef struct \{([^}]*)\} " + name + ";", text).group(1)
        fields = re.findall(r"\*?\b([a-z_0-9]+)(?:\[\d+\])?\s*[,;]", body)
        assert [f for f, _ in cls._fields_] == fields, name
