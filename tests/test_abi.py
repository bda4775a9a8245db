"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import paper_2512_07503_b200 as sjd
from paper_2512_07503_b200 import build as sjd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(sjd_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(sjd_build.build())
    names = _declared_functions()
    assert "sjd_step" in names and "sjd_workspace_bytes" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"


def test_host_only_entry_points():
    assert sjd.sjd_version() == 1
    assert sjd.sjd_status_string(0) == "ok"
    assert "workspace" in sjd.sjd_status_string(-5)
    p = sjd.sjd_params()
    p.B, p.W = 16, 64
    n = sjd.sjd_workspace_bytes(p)
    assert n >= 16 * 64 * 16 and n % 256 == 0


def test_params_struct_matches_header_layout():
    # field order and count of the ctypes mirror follow the header
    text = open(os.path.join(ROOT, "include", "sjd.h")).read()
    body = text[text.index("typedef struct {", text.index("HOST struct")):]
    body = body[:body.index("} sjd_params;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        for part in decl.split(","):
            fields.append(re.findall(r"([A-Za-z_][A-Za-z0-9_]*)\s*$", part.strip())[0])
    assert fields == [f for f, _ in sjd.sjd_params._fields_]


def test_row_kernel_query_needs_no_gpu_and_follows_the_shape_rules():
    import ctypes as C
    from paper_2512_07503_b200 import binding as B

    def params(V, top_k, dtype=B.SJD_BF16, flags=0, W=8):
        p = B.sjd_params()
        p.struct_size = C.sizeof(B.sjd_params)
        p.B, p.W, p.V, p.logits_dtype, p.top_k, p.flags = 2, W, V, dtype, top_k, flags
        p.stride_b, p.stride_w = W * V, V
        return p

    assert B.sjd_row_kernel(params(65536, 2000)) == B.SJD_ROWS_RANGES
    assert B.sjd_row_kernel(params(65536, 1000, flags=B.SJD_FLAG_FORCE_TILES)) == B.SJD_ROWS_TILES
    assert B.sjd_row_kernel(params(65536, 2000, flags=B.SJD_FLAG_FORCE_GENERIC)) == B.SJD_ROWS_GENERIC
    assert B.sjd_row_kernel(params(65536, 8192)) == B.SJD_ROWS_GENERIC      # kcap above what the on-chip path stages
    assert B.sjd_row_kernel(params(1032, 7, dtype=B.SJD_F32)) == B.SJD_ROWS_GENERIC
    import pytest
    with pytest.raises(B.SjdError):
        B.sjd_row_kernel(params(65530, 10))
