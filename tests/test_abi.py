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
