"""The shared library builds, loads without a GPU and exports every declared entry point."""
import ctypes
import os
import re

from paper_2604_10235_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "codecomp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cc_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in codecomp.h but not exported"
    assert set(names) == set(binding.EXPORTS)


def test_binding_struct_matches_header_field_order():
    text = open(os.path.join(ROOT, "include", "codecomp.h")).read()
    body = text[text.index("typedef struct cc_layer_desc {"):text.index("} cc_layer_desc;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split("{", 1)[1].split(";"):
        decl = decl.strip()
        if not decl:
            continue
        names = decl.replace("*", " ").split()
        kinds = {"int32_t", "int64_t", "float", "double", "const"}
        rest = " ".join(x for x in names if x not in kinds)
        fields += [n.strip() for n in rest.split(",")]
    assert fields == [f[0] for f in binding.cc_layer_desc._fields_]


def test_status_strings_without_gpu():
    lib = binding.load_library()
    assert lib.cc_status_string(0) == b"ok"
    assert b"workspace" in lib.cc_status_string(binding.CC_ERR_WORKSPACE)
    assert lib.cc_workspace_bytes(None, None) == 0
