"""The shared library loads and exports every entry point include/dslide.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dslide.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dslide_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2201_12667_b200 import build
    lib = ctypes.CDLL(build.build())
    names = declared_functions()
    assert "dslide_train_step" in names and "dslide_init" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n


def test_binding_wraps_every_declared_symbol():
    from paper_2201_12667_b200 import build
    build.build()
    from paper_2201_12667_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()
    lib = ctypes.CDLL(binding.LIB_PATH)
    lib.dslide_status_str.restype = ctypes.c_char_p
    assert lib.dslide_status_str(0) == b"ok"
    assert b"range" in lib.dslide_status_str(5)


def test_config_struct_layout_matches_header_field_order():
    from paper_2201_12667_b200 import build
    build.build()
    from paper_2201_12667_b200 import binding
    text = open(os.path.join(ROOT, "include", "dslide.h")).read()
    body = text[text.index("typedef struct {"):text.index("} dslide_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        names = decl.split(None, 1)[1]
        fields += [n.strip().lstrip("*") for n in names.split(",")]
    assert fields == [f[0] for f in binding.Config._fields_]
