"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares;
the struct layouts of the Python binding match the header's field order."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gs.h")


@pytest.fixture(scope="module")
def lib_path():
    from paper_2609_05255_b200 import build
    return build.build()


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(gs_[a-z_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = declared_functions()
    for must in ("gs_preprocess", "gs_render_forward", "gs_render_backward", "gs_appearance_forward",
                 "gs_appearance_backward", "gs_create", "gs_destroy", "gs_workspace_bytes", "gs_last_error"):
        assert must in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in gs.h but not exported"


def test_workspace_size_is_monotone_and_rejects_bad_arguments(lib_path):
    lib = ctypes.CDLL(lib_path)
    f = lib.gs_workspace_bytes
    f.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64]
    f.restype = ctypes.c_size_t
    assert f(-1, 64, 64, 10) == 0 and f(10, 0, 64, 10) == 0 and f(10, 64, 64, -1) == 0
    a, b, c = f(1000, 64, 64, 5000), f(2000, 64, 64, 5000), f(2000, 64, 64, 50000)
    assert 0 < a < b < c
    assert c >= 4 * 4 * 50000 + 3 * 4 * 2000          # two ping-pong instance lists + the depth sort
    assert f(1_000_000, 1256, 828, 0) >= 48 * 1_000_000  # the backward's per-Gaussian 2D gradients


def test_binding_struct_fields_follow_the_header():
    import importlib.util
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    spec = importlib.util.find_spec("paper_2609_05255_b200.api")
    src = open(spec.origin).read()
    bodies = {name: body for body, name in re.findall(r"typedef struct \{([^}]*)\}\s*(\w+);", text)}
    for struct in ("GsCamera", "GsScene", "GsProjected", "GsBinning", "GsGrads"):
        body = bodies[struct]
        fields = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            for part in decl.split(","):
                fields.append(re.sub(r"\[.*\]", "", part.strip().split()[-1].lstrip("*")))
        py = re.search(r"class " + struct + r"\(C\.Structure\):\s*_fields_ = \[(.*?)\]\n", src, re.S).group(1)
        py_fields = re.findall(r'\("(\w+)"', py)
        assert py_fields == fields, (struct, fields, py_fields)
