"""CPU-side checks of the boundary: the shared library loads and exports every symbol the
header declares; the binding's structs match the header's field order."""
import ctypes
import os
import re

import pytest

from paper_2603_14549_b200 import binding as A
from paper_2603_14549_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = open(os.path.join(ROOT, "include", "asap.h")).read()


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return ctypes.CDLL(A.LIB_PATH)


def test_every_declared_symbol_is_exported(lib):
    declared = set(re.findall(r"\b(asap_[a-z_]+)\s*\(", HEADER))
    assert declared == set(A.EXPORTS), declared ^ set(A.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def _struct_fields(name):
    body = re.search(r"typedef struct \{([^}]*)\}\s*" + name + ";", HEADER, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        for part in decl.split(","):
            fields.append(re.findall(r"\*?\s*([A-Za-z_0-9]+)\s*$", part.strip())[0])
    return fields


@pytest.mark.parametrize("cname,cls", [("asap_inputs", A.CInputs), ("asap_params", A.CParams),
                                       ("asap_outputs", A.COutputs)])
def test_binding_struct_matches_header(cname, cls):
    assert _struct_fields(cname) == [f[0] for f in cls._fields_]


def test_init_without_gpu_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(A.AsapError):
        A.asap_init(0, 1000, 1, 1, 128)


def test_missing_library_is_a_loud_error(monkeypatch, tmp_path):
    monkeypatch.setattr(A, "_lib", None)
    monkeypatch.setattr(A, "LIB_PATH", str(tmp_path / "libasap.so"))
    with pytest.raises(FileNotFoundError):
        A.load_library()
