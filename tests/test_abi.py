"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

import paper_2605_20022_b200 as fd
from paper_2605_20022_b200 import _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, f)).read(), flags=re.S)
            names |= set(re.findall(r"\b(fd_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    _build.build()
    lib = ctypes.CDLL(_build.SO)
    decl = declared_symbols()
    assert {"fd_create", "fd_destroy", "fd_attn_draft_verify", "fd_verify_accept", "fd_kv_commit",
            "fd_last_device_status"} <= decl
    for name in decl:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert decl == set(fd.EXPORTS), "binding and header disagree"


def test_status_strings_and_struct_layout():
    assert fd.status_string(fd.FD_OK) == "FD_OK"
    assert fd.status_string(fd.FD_ERR_UNSUPPORTED) == "FD_ERR_UNSUPPORTED"
    assert ctypes.sizeof(fd.fd_config) == 40                  # ten 4-byte fields, as in the header
    header = open(os.path.join(ROOT, "include", "flexdraft.h")).read()
    body = header[header.index("typedef struct {"):header.index("} fd_config;")]
    fields = re.findall(r"^\s*(?:int|float)\s+(\w+);", body, flags=re.M)
    assert fields == [f[0] for f in fd.fd_config._fields_]
