"""The C-ABI library loads without a GPU and exports every symbol include/hq.h declares."""
import ctypes
import os
import re

from paper_2105_04246_b200 import build as hq_build
from paper_2105_04246_b200 import hq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "hq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hq_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree():
    assert _declared() == sorted(hq.EXPORTS)


def test_library_exports_every_declared_symbol():
    path = hq_build.build()
    lib = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(lib, name), name
    lib.hq_status_string.restype = ctypes.c_char_p
    assert lib.hq_status_string(0) == b"ok"
    assert b"wait" in lib.hq_status_string(6)


def test_range_state_layout_matches_header():
    text = open(os.path.join(ROOT, "include", "hq.h")).read()
    body = re.search(r"typedef struct \{([^}]*)\} hq_range_state;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            names += [re.sub(r"\[.*\]", "", n).strip() for n in decl.split(None, 1)[1].split(",")]
    assert names == list(hq.RANGE_STATE_DTYPE.names)
    assert hq.RANGE_STATE_DTYPE.itemsize == 64
