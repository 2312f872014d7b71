"""The C-ABI library builds, loads and exports every function include/tw.h declares (no GPU needed)."""
import os
import re

import paper_2302_14357_b200 as pkg
from paper_2302_14357_b200 import build as tw_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "tw.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tw_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    tw_build.build()
    lib = pkg.load_library()
    names = _declared()
    assert "tw_init" in names and "tw_decode" in names and "tw_joiner_segment" in names and "tw_expand" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(pkg.EXPORTED_SYMBOLS) == names


def test_strerror_needs_no_device():
    lib = pkg.load_library()
    assert lib.tw_strerror(0) == b"ok"
    assert b"argument" in lib.tw_strerror(1)
    assert lib.tw_init(None, None, None) == 1          # TW_ERR_ARG before any CUDA call
    assert lib.tw_destroy(None) == 1
