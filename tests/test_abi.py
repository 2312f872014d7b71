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


def test_binding_structs_match_the_header_layout(tmp_path):
    """tw_model / tw_config / tw_stats as the ctypes binding lays them out against what a C compiler makes of
    include/tw.h: size and the offset of every field (dtype, pred_init_state and pred_init_out included)."""
    import ctypes
    import shutil
    import subprocess
    import pytest
    from paper_2302_14357_b200 import binding
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    structs = {"tw_model": binding._Model, "tw_config": binding._Config, "tw_stats": binding._Stats}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "tw.h"', 'int main(void) {']
    for cname, cls in structs.items():
        lines.append('printf("%s %%zu\\n", sizeof(%s));' % (cname, cname))
        for field, _ in cls._fields_:
            lines.append('printf("%s.%s %%zu\\n", offsetof(%s, %s));' % (cname, field, cname, field))
    lines += ['printf("enums %d %d %d %d\\n", TW_F32, TW_BF16, TW_ACT_RELU, TW_ERR_TIMEOUT);', 'return 0; }']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run([cc, "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = dict(l.split(" ", 1) for l in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.splitlines())
    for cname, cls in structs.items():
        assert int(out[cname]) == ctypes.sizeof(cls), cname
        for field, _ in cls._fields_:
            assert int(out["%s.%s" % (cname, field)]) == getattr(cls, field).offset, (cname, field)
    assert out["enums"] == "%d %d %d %d" % (binding.DT_F32, binding.DT_BF16, binding.ACT_RELU, binding.TW_ERR_TIMEOUT)
