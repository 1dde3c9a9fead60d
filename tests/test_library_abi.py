"""The C-ABI library builds, loads and exports every entry point the header declares, and the
Python argument structs have the header's layout.  No GPU needed (no compute call is made)."""
import ctypes
import os
import re
import shutil
import subprocess

import pytest

from paper_2512_14069_b200 import binding as rb
from paper_2512_14069_b200 import build as rbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "radar.h")

needs_nvcc = pytest.mark.skipif(not os.path.exists(os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")),
                                reason="nvcc not available")


@needs_nvcc
def test_library_builds_and_exports_every_declared_symbol():
    path = rbuild.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(radar_[a-z_]+)\s*\(", text))
    assert {"radar_expand_step", "radar_rerank_build_tree", "radar_tree_attention", "radar_verify_accept",
            "radar_create", "radar_destroy", "radar_read_device_status", "radar_status_string"} <= names
    for n in names:
        assert hasattr(L, n), n
    L.radar_status_string.restype = ctypes.c_char_p
    assert L.radar_status_string(0) == b"ok"
    assert b"NaN" in L.radar_status_string(-6)


def test_python_structs_match_the_header_layout(tmp_path):
    """Compile a C program that prints sizeof/offsetof of every field and compare with ctypes."""
    structs = {"radar_expand_args": rb.ExpandArgs, "radar_tree_args": rb.TreeArgs,
               "radar_attn_args": rb.AttnArgs, "radar_accept_args": rb.AcceptArgs, "radar_acclen_args": rb.AccLenArgs,
               "radar_train_args": rb.TrainArgs}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "radar.h"', "int main(void){"]
    for cname, st in structs.items():
        lines.append('printf("%s %%zu\\n", sizeof(%s));' % (cname, cname))
        for f, _ in st._fields_:
            lines.append('printf("%s.%s %%zu\\n", offsetof(%s, %s));' % (cname, f, cname, f))
    lines.append("return 0;}")
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.check_call([shutil.which("gcc") or "gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    out = dict(l.split() for l in subprocess.check_output([str(exe)], text=True).splitlines())
    for cname, st in structs.items():
        assert int(out[cname]) == ctypes.sizeof(st), cname
        for f, _ in st._fields_:
            assert int(out["%s.%s" % (cname, f)]) == getattr(st, f).offset, (cname, f)


def test_binding_fails_loudly_without_the_library(monkeypatch):
    monkeypatch.setattr(rb, "_lib", None)
    monkeypatch.setattr(rb, "LIB_PATH", "/nonexistent/libradar_b200.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        rb.lib()
