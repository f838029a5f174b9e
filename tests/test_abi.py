"""The C-ABI library loads and exports every symbol include/xlog.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "xlog.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(xlog_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    from paper_2609_27203_b200 import build, xlog
    lib = ctypes.CDLL(build.build())
    names = declared_symbols()
    assert "xlog_fixpoint" in names and "xlog_relation_load" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"libxlog.so does not export {n}"
    assert set(xlog.EXPORTS) <= set(names)


def test_struct_sizes_match_the_header():
    # compile a tiny C program against the header and compare sizeof() with the ctypes mirrors
    import subprocess
    import tempfile
    from paper_2609_27203_b200 import xlog
    src = ('#include "xlog.h"\n#include <stdio.h>\nint main(){printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(xlog_config),'
           'sizeof(xlog_plan), sizeof(xlog_receipt), sizeof(xlog_arg), sizeof(xlog_atom), sizeof(xlog_expr));return 0;}\n')
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "s.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "s")
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", exe, c])
        got = [int(x) for x in subprocess.check_output([exe]).split()]
    want = [ctypes.sizeof(t) for t in (xlog.Config, xlog.Plan, xlog.Receipt, xlog.Arg, xlog.AtomS, xlog.Expr)]
    assert got == want


def test_binding_refuses_to_run_without_a_gpu():
    import pytest
    import torch
    from paper_2609_27203_b200 import xlog
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        xlog.Context(arena_bytes=1 << 20)
