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


def test_binding_rejects_bad_shapes_before_any_launch():
    # the checks the wrapper makes on its own, so that a short or mistyped buffer never reaches a kernel
    import numpy as np
    import pytest
    import torch
    from paper_2609_27203_b200 import xlog
    a, b = np.zeros(5, np.int32), np.zeros(4, np.int32)
    assert xlog.check_load_shapes([a, a], np.zeros(5, np.float32), None) == 5
    with pytest.raises(ValueError, match="column 1 has 4 rows"):
        xlog.check_load_shapes([a, b], None, None)
    with pytest.raises(ValueError, match="tags have 3 rows"):
        xlog.check_load_shapes([a, a], np.zeros(3, np.float32), None)
    with pytest.raises(ValueError, match="one-dimensional"):
        xlog.check_load_shapes([np.zeros((5, 2), np.int32)], None, None)
    with pytest.raises(ValueError, match="does not live on cuda:0"):
        xlog.check_load_shapes([torch.zeros(5, dtype=torch.int32)], None, 0)            # a host tensor passed as a device input
    k, t = torch.zeros(8, dtype=torch.int32), torch.zeros(8, dtype=torch.float32)
    with pytest.raises(ValueError, match="must be torch.int32"):
        xlog.check_static_reduce_args(k.to(torch.int64), t, k, t)
    with pytest.raises(ValueError, match="must be a torch tensor"):
        xlog.check_static_reduce_args(np.zeros(8, np.int32), t, k, t)
    with pytest.raises(ValueError, match="must be a CUDA tensor"):
        xlog.check_static_reduce_args(k, t, k, t)
    with pytest.raises(ValueError):
        xlog.reduce_by_key_static("minplus", k, t, k, t)                                 # the public call makes the same checks first
