"""The C-ABI library builds, loads and exports every symbol include/sfb.h declares (no compute, no GPU)."""
import ctypes
import os
import re

import paper_1409_5705_b200 as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "sfb.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(sfb_[a-z_]+)\s*\(", src)))


def test_library_builds_and_exports_every_declared_symbol():
    S.build()
    L = ctypes.CDLL(S.LIB)
    names = _declared()
    assert "sfb_step" in names and "sfb_init" in names and len(names) >= 14
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(S.EXPORTS)


def test_host_only_calls():
    cfg = S.make_config(S.MLR, 325_000, 10_000, 16, 64, 0.05)
    n = S.sfb_workspace_bytes(cfg)
    # gathered fp32 factors: K*(rows+cols)*4 bytes, plus the staging copy of X and small buffers
    assert n >= 1024 * (325_000 + 10_000) * 4
    assert S.strerror(0) == "ok" and "argument" in S.strerror(-1)
    bad = S.make_config(S.MLR, 10, 6, 2, 2, 0.1)           # cols not a multiple of 4
    out = ctypes.c_size_t()
    assert S.lib().sfb_workspace_bytes(ctypes.byref(bad), ctypes.byref(out)) == -3
    assert S.lib().sfb_workspace_bytes(None, ctypes.byref(out)) == -1
    h = ctypes.c_void_p()
    assert S.lib().sfb_init(ctypes.byref(cfg), None, None, 0, ctypes.byref(h)) == -1
    assert S.lib().sfb_step(None, None, None, None) == -1


def test_struct_layouts_match_the_header():
    """ctypes mirrors of sfb_config / sfb_stats have the C compiler's sizes."""
    import subprocess, tempfile
    prog = '#include <stdio.h>\n#include "sfb.h"\nint main(){printf("%zu %zu", sizeof(sfb_config), sizeof(sfb_stats));return 0;}\n'
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "t.c")
        open(c, "w").write(prog)
        exe = os.path.join(d, "t")
        subprocess.check_call(["gcc", "-I" + os.path.join(ROOT, "include"), c, "-o", exe])
        a, b = map(int, subprocess.check_output([exe]).split())
    assert a == ctypes.sizeof(S.sfb_config) and b == ctypes.sizeof(S.sfb_stats)


def test_binding_error_checks_name_the_call_they_wrap():
    """Every ``self._ck(lib().sfb_x(...), "sfb_x")`` in the binding passes exactly the return code and the name of the
    entry point it called (a slip here only shows when that method runs on a GPU)."""
    import ast
    import os
    src = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_1409_5705_b200",
                            "__init__.py")).read()
    seen = 0
    for node in ast.walk(ast.parse(src)):
        if isinstance(node, ast.Call) and isinstance(node.func, ast.Attribute) and node.func.attr == "_ck":
            assert len(node.args) == 2 and not node.keywords, ast.unparse(node)
            call, name = node.args
            assert isinstance(name, ast.Constant) and isinstance(call, ast.Call) and isinstance(call.func, ast.Attribute)
            assert call.func.attr == name.value, ast.unparse(node)
            seen += 1
    assert seen >= 25
