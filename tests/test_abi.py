"""The C-ABI library builds, loads without a GPU and exports every symbol include/grouter.h declares."""
import ctypes
import os
import re

from paper_2603_06626_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "grouter.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(grouter_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(build.build())
    names = _declared_functions()
    assert "grouter_plan" in names and "grouter_moe_fwd" in names and "grouter_moe_bwd" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_entry_points():
    from paper_2603_06626_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_functions()


def test_host_only_calls_need_no_gpu():
    from paper_2603_06626_b200 import binding
    lib = binding.load_library()
    assert lib.grouter_strerror(0) == b"ok"
    assert b"aligned" in lib.grouter_strerror(-2)
    dims = binding.GrouterDims(512, 256, 512, 8, 8, 2, 0, 0, 0)
    n = lib.grouter_workspace_bytes(ctypes.byref(dims))
    rows = 512 * 2 + 128 * 8                       # T*k rounded to 128 plus one tile of padding per expert
    assert n >= rows * (3 * 256 + 5 * 512) * 2     # Xp, O, dYp [rows,d]; G, U, H, dG|dU [rows,F]
    bad = binding.GrouterDims(512, 250, 512, 8, 8, 2, 0, 0, 0)
    assert lib.grouter_workspace_bytes(ctypes.byref(bad)) == 0
    assert lib.grouter_wgrad_chunk_rows(None) == 0   # null context
