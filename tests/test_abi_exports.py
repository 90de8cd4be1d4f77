"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2502_11417_b200 import lib, library_path
from paper_2502_11417_b200.api import EXPORTS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(disco_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_header_symbols_are_exported():
    L = lib()
    assert os.path.exists(library_path())
    decl = declared_functions()
    assert set(EXPORTS) <= set(decl) and len(decl) >= 9
    for name in decl:
        assert hasattr(L, name), name
    raw = ctypes.CDLL(library_path())
    for name in decl:
        getattr(raw, name)


def test_calls_without_a_context_fail_cleanly():
    L = lib()
    assert L.disco_eval_policies(None, None, 0, 0, None, None) == -1
    assert b"null" in L.disco_last_error()
    assert L.disco_reduce_stats(None, None, None) == -1
    L.disco_free_trace(None)
