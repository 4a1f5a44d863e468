"""Host-only checks of the C-ABI library: it loads and exports every symbol the
header declares.  No kernel is launched."""
import os
import re

import paper_2505_24196_b200 as clasp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "clasp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(clasp_[a-zA-Z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = clasp.load_library()
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(clasp.SYMBOLS) == names


def test_host_only_entry_points():
    lib = clasp.load_library()
    import datagen
    cfg = clasp.make_config(datagen.CONFIGS["8b"], max_ctx=1024, max_rows=64, max_M=16)
    nbytes = lib.clasp_workspace_bytes(cfg)
    assert 10 << 20 < nbytes < 2 << 30
    bad = clasp.make_config(datagen.CONFIGS["8b"], max_ctx=1024, max_rows=64, max_M=16)
    bad.head_dim = 96
    assert lib.clasp_workspace_bytes(bad) == 0
    assert clasp.strerror(0) == "ok" and "capacity" in clasp.strerror(-3)


def test_accept_rule_on_host():
    """Greedy acceptance: longest matching prefix, then the full model's own token."""
    import ctypes as C
    lib = clasp.load_library()

    def run(draft, full):
        K = len(draft)
        d = (C.c_int32 * max(K, 1))(*draft)
        f = (C.c_int32 * (K + 1))(*full)
        a = C.c_int32()
        out = (C.c_int32 * (K + 1))()
        assert lib.clasp_accept(d, f, K, C.byref(a), out) == 0
        return a.value, list(out[:a.value + 1])

    assert run([5, 6, 7], [5, 6, 7, 8]) == (3, [5, 6, 7, 8])
    assert run([5, 6, 7], [5, 9, 7, 8]) == (1, [5, 9])
    assert run([5, 6, 7], [1, 6, 7, 8]) == (0, [1])
    assert run([], [4]) == (0, [4])
