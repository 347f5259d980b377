"""The C-ABI library loads and exports every symbol include/qdit.h declares (no compute without a GPU)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "qdit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qdit_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2503_02508_b200 as q
    names = declared_symbols()
    assert len(names) >= 30
    lib = ctypes.CDLL(q.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(q.EXPORTS) == names        # the binding covers exactly the declared ABI


def test_host_only_entry_points():
    import paper_2503_02508_b200 as q
    assert q.lib.qdit_status_string(0) == b"ok"
    assert q.lib.qdit_status_string(q.QDIT_ERR_TIMEOUT) == b"device-side wait timed out"
    assert q.lib.qdit_create(None, 0, None) == q.QDIT_ERR_INVALID_ARG
    assert q.lib.qdit_destroy(None) == q.QDIT_ERR_INVALID_ARG
