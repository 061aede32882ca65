"""The shared library loads without a GPU and exports every symbol the header declares."""
import os
import re

from paper_2605_07230_b200 import binding as cb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "cascade.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cascade_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 19
    L = cb.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(cb.EXPORTS) == names


def test_strerror_and_struct_sizes():
    L = cb.lib()
    assert L.cascade_strerror(0) == b"ok"
    assert b"tree" in L.cascade_strerror(cb.ERR_BAD_TREE)
    import ctypes as C
    assert C.sizeof(cb.Shape) == 40 and C.sizeof(cb.Params) == 16 and C.sizeof(cb.Layer) == 88


def test_null_arguments_do_not_need_a_device():
    L = cb.lib()
    assert L.cascade_create(None, None) == cb.ERR_INVALID_ARG
    assert L.cascade_destroy(None) == cb.ERR_INVALID_ARG
    assert L.cascade_tree_destroy(None) == cb.ERR_INVALID_ARG
    assert L.cascade_workspace_bytes(None) == 0
