"""The C-ABI library loads without a GPU, exports every symbol the header declares, and
rejects host-checkable misuse before touching the device (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "treewy.h")


@pytest.fixture(scope="module")
def tw():
    from paper_2608_20961_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(treewy_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(tw):
    names = declared_functions()
    assert {"treewy_tree_prepare", "treewy_verify", "treewy_verify_generic", "treewy_commit",
            "treewy_status_string", "treewy_version"} <= set(names)
    lib = ctypes.CDLL(tw.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), name
    assert tw.version() >= 100
    assert tw.status_string(0) == "ok" and "invalid" in tw.status_string(1)


def test_struct_mirror_matches_header_field_order(tw):
    text = open(HEADER).read()
    body = text[text.index("typedef struct {"):text.index("} treewy_tree_t;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"\b\*?(\w+);", body)
    assert fields == [f[0] for f in tw.TreeStruct._fields_]


A = 0x1000  # any 16-byte aligned, never dereferenced: every call below fails its checks first


def _tree(tw, **kw):
    base = dict(B=2, T=8, H_v=4, max_nodes=0, node_offsets=A, parent=A, depth=A, anc_mask=A,
                cum_log_gate=A, level_order=A)
    base.update(kw)
    return tw.TreeStruct(**base)


def test_argument_errors_are_reported_before_any_launch(tw):
    lib = tw.load_library()
    vp = ctypes.c_void_p
    ok_args = lambda t: (vp(A), vp(A), vp(A), vp(A), vp(A), ctypes.byref(t), 2, tw.TREEWY_BF16,
                         tw.TREEWY_BF16, vp(A), vp(A), None, None)
    # null tree / null data pointers / misaligned pointers
    assert lib.treewy_tree_prepare(None, vp(A), None, None) == tw.TREEWY_ERR_INVALID_ARG
    t = _tree(tw)
    assert lib.treewy_tree_prepare(ctypes.byref(t), None, None, None) == tw.TREEWY_ERR_INVALID_ARG
    assert lib.treewy_tree_prepare(ctypes.byref(t), vp(A + 4), None, None) == tw.TREEWY_ERR_INVALID_ARG
    t = _tree(tw, anc_mask=None)
    assert lib.treewy_tree_prepare(ctypes.byref(t), vp(A), None, None) == tw.TREEWY_ERR_INVALID_ARG
    # bad sizes
    for bad in (dict(B=-1), dict(T=-3), dict(H_v=0), dict(max_nodes=-1)):
        t = _tree(tw, **bad)
        assert lib.treewy_verify(*ok_args(t)) == tw.TREEWY_ERR_INVALID_ARG
    t = _tree(tw, max_nodes=65)
    assert lib.treewy_verify(*ok_args(t)) == tw.TREEWY_ERR_UNSUPPORTED
    # H_v not a multiple of H_qk, unknown dtypes
    t = _tree(tw)
    args = list(ok_args(t))
    args[6] = 3
    assert lib.treewy_verify(*args) == tw.TREEWY_ERR_INVALID_ARG
    args = list(ok_args(t))
    args[7] = 7
    assert lib.treewy_verify(*args) == tw.TREEWY_ERR_UNSUPPORTED
    args = list(ok_args(t))
    args[0] = None
    assert lib.treewy_verify(*args) == tw.TREEWY_ERR_INVALID_ARG
    assert lib.treewy_verify_generic(*args) == tw.TREEWY_ERR_INVALID_ARG
    # commit: null accepted, bad dtype
    assert lib.treewy_commit(vp(A), vp(A), vp(A), ctypes.byref(t), 2, None, tw.TREEWY_BF16, None, None,
                             None) == tw.TREEWY_ERR_INVALID_ARG
    assert lib.treewy_commit(vp(A), vp(A), vp(A), ctypes.byref(t), 2, vp(A), 9, None, None,
                             None) == tw.TREEWY_ERR_UNSUPPORTED
    # empty batches are accepted without touching anything
    t = _tree(tw, B=0, T=0)
    assert lib.treewy_verify(*ok_args(t)) == tw.TREEWY_OK
    assert lib.treewy_commit(None, None, None, ctypes.byref(t), 2, None, tw.TREEWY_BF16, None, None,
                             None) == tw.TREEWY_OK


def test_missing_library_fails_loudly(tw, tmp_path):
    with pytest.raises(ImportError):
        tw.load_library(str(tmp_path / "libtreewy.so"))
    tw.load_library(tw.LIB_PATH)
