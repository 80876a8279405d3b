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


def test_commit_verify_checks_both_halves_before_it_launches_anything(tw):
    """The two-kernel form of treewy_commit_verify must not have committed when the verify half is going
    to be rejected: with no GPU here a launch would show up as TREEWY_ERR_CUDA, a clean rejection as
    TREEWY_ERR_INVALID_ARG / TREEWY_ERR_UNSUPPORTED."""
    lib = tw.load_library()
    vp = ctypes.c_void_p
    tp, t = _tree(tw), _tree(tw)

    def call(q=vp(A), o_dtype=tw.TREEWY_BF16, O=vp(A), single=0, tree=t, pool=None):
        args = [vp(A), vp(A), ctypes.byref(tp), vp(A), q, vp(A), vp(A), vp(A), ctypes.byref(tree), 2,
                tw.TREEWY_BF16, o_dtype, O, vp(A), single, None, None]
        if pool is not None:
            return lib.treewy_commit_verify_pool(ctypes.byref(pool), *args)
        return lib.treewy_commit_verify(vp(A), *args)

    for single in (0, 1):
        assert call(q=None, single=single) == tw.TREEWY_ERR_INVALID_ARG
        assert call(O=vp(A + 2), single=single) == tw.TREEWY_ERR_INVALID_ARG
        assert call(o_dtype=5, single=single) == tw.TREEWY_ERR_UNSUPPORTED
        assert call(tree=_tree(tw, B=3), single=single) == tw.TREEWY_ERR_INVALID_ARG   # B differs between the rounds
    pool = tw.PoolStruct(A, A, 4)
    assert call(q=None, pool=pool) == tw.TREEWY_ERR_INVALID_ARG


def test_debug_hook_is_exported_and_resets(tw):
    tw.treewy_debug_inject(1000, 3)
    tw.treewy_debug_inject(0, -1)


def test_missing_library_fails_loudly(tw, tmp_path):
    with pytest.raises(ImportError):
        tw.load_library(str(tmp_path / "libtreewy.so"))
    tw.load_library(tw.LIB_PATH)
