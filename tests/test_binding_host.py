"""Host-side behaviour of the Python binding that needs no GPU: marshalled ("prebound") calls replay
the C call with the same arguments and report the same error codes, recording does not nest, and the
status bits the binding names are the header's."""
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tw():
    from paper_2608_20961_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _empty_tree(tw, B=0):
    off = torch.zeros(B + 1, dtype=torch.int32)
    par = torch.zeros(0, dtype=torch.int32)
    return tw.Tree.empty(off, par, H_v=4, max_nodes=0)


def test_prebound_replays_the_call_and_its_status(tw):
    tree = _empty_tree(tw)                      # B = 0: valid, nothing to launch, so it runs without a GPU
    alpha = torch.zeros((1, 4), dtype=torch.float32)

    class FakeStream:                           # (no CUDA here: any object with a cuda_stream handle)
        cuda_stream = 0
    call = tw.prebound(tw.treewy_tree_prepare, tree, alpha, None, FakeStream())
    call()
    call()                                      # replays; TREEWY_OK both times
    bad = _empty_tree(tw)
    bad.H_v = 0                                 # host-checkable misuse: the replay raises like the call
    with pytest.raises(tw.TreewyError) as e:
        tw.prebound(tw.treewy_tree_prepare, bad, alpha, None, FakeStream())()
    assert e.value.code == tw.TREEWY_ERR_INVALID_ARG


def test_prebound_records_every_call_of_a_composite_and_does_not_nest(tw):
    tree = _empty_tree(tw)
    alpha = torch.zeros((1, 4), dtype=torch.float32)

    class FakeStream:
        cuda_stream = 0

    def two_calls():
        tw.treewy_tree_prepare(tree, alpha, None, FakeStream())
        tw.treewy_tree_prepare_log(tree, alpha, None, FakeStream())
    call = tw.prebound(two_calls)
    assert [c[0] for c in call._calls] == ["treewy_tree_prepare", "treewy_tree_prepare_log"]
    call()
    with pytest.raises(AssertionError):
        tw.prebound(lambda: tw.prebound(two_calls))
    tw.prebound(two_calls)()                    # a failed recording leaves the module usable


def test_status_bits_match_the_header(tw):
    text = open(os.path.join(ROOT, "include", "treewy.h")).read()
    bits = dict(re.findall(r"TREEWY_SEQ_(\w+) = (\d+)", text))
    assert {k: int(v) for k, v in bits.items()} == {
        "BAD_PARENT": tw.SEQ_BAD_PARENT, "TOO_MANY_NODES": tw.SEQ_TOO_MANY_NODES,
        "BAD_ACCEPTED": tw.SEQ_BAD_ACCEPTED, "TIMEOUT": tw.SEQ_TIMEOUT, "BAD_STATE": tw.SEQ_BAD_STATE,
        "BAD_OFFSETS": tw.SEQ_BAD_OFFSETS}
