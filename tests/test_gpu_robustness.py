"""Data-dependent misuse and the give-up path, on the GPU, without a fault.

* node_offsets that leave the T packed nodes the caller declared (a stale or non-monotone offsets
  array): the sequence is flagged TREEWY_SEQ_BAD_OFFSETS and skipped by every kernel before any of its
  rows is addressed.  All buffers here are allocated for the true node count, so nothing could leave
  its allocation either way; what is asserted is the flag, the untouched rows and states of the
  flagged sequences, and bit-identical results for all the others.
* a wait that runs out: with the test hook a kernel's bounded waits get a limit of about a
  millisecond and one item's loads are never issued (nothing is left in flight for it).  Every role
  must leave its loop, TREEWY_SEQ_TIMEOUT must be raised, the call must return, and the next ordinary
  call on the same stream must give the right answer.  No trap, no bad address, no endless loop.
"""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import _custom

pytestmark = pytest.mark.gpu

CANARY = 7.25


def _run(w, path, T_decl=None, offsets=None, hint=0):
    """prepare -> verify -> commit of workload w through one family of kernels, with the tree
    declaring T_decl packed nodes (default: all) and, optionally, other node offsets."""
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    d = lambda t: t.to(dev)
    off = d(w.node_offsets if offsets is None else torch.tensor(offsets, dtype=torch.int32))
    tree = tw.Tree.empty(off, d(w.parent), w.H_v, hint)
    tree.depth.fill_(-7)
    if T_decl is not None:
        tree.T = T_decl
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    q, k, v, S = d(w.q), d(w.k), d(w.v), d(w.S0).clone()
    O = torch.full((w.T, w.H_v, 128), CANARY, dtype=torch.float32, device=dev)
    U = torch.full((w.T, w.H_v, 128), CANARY, dtype=torch.float32, device=dev)
    alpha, beta, acc = d(w.alpha), d(w.beta), d(w.accepted)
    if path == "wide":
        tw.treewy_tree_prepare_wide(tree, alpha, status)
        tw.treewy_verify_wide(S, q, k, v, beta, tree, w.H_qk, O, U, status)
        tw.treewy_commit_wide(S, U, k, tree, w.H_qk, acc, None, status)
    else:
        tw.treewy_tree_prepare(tree, alpha, status)
        tw.treewy_verify(S, q, k, v, beta, tree, w.H_qk, O, U, status, generic=(path == "generic"))
        tw.treewy_commit(S, U, k, tree, w.H_qk, acc, None, status)
    torch.cuda.synchronize()
    return dict(O=O.cpu(), U=U.cpu(), S=S.cpu(), status=status.cpu().numpy(), depth=tree.depth.cpu())


PATHS = {
    # name: (workload, keyword arguments, max_nodes hint)
    "generic": (0, dict(B=6, H_v=2), 0),            # fp32 inputs: SIMT verify and commit
    "small": (1, dict(B=6, H_v=4), 8),              # bf16, the small-tree kernel
    "np16": (1, dict(B=6, H_v=4), 16),              # role pipeline, 16-node instance
    "np32": (2, dict(B=6, H_v=4), 32),              # ... 32-node instance
    "np64": (3, dict(B=5, H_v=2), 64),              # ... both size classes
    "mixed": (4, dict(B=12, H_v=2, prefix_tokens=8), 64),
    "wide": (6, dict(B=4, H_v=2), 128),
}


@pytest.mark.parametrize("name", sorted(PATHS))
def test_offsets_past_the_declared_node_count_are_flagged_and_skipped(oracle, name):
    from paper_2608_20961_b200 import binding as tw
    cid, kw, hint = PATHS[name]
    w = wl.make_workload(cid, **kw)
    path = name if name in ("generic", "wide") else "main"
    good = _run(w, path, hint=hint)
    assert not good["status"].any()
    off = w.node_offsets.tolist()
    cut = w.B - 2
    T_decl = off[cut] + 1 if off[cut + 1] - off[cut] > 1 else off[cut]   # sequence `cut` sticks out (or starts at the end)
    got = _run(w, path, T_decl=T_decl, hint=hint)
    bad = [b for b in range(w.B) if off[b + 1] > T_decl]
    assert bad and bad[0] >= cut
    # the oracle restates the rule: same status words
    oracle.set_max_nodes(128 if name == "wide" else 64)
    try:
        ref = oracle.verify_commit(w.node_offsets.numpy(), w.parent.numpy(), pu.f64(w.S0), pu.f64(w.q), pu.f64(w.k),
                                   pu.f64(w.v), pu.f64(w.alpha), pu.f64(w.beta), w.accepted.numpy(), T_declared=T_decl)
    finally:
        oracle.set_max_nodes(64)
    assert list(ref.seq_status) == list(got["status"])
    for b in range(w.B):
        sl = slice(off[b], off[b + 1])
        if b in bad:
            assert got["status"][b] == tw.SEQ_BAD_OFFSETS, (b, got["status"])
            assert torch.all(got["O"][sl] == CANARY) and torch.all(got["U"][sl] == CANARY)
            assert torch.all(got["depth"][sl] == -7)
            assert torch.equal(got["S"][b], w.S0[b])
        else:
            assert got["status"][b] == 0
            assert torch.equal(got["O"][sl], good["O"][sl]) and torch.equal(got["U"][sl], good["U"][sl])
            assert torch.equal(got["S"][b], good["S"][b])


@pytest.mark.parametrize("path,hint", [("generic", 0), ("main", 32), ("main", 64), ("wide", 128)])
def test_negative_and_decreasing_offsets_are_flagged_and_skipped(path, hint):
    from paper_2608_20961_b200 import binding as tw
    g = torch.Generator().manual_seed(3)
    trees = [wl.random_parent_tree(g, 20, 5) for _ in range(5)]
    w = _custom(trees, H_v=2, H_qk=1, seed=4, accepted=[3, 19, 0, 7, 11])
    good = _run(w, path, hint=hint)
    off = w.node_offsets.tolist()                 # 0 20 40 60 80 100
    broken = list(off)
    broken[0] = -20                               # sequence 0: starts before the arrays (40 "nodes")
    broken[3] = 30                                # sequence 2 runs backwards (40 -> 30); sequence 3 = [30, 80)
    got = _run(w, path, offsets=broken, hint=hint)
    # sequences 1 and 4 are intact; 0 and 2 have ranges outside 0..T / of negative length; 3 is a range
    # inside the arrays but of 50 nodes with parents that are not a tree of that size (or too many nodes)
    assert got["status"][0] == tw.SEQ_BAD_OFFSETS and got["status"][2] == tw.SEQ_BAD_OFFSETS
    assert got["status"][1] == 0 and got["status"][4] == 0
    assert got["status"][3] != 0
    for b in (1, 4):
        sl = slice(off[b], off[b + 1])
        assert torch.equal(got["O"][sl], good["O"][sl]) and torch.equal(got["U"][sl], good["U"][sl])
        assert torch.equal(got["S"][b], good["S"][b])
    for b in (0, 2):
        assert torch.equal(got["S"][b], w.S0[b])
    assert torch.all(got["O"][0:20] == CANARY) and torch.all(got["U"][0:20] == CANARY)


def test_fused_round_checks_both_rounds_offsets():
    """treewy_commit_verify(single_kernel=1): a previous-round range past its T stops that sequence's
    commit, a new-round range past its T stops its verify; the other sequences are as without."""
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    d = lambda t: t.to(dev)
    for cid, kw, hint in ((2, dict(B=6, H_v=4), 32), (1, dict(B=6, H_v=4), 8)):
        w1, w2 = wl.make_workload(cid, seed=11, **kw), wl.make_workload(cid, seed=12, **kw)

        def rounds(T1=None, T2=None):
            S = d(w1.S0).clone()
            status = torch.zeros(w1.B, dtype=torch.int32, device=dev)
            t1 = tw.Tree.empty(d(w1.node_offsets), d(w1.parent), w1.H_v, hint)
            t2 = tw.Tree.empty(d(w2.node_offsets), d(w2.parent), w2.H_v, hint)
            U1 = torch.empty((w1.T, w1.H_v, 128), dtype=torch.float32, device=dev)
            O1 = torch.empty((w1.T, w1.H_v, 128), dtype=torch.float32, device=dev)
            O2 = torch.full((w2.T, w2.H_v, 128), CANARY, dtype=torch.float32, device=dev)
            U2 = torch.full((w2.T, w2.H_v, 128), CANARY, dtype=torch.float32, device=dev)
            k1 = d(w1.k)
            tw.treewy_tree_prepare(t1, d(w1.alpha), status)
            tw.treewy_verify(S, d(w1.q), k1, d(w1.v), d(w1.beta), t1, w1.H_qk, O1, U1, status)
            tw.treewy_tree_prepare(t2, d(w2.alpha), status)
            if T1 is not None:
                t1.T = T1
            if T2 is not None:
                t2.T = T2
            tw.treewy_commit_verify(S, U1, k1, t1, d(w1.accepted), d(w2.q), d(w2.k), d(w2.v), d(w2.beta), t2,
                                    w2.H_qk, O2, U2, True, status)
            torch.cuda.synchronize()
            return S.cpu(), O2.cpu(), U2.cpu(), status.cpu().numpy()

        S0g, Og, Ug, sg = rounds()
        assert not sg.any()
        off1, off2 = w1.node_offsets.tolist(), w2.node_offsets.tolist()
        S1, O1_, U1_, s1 = rounds(T1=off1[-2])       # last sequence of the previous round is out of range
        assert list(s1[:-1]) == [0] * (w1.B - 1) and s1[-1] == tw.SEQ_BAD_OFFSETS
        assert torch.equal(S1[-1], w1.S0[-1])        # not committed ...
        assert torch.equal(S1[:-1], S0g[:-1]) and torch.equal(O1_[:off2[-2]], Og[:off2[-2]])
        S2, O2_, U2_, s2 = rounds(T2=off2[-2])       # last sequence of the new round is out of range
        assert list(s2[:-1]) == [0] * (w1.B - 1) and s2[-1] == tw.SEQ_BAD_OFFSETS
        assert torch.equal(S2, S0g)                  # every commit happened
        assert torch.all(O2_[off2[-2]:] == CANARY) and torch.all(U2_[off2[-2]:] == CANARY)
        assert torch.equal(O2_[:off2[-2]], Og[:off2[-2]]) and torch.equal(U2_[:off2[-2]], Ug[:off2[-2]])


@pytest.mark.parametrize("cid,kw,hint,skip", [(2, dict(B=40, H_v=8, H_qk=8), 32, 200),
                                               (2, dict(B=40, H_v=8, H_qk=4), 32, 201),
                                               (3, dict(B=30, H_v=8), 64, 170)])
def test_a_wait_that_runs_out_raises_timeout_and_leaves_the_stream_usable(oracle, cid, kw, hint, skip):
    from paper_2608_20961_b200 import binding as tw
    w = wl.make_workload(cid, **kw)
    tree_ref, ref = pu.run_oracle(oracle, w)
    dev = torch.device("cuda:0")
    try:
        tw.treewy_debug_inject(2_000_000, skip)      # about a millisecond of SM clocks
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        gpu = pu.run_gpu(w, torch.float32, max_nodes=hint, want_s32=False)
        t1.record()
        torch.cuda.synchronize(dev)
    finally:
        tw.treewy_debug_inject(0, -1)
    assert t0.elapsed_time(t1) < 2000.0             # one deadline per kernel, not one per waiting role
    assert (gpu["status"] & tw.SEQ_TIMEOUT).any()
    assert not (gpu["status"] & ~tw.SEQ_TIMEOUT).any()
    # the context is intact and the next ordinary call is right
    gpu = pu.run_gpu(w, torch.float32, max_nodes=hint)
    assert not gpu["status"].any()
    pu.assert_parity(w, gpu, tree_ref, ref)
