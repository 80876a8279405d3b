"""The full-state-snapshotting comparator: every node's state, against the oracle's snapshots and
against treewy_commit (the accepted node's snapshot IS the committed state, bit for bit)."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cid,kw", [(2, dict(B=4, H_v=4)), (4, dict(B=12, H_v=2, prefix_tokens=16)),
                                    (3, dict(B=2, H_v=2))])
def test_snapshots_match_oracle_and_commit(oracle, cid, kw):
    from paper_2608_20961_b200 import binding as tw
    w = wl.make_workload(cid, **kw)
    dev = torch.device("cuda:0")
    d = lambda t: t.to(dev)
    tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, w.max_nodes)
    S0, q, k, v = d(w.S0), d(w.q), d(w.k), d(w.v)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    O = torch.empty((w.T, w.H_v, 128), dtype=torch.float32, device=dev)
    U = torch.empty((w.T, w.H_v, 128), dtype=torch.float32, device=dev)
    Snap = torch.full((w.T, w.H_v, 128, 128), 3.0, dtype=torch.bfloat16, device=dev)
    tw.treewy_tree_prepare(tree, d(w.alpha), status)
    tw.treewy_verify(S0, q, k, v, d(w.beta), tree, w.H_qk, O, U, status)
    S_before = S0.clone()
    tw.treewy_snapshot_all(S0, U, k, tree, w.H_qk, Snap, status)
    torch.cuda.synchronize()
    assert not status.any() and torch.equal(S0, S_before)          # out of place

    _, ref = pu.run_oracle(oracle, w, want_snapshots=True)
    got = Snap.cpu().double().numpy()
    for t in range(w.T):
        for h in range(w.H_v):
            m, f = pu.unit_errors(got[t, h], ref.Snap[t, h])
            assert f <= pu.FROB_GATE, (t, h, m, f)

    # commit of the accepted node == that node's snapshot
    tw.treewy_commit(S0, U, k, tree, w.H_qk, d(w.accepted), None, status)
    torch.cuda.synchronize()
    off = w.node_offsets.tolist()
    for b in range(w.B):
        a = int(w.accepted[b])
        assert torch.equal(S0[b], Snap[off[b] + a])


def test_snapshot_argument_checks():
    import ctypes
    from paper_2608_20961_b200 import binding as tw
    lib = tw.load_library()
    A = 0x1000
    t = tw.TreeStruct(B=1, T=4, H_v=2, max_nodes=0, node_offsets=A, parent=A, depth=A, anc_mask=A,
                      cum_log_gate=A, level_order=A)
    vp = ctypes.c_void_p
    assert lib.treewy_snapshot_all(vp(A), vp(A), vp(A), ctypes.byref(t), 2, tw.TREEWY_F32, vp(A), None,
                                   None) == tw.TREEWY_ERR_UNSUPPORTED
    assert lib.treewy_snapshot_all(vp(A), vp(A), vp(A), ctypes.byref(t), 2, tw.TREEWY_BF16, None, None,
                                   None) == tw.TREEWY_ERR_INVALID_ARG
