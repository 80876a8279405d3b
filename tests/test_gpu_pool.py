"""Block-pool addressing of the states: treewy_verify_pool / treewy_commit_pool on states scattered in
a pool must give, bit for bit, what the plain calls give on the gathered states; blocks that no
sequence points to stay untouched; an index outside the pool flags the sequence and skips it."""
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run(w, dev, pool_index=None, n_states=None):
    from paper_2608_20961_b200 import binding as tw
    d = lambda t: t.to(dev)
    tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, w.max_nodes)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    q, k, v, beta, acc = d(w.q), d(w.k), d(w.v), d(w.beta), d(w.accepted)
    O = torch.full((w.T, w.H_v, 128), 3.0, dtype=torch.bfloat16, device=dev)
    U = torch.full((w.T, w.H_v, 128), 3.0, dtype=torch.float32, device=dev)
    tw.treewy_tree_prepare(tree, d(w.alpha), status)
    if pool_index is None:
        S = d(w.S0).clone()
        tw.treewy_verify(S, q, k, v, beta, tree, w.H_qk, O, U, status)
        tw.treewy_commit(S, U, k, tree, w.H_qk, acc, None, status)
    else:
        S = torch.full((n_states,) + tuple(w.S0.shape[1:]), 0.5, dtype=w.S0.dtype, device=dev)
        idx = pool_index.to(dev)
        ok = (pool_index >= 0) & (pool_index < n_states)
        S[idx[ok.to(dev)].long()] = d(w.S0)[ok.to(dev)]
        tw.treewy_verify_pool(S, idx, q, k, v, beta, tree, w.H_qk, O, U, status)
        tw.treewy_commit_pool(S, idx, U, k, tree, w.H_qk, acc, status)
    torch.cuda.synchronize()
    return S.cpu(), O.cpu(), U.cpu(), status.cpu()


@pytest.mark.parametrize("cid,dtype", [(2, torch.bfloat16), (4, torch.bfloat16), (2, torch.float32)])
def test_pool_calls_equal_plain_calls(cid, dtype):
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w = wl.make_workload(cid, B=7, H_v=4, seed=5, io_dtype=dtype)
    S_ref, O_ref, U_ref, st_ref = _run(w, dev)
    assert not st_ref.any()
    n_states = 11
    perm = torch.randperm(n_states, generator=torch.Generator().manual_seed(1))[: w.B].to(torch.int32)
    S, O, U, st = _run(w, dev, perm, n_states)
    assert not st.any()
    assert torch.equal(O, O_ref) and torch.equal(U, U_ref)
    assert torch.equal(S[perm.long()], S_ref)
    unused = sorted(set(range(n_states)) - set(perm.tolist()))
    assert torch.all(S[unused] == 0.5)
    # one index outside the pool: that sequence is flagged and skipped, the others are unaffected
    bad = perm.clone()
    bad[3] = n_states + 2
    S2, O2, U2, st2 = _run(w, dev, bad, n_states)
    assert list(st2) == [0, 0, 0, tw.SEQ_BAD_STATE, 0, 0, 0]
    off = w.node_offsets.tolist()
    assert torch.all(U2[off[3]:off[4]] == 3.0) and torch.all(O2[off[3]:off[4]] == 3.0)
    keep = [b for b in range(w.B) if b != 3]
    rows = [i for b in keep for i in range(off[b], off[b + 1])]
    assert torch.equal(U2[rows], U_ref[rows]) and torch.equal(S2[bad[keep].long()], S_ref[keep])


@pytest.mark.parametrize("single", [False, True])
def test_fused_round_on_a_pool_equals_the_plain_fused_round(single):
    """commit(r) + verify(r+1) with the states in a pool: bit for bit the plain call's result."""
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w1 = wl.make_workload(2, B=6, H_v=4, seed=41)
    w2 = wl.make_workload(2, B=6, H_v=4, seed=42)
    n_states = 9
    perm = torch.randperm(n_states, generator=torch.Generator().manual_seed(2))[: w1.B].to(torch.int32)

    def run(pool):
        d = lambda t: t.to(dev)
        status = torch.zeros(w1.B, dtype=torch.int32, device=dev)
        t1 = tw.Tree.empty(d(w1.node_offsets), d(w1.parent), w1.H_v, 32)
        t2 = tw.Tree.empty(d(w2.node_offsets), d(w2.parent), w2.H_v, 32)
        O1 = torch.empty((w1.T, w1.H_v, 128), dtype=torch.bfloat16, device=dev)
        U1 = torch.empty((w1.T, w1.H_v, 128), dtype=torch.float32, device=dev)
        O2 = torch.full((w2.T, w2.H_v, 128), 2.0, dtype=torch.bfloat16, device=dev)
        U2 = torch.full((w2.T, w2.H_v, 128), 2.0, dtype=torch.float32, device=dev)
        tw.treewy_tree_prepare(t1, d(w1.alpha), status)
        tw.treewy_tree_prepare(t2, d(w2.alpha), status)
        if pool:
            S = torch.full((n_states,) + tuple(w1.S0.shape[1:]), 0.25, dtype=w1.S0.dtype, device=dev)
            idx = perm.to(dev)
            S[idx.long()] = d(w1.S0)
            tw.treewy_verify_pool(S, idx, d(w1.q), d(w1.k), d(w1.v), d(w1.beta), t1, w1.H_qk, O1, U1, status)
            tw.treewy_commit_verify_pool(S, idx, U1, d(w1.k), t1, d(w1.accepted), d(w2.q), d(w2.k), d(w2.v),
                                         d(w2.beta), t2, w2.H_qk, O2, U2, single, status)
            torch.cuda.synchronize()
            assert torch.all(S[sorted(set(range(n_states)) - set(perm.tolist()))] == 0.25)
            S = S[idx.long()]
        else:
            S = d(w1.S0).clone()
            tw.treewy_verify(S, d(w1.q), d(w1.k), d(w1.v), d(w1.beta), t1, w1.H_qk, O1, U1, status)
            tw.treewy_commit_verify(S, U1, d(w1.k), t1, d(w1.accepted), d(w2.q), d(w2.k), d(w2.v), d(w2.beta), t2,
                                    w2.H_qk, O2, U2, single, status)
            torch.cuda.synchronize()
        return S.cpu(), O2.cpu(), U2.cpu(), status.cpu()

    a, b = run(False), run(True)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert not a[3].any()
