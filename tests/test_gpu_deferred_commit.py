"""Deferred state write over several rounds (the periodic-flush form of reconstruct-on-commit, Section 3,
Eq. 3; the paper's ReplaySSM appendix names deferring the state write as the lever): the committed
state stays as it is for m rounds, the accepted paths of the rounds in between are carried as a chain
in front of every new draft tree, and ONE commit over the concatenated path writes the state.

The library needs nothing new for this: a tree whose first nodes are the carried path (a chain) and
whose draft nodes hang off its end is an ordinary tree, its verify from the old state gives the draft
nodes' outputs, and its commit at the accepted draft node is Eq. 3 over the concatenated accepted
paths.  Checked here over two and three rounds: against the oracle on the extended tree (same
arithmetic, tight gate) and against the oracle run round by round with a state committed every round
and never rounded in between (Eq. 3 over the concatenated path IS the chain of per-round commits).
With the kernels as they are this form is a correctness statement, not a faster path: the carried
nodes push a tree into the next larger kernel instance."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import _custom

pytestmark = pytest.mark.gpu


def _path(tree, a):
    p = []
    while a >= 0:
        p.append(a)
        a = tree[a]
    return p[::-1]


def _extend(w_rounds, trees_rounds, accepted_rounds):
    """Round r's trees with the accepted paths of rounds 0..r-1 carried in front of them as a chain.
    Returns the extended workload of the last round and, per sequence, how many carried nodes it has."""
    last = len(w_rounds) - 1
    wl_last = w_rounds[last]
    B = wl_last.B
    rows = {name: [] for name in ("q", "k", "v", "alpha", "beta")}
    trees, carried = [], []
    for b in range(B):
        ext, n_carried = [], 0
        for r in range(last):
            w, off = w_rounds[r], w_rounds[r].node_offsets.tolist()
            for j in _path(trees_rounds[r][b], accepted_rounds[r][b]):
                for name in rows:
                    rows[name].append(getattr(w, name)[off[b] + j])
                ext.append(n_carried - 1)          # a chain: every carried node hangs off the one before
                n_carried += 1
        off = wl_last.node_offsets.tolist()
        for i, p in enumerate(trees_rounds[last][b]):
            for name in rows:
                rows[name].append(getattr(wl_last, name)[off[b] + i])
            ext.append(p + n_carried if p >= 0 else n_carried - 1)
        trees.append(ext)
        carried.append(n_carried)
    offs = [0]
    for t in trees:
        offs.append(offs[-1] + len(t))
    acc = [accepted_rounds[last][b] + carried[b] for b in range(B)]
    w0 = w_rounds[0]
    ext_w = wl.Workload(name="deferred", config_id=-1, B=B, H_v=w0.H_v, H_qk=w0.H_qk, io_dtype=w0.io_dtype,
                        node_offsets=torch.tensor(offs, dtype=torch.int32),
                        parent=torch.tensor([p for t in trees for p in t], dtype=torch.int32),
                        q=torch.stack(rows["q"]), k=torch.stack(rows["k"]), v=torch.stack(rows["v"]),
                        alpha=torch.stack(rows["alpha"]), beta=torch.stack(rows["beta"]), S0=w0.S0,
                        accepted=torch.tensor(acc, dtype=torch.int32))
    return ext_w, carried


@pytest.mark.parametrize("n_rounds", [2, 3])
def test_one_commit_over_the_concatenated_paths_equals_a_commit_every_round(oracle, n_rounds):
    g = torch.Generator().manual_seed(40 + n_rounds)
    B, H_v, H_qk = 5, 4, 2
    trees_rounds = [[wl.random_parent_tree(g, 12 + 4 * r, 4) for _ in range(B)] for r in range(n_rounds)]
    accepted_rounds = [[int(torch.randint(0, len(t), (1,), generator=g)) for t in trees] for trees in trees_rounds]
    w_rounds = [_custom(trees_rounds[r], H_v=H_v, H_qk=H_qk, seed=60 + r, accepted=accepted_rounds[r])
                for r in range(n_rounds)]
    ext, carried = _extend(w_rounds, trees_rounds, accepted_rounds)
    assert ext.max_nodes <= 64

    # the library on the extended trees, from the OLD state: one verify, one commit
    gpu = pu.run_gpu(ext, torch.float32, max_nodes=64)
    assert not gpu["status"].any()
    tree_ref, ref = pu.run_oracle(oracle, ext)
    pu.assert_parity(ext, gpu, tree_ref, ref)

    # the oracle round by round, the state committed after every round (fp64, never rounded in between)
    S = pu.f64(w_rounds[0].S0)
    for r, w in enumerate(w_rounds):
        res = oracle.verify_commit(w.node_offsets.numpy(), w.parent.numpy(), S, pu.f64(w.q), pu.f64(w.k), pu.f64(w.v),
                                   pu.f64(w.alpha), pu.f64(w.beta), w.accepted.numpy())
        assert not res.seq_status.any()
        S = res.S_commit
    O_last = res.O                                   # the last round's outputs, from the state before it
    # draft rows of the extended verify = the last round's outputs; the one commit = the chain of commits
    eoff, loff = ext.node_offsets.tolist(), w_rounds[-1].node_offsets.tolist()
    O_gpu = gpu["O"].double().numpy()
    for b in range(B):
        got = O_gpu[eoff[b] + carried[b]:eoff[b + 1]]
        want = O_last[loff[b]:loff[b + 1]]
        for h in range(H_v):
            m, f = pu.unit_errors(got[:, h], want[:, h])
            assert m <= pu.ARITH_MAXABS and f <= pu.ARITH_FROB, ("O", b, h, m, f)
    m, f = pu.worst_errors(gpu["S32"].double().numpy(), S, np.arange(B + 1), False)
    assert m <= pu.ARITH_MAXABS and f <= pu.ARITH_FROB, ("S", m, f)
