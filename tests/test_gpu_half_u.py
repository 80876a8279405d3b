"""16-bit pseudo-values: treewy_verify_half_u writes U as fp16, treewy_commit_half_u reads it.
Every u is formed exactly as in treewy_verify and rounded once on the store, so U16 must equal
RNE(U32) bit for bit and O must not change; the commit must do with the widened values exactly what
treewy_commit does; and the committed state must still meet the parity gates against the oracle."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import _custom

pytestmark = pytest.mark.gpu


def _run(w, max_nodes, half):
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    d = lambda t: t.to(dev)
    tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, max_nodes)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    S = d(w.S0).clone()
    q, k, v, beta, acc = d(w.q), d(w.k), d(w.v), d(w.beta), d(w.accepted)
    O = torch.full((w.T, w.H_v, 128), 3.0, dtype=torch.float32, device=dev)
    U = torch.full((w.T, w.H_v, 128), 3.0, dtype=torch.float16 if half else torch.float32, device=dev)
    S32 = torch.zeros(S.shape, dtype=torch.float32, device=dev)
    tw.treewy_tree_prepare(tree, d(w.alpha), status)
    if half:
        tw.treewy_verify_half_u(S, q, k, v, beta, tree, w.H_qk, O, U, status)
        tw.treewy_commit_half_u(S, U, k, tree, w.H_qk, acc, S32, status)
    else:
        tw.treewy_verify(S, q, k, v, beta, tree, w.H_qk, O, U, status)
        # the reference for the commit: the stand-alone commit fed the widened fp16 values
        tw.treewy_commit(S, U.half().float(), k, tree, w.H_qk, acc, S32, status)
    torch.cuda.synchronize()
    return S.cpu(), S32.cpu(), O.cpu(), U.cpu(), status.cpu()


CASES = [
    ("tree32", lambda: wl.make_workload(2, B=5, H_v=4, seed=71), 32),
    ("chain5-small-kernel", lambda: wl.make_workload(1, B=5, H_v=4, seed=72), 5),
    ("wide64", lambda: wl.make_workload(3, B=3, H_v=2, seed=73), 64),
    ("ragged", lambda: wl.make_workload(4, B=9, H_v=2, seed=74, prefix_tokens=16), 64),
    ("fp32-inputs", lambda: wl.make_workload(2, B=3, H_v=2, seed=75, io_dtype=torch.float32), 32),
]


@pytest.mark.parametrize("name,make,hint", CASES, ids=[c[0] for c in CASES])
def test_half_u_is_the_rounded_u_and_commit_follows(oracle, name, make, hint):
    w = make()
    S, S32, O, U, st = _run(w, hint, half=False)
    Sh, S32h, Oh, Uh, sth = _run(w, hint, half=True)
    assert not st.any() and not sth.any()
    assert torch.equal(Oh, O), "O must not depend on how U is stored"
    assert torch.equal(Uh, U.half()), "U16 = RNE(U32)"
    assert torch.equal(Sh, S) and torch.equal(S32h, S32), "commit of fp16 U = commit of the widened values"
    # against the oracle: the committed state built from 16-bit pseudo-values still meets the gates
    _, ref = pu.run_oracle(oracle, w)
    worst_m, worst_f = pu.worst_errors(S32h.double().numpy(), ref.S_commit, w.node_offsets.numpy(), per_node=False)
    print(f"{name}: committed state from fp16 U: max-abs/rms {worst_m:.2e}, rel. Frobenius {worst_f:.2e}")
    assert worst_m <= 2e-2 and worst_f <= 5e-3


def test_half_u_leaves_skipped_sequences_alone():
    from paper_2608_20961_b200 import binding as tw
    w = _custom([[-1, 0, 0, 2], [-1, 2, 0], [-1, 0]], H_v=2, H_qk=2, accepted=[3, 1, 7])
    S, S32, O, U, st = _run(w, 32, half=True)
    assert list(st) == [0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED]
    off = w.node_offsets.tolist()
    assert torch.all(U[off[1]:off[2]] == 3.0) and torch.all(O[off[1]:off[2]] == 3.0)
    assert torch.equal(S[1], w.S0[1]) and torch.equal(S[2], w.S0[2])
    assert not torch.equal(S[0], w.S0[0])
