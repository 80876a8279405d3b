"""treewy_commit_verify (commit of round r fused into verify of round r+1) must give what
treewy_commit followed by treewy_verify gives -- state, outputs, pseudo-values and status.  The
single-kernel mode forms the rank-P update on the tensor cores (fp32 split into two tf32 parts,
2^-22 relative), so the stored bf16 state may differ from the stand-alone commit's by one rounding
step in a few elements; everything that is not floating point must be identical."""
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests.test_gpu_parity import _custom

pytestmark = pytest.mark.gpu


def _device_round(tw, w, dev, max_nodes):
    d = lambda t: t.to(dev)
    tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, max_nodes)
    r = dict(tree=tree, q=d(w.q), k=d(w.k), v=d(w.v), alpha=d(w.alpha), beta=d(w.beta),
             acc=d(w.accepted),
             O=torch.full((w.T, w.H_v, 128), 5.0, dtype=torch.bfloat16, device=dev),
             U=torch.full((w.T, w.H_v, 128), 5.0, dtype=torch.float32, device=dev))
    return r


def _two_rounds(w1, w2, fused, hint1, hint2):
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    S = w1.S0.to(dev).clone()
    status = torch.zeros(w1.B, dtype=torch.int32, device=dev)
    r1, r2 = _device_round(tw, w1, dev, hint1), _device_round(tw, w2, dev, hint2)
    tw.treewy_tree_prepare(r1["tree"], r1["alpha"], status)
    tw.treewy_verify(S, r1["q"], r1["k"], r1["v"], r1["beta"], r1["tree"], w1.H_qk, r1["O"], r1["U"], status)
    status.zero_()
    tw.treewy_tree_prepare(r2["tree"], r2["alpha"], status)
    if fused:
        tw.treewy_commit_verify(S, r1["U"], r1["k"], r1["tree"], r1["acc"], r2["q"], r2["k"], r2["v"],
                                r2["beta"], r2["tree"], w2.H_qk, r2["O"], r2["U"], True, status)
    else:
        tw.treewy_commit(S, r1["U"], r1["k"], r1["tree"], w1.H_qk, r1["acc"], None, status)
        tw.treewy_verify(S, r2["q"], r2["k"], r2["v"], r2["beta"], r2["tree"], w2.H_qk, r2["O"], r2["U"], status)
    torch.cuda.synchronize()
    return S.cpu(), r2["O"].cpu(), r2["U"].cpu(), status.cpu()


def _check(w1, w2, hint1, hint2):
    a = _two_rounds(w1, w2, False, hint1, hint2)
    b = _two_rounds(w1, w2, True, hint1, hint2)
    (Sa, Oa, Ua, sa), (Sb, Ob, Ub, sb) = a, b
    assert torch.equal(sa, sb), "status"
    Sa32, Sb32 = Sa.float(), Sb.float()
    diff = (Sa32 - Sb32).abs()
    floor = 1e-6 * float(Sa32.abs().max())   # results of cancellations: absolute, not relative, agreement
    assert not bool((diff > 2.0 ** -7 * Sa32.abs() + floor).any()), "S: more than one bf16 step apart"
    assert float((diff > 0).float().mean()) < 2e-3, "S: too many elements differ"
    untouched = (Ua == 5.0)
    assert torch.equal(untouched, Ub == 5.0), "rows written"
    for x, y, name in ((Oa.float(), Ob.float(), "O"), (Ua, Ub, "U")):
        scale = float(x[~untouched if name == "U" else slice(None)].abs().max()) if x.numel() else 1.0
        assert float((x - y).abs().max()) <= 2.0 ** -6 * scale, name
    return a


@pytest.mark.parametrize("cid,kw", [(2, dict(B=9, H_v=4)), (1, dict(B=5, H_v=8)), (5, dict(B=3, H_v=4))])
def test_fused_equals_commit_then_verify(cid, kw):
    w1 = wl.make_workload(cid, seed=11, **kw)
    w2 = wl.make_workload(cid, seed=12, **kw)
    hint = 32 if w1.max_nodes <= 32 else 64
    S, O, U, status = _check(w1, w2, hint, hint)
    assert not status.any() and not torch.equal(S, w1.S0)      # something was committed


def test_fused_with_ragged_rounds_and_edge_cases():
    from paper_2608_20961_b200 import binding as tw
    chain40 = [i - 1 for i in range(40)]                     # previous round: a path deeper than 16
    prev = [chain40, [-1, 0, 0, 2], [-1], [-1, 0, 1], [-1, 0], [-1, 0, 1, 1]]
    new = [[-1, 0, 1, 1, 0], [-1] + [0] * 20, [-1, 2, 0], [i - 1 for i in range(32)], [-1], [-1, 0]]
    #       ok                ok              malformed     ok (deep chain)             ok    ok
    w1 = _custom(prev, H_v=4, H_qk=2, seed=3, accepted=[39, 3, -1, 7, 1, 2])   # seq 3: accepted out of range
    w2 = _custom(new, H_v=4, H_qk=2, seed=4)
    w2.S0 = w1.S0
    S, O, U, status = _check(w1, w2, 64, 32)
    assert list(status) == [0, 0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED, 0, 0]
    assert torch.equal(S[2], w1.S0[2]) and torch.equal(S[3], w1.S0[3])     # nothing committed there
    assert not torch.equal(S[0], w1.S0[0])                                  # the deep path was committed
    off = w2.node_offsets.tolist()
    assert torch.all(U[off[2]:off[3]] == 5.0)                                # malformed tree: rows untouched
    # sequence 4: commit happened although ... and verify ran on the committed state
    assert not torch.equal(S[4], w1.S0[4])


def test_fused_falls_back_for_large_new_trees():
    w1 = wl.make_workload(2, B=3, H_v=4, seed=21)
    w2 = wl.make_workload(3, B=3, H_v=4, seed=22)
    w2.S0 = w1.S0
    w2.H_qk = w1.H_qk
    w2.q, w2.k = w2.q[:, :w1.H_qk].contiguous(), w2.k[:, :w1.H_qk].contiguous()
    _check(w1, w2, 32, 64)


def test_fused_round_matches_the_oracle(oracle):
    """Two rounds against the oracle itself (not against the two-kernel path): round 1 is verified
    and committed by the oracle, its committed state -- rounded to the bf16 the library stores --
    starts the oracle's round 2; the GPU runs verify(1), then commit(1) + verify(2) in ONE kernel."""
    import numpy as np
    from tests import parity_util as pu
    w1 = wl.make_workload(2, seed=31, B=6, H_v=4)
    w2 = wl.make_workload(2, seed=32, B=6, H_v=4)
    _, ref1 = pu.run_oracle(oracle, w1)
    w2.S0 = torch.from_numpy(ref1.S_commit).to(torch.bfloat16)
    _, ref2 = pu.run_oracle(oracle, w2)
    S, O, U, status = _two_rounds(w1, w2, True, 32, 32)
    assert not status.any()
    off = w2.node_offsets.numpy()
    for name, got, want, offs, per_node in (
            ("O", O.double().numpy(), ref2.O, off, True), ("U", U.double().numpy(), ref2.U, off, True),
            ("S", S.double().numpy(), ref1.S_commit, np.arange(w1.B + 1), False)):
        m, f = pu.worst_errors(got, want, offs, per_node)
        # (the stored state is bf16: its largest elements are off by up to 2^-9 of their own size, which
        # is why the max-abs gate is applied to the fp32 outputs and the Frobenius gate to all three)
        assert f <= pu.FROB_GATE and (name == "S" or m <= pu.MAXABS_GATE), (name, m, f)
    want = torch.from_numpy(ref1.S_commit).to(torch.bfloat16).float()
    assert not bool(((S.float() - want).abs() > 2.0 ** -7 * want.abs() + 1e-6 * float(want.abs().max())).any())
