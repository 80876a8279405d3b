"""Properties of verify + commit that hold whatever the inputs, checked on the GPU path itself
(they need no oracle): packing, head sharing, linearity, sub-tree independence."""
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _run(w, **kw):
    return pu.run_gpu(w, torch.float32, max_nodes=kw.pop("max_nodes", w.max_nodes), **kw)


@pytest.mark.parametrize("cid", [2, 4])
def test_ragged_packing_equals_per_sequence_calls(cid):
    w = wl.make_workload(cid, B=9, H_v=4, prefix_tokens=8)
    whole = _run(w, max_nodes=64)
    off = w.node_offsets.tolist()
    for b in range(w.B):
        one = _run(w.select_sequences([b]), max_nodes=64)
        sl = slice(off[b], off[b + 1])
        assert torch.equal(one["O"], whole["O"][sl]) and torch.equal(one["U"], whole["U"][sl])
        assert torch.equal(one["S"][0], whole["S"][b])


def test_shared_qk_heads_equal_replicated_heads():
    w = wl.make_workload(2, B=4, H_v=8, H_qk=2)
    shared = _run(w)
    rep = w.select_sequences(range(w.B))
    rep.q = w.q.repeat_interleave(4, dim=1).contiguous()
    rep.k = w.k.repeat_interleave(4, dim=1).contiguous()
    rep.H_qk = 8
    repl = _run(rep)
    assert torch.equal(shared["O"], repl["O"]) and torch.equal(shared["U"], repl["U"])
    assert torch.equal(shared["S"], repl["S"])


def test_joint_linearity_in_state_and_values():
    # O, U and the committed state are linear in (S0, V) jointly: scaling both by 2 (exact in
    # binary floating point) scales every output by exactly 2
    w = wl.make_workload(2, B=3, H_v=4)
    a = _run(w)
    w2 = w.select_sequences(range(w.B))
    w2.S0 = (w.S0.float() * 2).to(w.S0.dtype)
    w2.v = (w.v.float() * 2).to(w.v.dtype)
    b = _run(w2)
    assert torch.equal(b["O"], a["O"] * 2) and torch.equal(b["U"], a["U"] * 2)
    assert torch.equal(b["S32"], a["S32"] * 2)


def test_unrelated_branches_do_not_change_a_node():
    # a tree and the same tree with extra leaves appended: the common nodes' outputs agree to
    # fp32 rounding (the tensor-core tiles have different padding, the arithmetic is the same)
    w = wl.make_workload(2, B=1, H_v=2, H_qk=1)
    big = _run(w)
    keep = 20
    small = w.select_sequences([0])
    small.node_offsets = torch.tensor([0, keep], dtype=torch.int32)
    for name in ("parent", "q", "k", "v", "alpha", "beta"):
        setattr(small, name, getattr(w, name)[:keep].clone())
    small.accepted = torch.tensor([min(int(w.accepted[0]), keep - 1)], dtype=torch.int32)
    cut = _run(small)
    torch.testing.assert_close(cut["O"], big["O"][:keep], rtol=0, atol=2e-5)
    torch.testing.assert_close(cut["U"], big["U"][:keep], rtol=0, atol=2e-5)


@pytest.mark.parametrize("hint", [8, 32, 64])
def test_beta_zero_is_pure_decay_on_every_kernel(hint):
    """beta = 0 switches the delta rule off (the scalar-gate case): every pseudo-value is exactly 0,
    o_i = g_i S0 q_i, and the committed state is g_a S0.  One tree size per kernel: the small-tree
    kernel, the role pipeline's 32-node and 64-node instances, and the SIMT kernel beside each."""
    from tests.test_gpu_parity import _custom
    g = torch.Generator().manual_seed(hint)
    trees = [wl.random_parent_tree(g, hint, 6), [i - 1 for i in range(hint)], [-1]]
    w = _custom(trees, H_v=4, H_qk=2, seed=hint, accepted=[hint - 1, hint // 2, 0])
    w.beta[:] = 0.0
    for generic in (False, True):
        gpu = pu.run_gpu(w, torch.float32, max_nodes=hint, generic=generic)
        assert not gpu["status"].any()
        assert not gpu["U"].any(), "u_i = beta_i (...) = 0 exactly"
        # gates from the library's own prepare, so that only the kernels under test are compared
        L = torch.from_numpy(gpu["cum_log_gate"]).double()
        S0, q = w.S0.double(), w.q.double()
        off = w.node_offsets.tolist()
        for b in range(w.B):
            for h in range(w.H_v):
                rows = slice(off[b], off[b + 1])
                want = torch.exp(L[rows, h])[:, None] * (q[rows, h // 2] @ S0[b, h].T)
                torch.testing.assert_close(gpu["O"][rows, h].double(), want, rtol=0, atol=2e-5 * float(want.abs().max()))
                a = int(w.accepted[b])
                torch.testing.assert_close(gpu["S32"][b, h].double(), torch.exp(L[off[b] + a, h]) * S0[b, h],
                                           rtol=1e-6, atol=1e-9)
