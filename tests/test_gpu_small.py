"""The small-tree kernel: batches whose trees have at most 8 nodes (the chain of a few drafts above
all) take one small CTA per (sequence, head) instead of the tensor-core pipeline.  It must match the
oracle like every other verify path, keep the status / skip semantics, and -- in the fused round --
store exactly the state the stand-alone commit stores."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import _custom
from tests.test_gpu_fused import _two_rounds

pytestmark = pytest.mark.gpu

CHAIN8 = [i - 1 for i in range(8)]
STAR8 = [-1] + [0] * 7
FOREST = [-1, -1, 0, 1, -1, 4, 5]
COMB = [-1, 0, 0, 1, 1, 3, 3, 5]
TREES = [CHAIN8, STAR8, FOREST, [-1], [-1, 0], COMB, CHAIN8[:5], [-1, 0, 0]]
ACCEPTED = [7, 3, 6, 0, -1, 7, 2, 1]


@pytest.mark.parametrize("H_v,H_qk", [(4, 2), (4, 4), (3, 1)])
def test_small_trees_match_the_oracle(oracle, H_v, H_qk):
    w = _custom(TREES, H_v=H_v, H_qk=H_qk, accepted=ACCEPTED, seed=5)
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, max_nodes=8)
    assert not gpu["status"].any()
    pu.assert_parity(w, gpu, tree_ref, ref)
    assert torch.equal(gpu["S"][4], w.S0[4])                    # accepted = -1
    gpu16 = pu.run_gpu(w, torch.bfloat16, max_nodes=8)
    assert torch.equal(gpu16["O"], gpu["O"].to(torch.bfloat16)) and torch.equal(gpu16["U"], gpu["U"])


def test_chain_configuration_matches_the_oracle(oracle):
    """The benchmark's chain configuration, shrunk, with the hint the benchmark gives (5 nodes)."""
    w = wl.make_workload(1, B=9, H_v=8, seed=7)
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, max_nodes=w.max_nodes)
    assert w.max_nodes == 5 and not gpu["status"].any()
    pu.assert_parity(w, gpu, tree_ref, ref)
    pu.assert_bf16_outputs(w, pu.run_gpu(w, torch.bfloat16, max_nodes=w.max_nodes), gpu, ref)


def test_small_kernel_agrees_with_the_tensor_core_kernel():
    w = _custom(TREES, H_v=4, H_qk=2, accepted=ACCEPTED, seed=6)
    small = pu.run_gpu(w, torch.float32, max_nodes=8)
    big = pu.run_gpu(w, torch.float32, max_nodes=16)
    torch.testing.assert_close(small["O"], big["O"], rtol=0, atol=2e-5)
    torch.testing.assert_close(small["U"], big["U"], rtol=0, atol=2e-5)
    torch.testing.assert_close(small["S32"], big["S32"], rtol=0, atol=2e-5)


def test_small_malformed_sequences_are_skipped_not_trapped(oracle):
    from paper_2608_20961_b200 import binding as tw
    good = [-1, 0, 0, 2]
    trees = [good, [-1, 2, 0], good, [i - 1 for i in range(9)], [-1, 0]]
    w = _custom(trees, H_v=2, H_qk=2, accepted=[3, 1, 9, 1, 1])
    gpu = pu.run_gpu(w, torch.float32, max_nodes=8)
    assert list(gpu["status"]) == [0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED, tw.SEQ_TOO_MANY_NODES, 0]
    off = w.node_offsets.tolist()
    for b in (1, 3):
        assert torch.all(gpu["O"][off[b]:off[b + 1]] == gpu["canary"])
        assert torch.all(gpu["U"][off[b]:off[b + 1]] == gpu["canary"])
        assert torch.equal(gpu["S"][b], w.S0[b])
    _, ref = pu.run_oracle(oracle, w.select_sequences([0, 4]))
    got = torch.cat([gpu["O"][off[0]:off[1]], gpu["O"][off[4]:off[5]]]).double().numpy()
    np.testing.assert_allclose(got, ref.O, atol=1e-4)


def _fused_pair(w1, w2):
    two = _two_rounds(w1, w2, False, 8, 8)
    one = _two_rounds(w1, w2, True, 8, 8)
    for x, y, name in zip(two, one, ("S", "O", "U", "status")):
        assert torch.equal(x, y), name      # same operation order as the stand-alone kernels: bit-identical
    return one


def test_fused_small_round_is_bit_identical_to_commit_then_verify():
    w1 = wl.make_workload(1, B=6, H_v=8, seed=51)
    w2 = wl.make_workload(1, B=6, H_v=8, seed=52)
    S, O, U, status = _fused_pair(w1, w2)
    assert not status.any() and not torch.equal(S, w1.S0)


def test_fused_small_round_with_edge_cases():
    from paper_2608_20961_b200 import binding as tw
    prev = [CHAIN8, [-1, 0, 0, 2], [-1], [-1, 0, 1], [-1, 0], COMB]
    new = [[-1, 0, 1, 1, 0], STAR8, [-1, 2, 0], CHAIN8, [-1], [-1, 0]]
    #       ok               ok     malformed   ok      ok    ok
    w1 = _custom(prev, H_v=4, H_qk=2, seed=3, accepted=[7, 3, -1, 7, 1, 5])   # seq 3: accepted out of range
    w2 = _custom(new, H_v=4, H_qk=2, seed=4)
    w2.S0 = w1.S0
    S, O, U, status = _fused_pair(w1, w2)
    assert list(status) == [0, 0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED, 0, 0]
    assert torch.equal(S[2], w1.S0[2]) and torch.equal(S[3], w1.S0[3])
    assert not torch.equal(S[0], w1.S0[0]) and not torch.equal(S[4], w1.S0[4])
    off = w2.node_offsets.tolist()
    assert torch.all(U[off[2]:off[3]] == 5.0)


def test_fused_small_round_matches_the_oracle(oracle):
    """Round 1 verified and committed by the oracle; its committed state, rounded to bf16, starts the
    oracle's round 2.  The GPU runs verify(1), then commit(1) + verify(2) in the small fused kernel."""
    w1 = wl.make_workload(1, B=5, H_v=4, seed=61)
    w2 = wl.make_workload(1, B=5, H_v=4, seed=62)
    _, ref1 = pu.run_oracle(oracle, w1)
    S, O, U, status = _two_rounds(w1, w2, True, 5, 5)
    assert not status.any()
    want = torch.from_numpy(ref1.S_commit).to(torch.bfloat16)
    step = (S.float() - want.float()).abs()
    assert float((step > 2.0 ** -7 * want.float().abs() + 1e-6).float().mean()) < 1e-3   # one bf16 step, rarely
    w2.S0 = S
    _, ref2 = pu.run_oracle(oracle, w2)
    for got, ref in ((O.double().numpy(), ref2.O), (U.double().numpy(), ref2.U)):
        for b in range(w2.B):
            sl = slice(int(w2.node_offsets[b]), int(w2.node_offsets[b + 1]))
            mx, fro = pu.unit_errors(got[sl], ref[sl])
            assert fro <= 5e-3, (b, fro)


def test_small_kernel_on_a_state_pool():
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w = _custom(TREES, H_v=4, H_qk=2, accepted=ACCEPTED, seed=8)
    d = lambda t: t.to(dev)

    def run(pool):
        tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, 8)
        status = torch.zeros(w.B, dtype=torch.int32, device=dev)
        O = torch.full((w.T, w.H_v, 128), 3.0, dtype=torch.bfloat16, device=dev)
        U = torch.full((w.T, w.H_v, 128), 3.0, dtype=torch.float32, device=dev)
        tw.treewy_tree_prepare(tree, d(w.alpha), status)
        if pool:
            idx = torch.tensor([9, 2, 5, 0, 7, 3, 1, 12], dtype=torch.int32, device=dev)   # 12: outside the pool
            S = torch.zeros((10,) + tuple(w.S0.shape[1:]), dtype=w.S0.dtype, device=dev)
            S[idx[:7].long()] = d(w.S0)[:7]
            tw.treewy_verify_pool(S, idx, d(w.q), d(w.k), d(w.v), d(w.beta), tree, w.H_qk, O, U, status)
        else:
            S = d(w.S0).clone()
            tw.treewy_verify(S, d(w.q), d(w.k), d(w.v), d(w.beta), tree, w.H_qk, O, U, status)
        torch.cuda.synchronize()
        return O.cpu(), U.cpu(), status.cpu()

    (O, U, st), (Op, Up, stp) = run(False), run(True)
    off = w.node_offsets.tolist()
    assert not st.any() and list(stp) == [0] * 7 + [tw.SEQ_BAD_STATE]
    assert torch.equal(O[:off[7]], Op[:off[7]]) and torch.equal(U[:off[7]], Up[:off[7]])
    assert torch.all(Up[off[7]:] == 3.0)


def test_fused_small_round_at_the_chain_workloads_full_size():
    """The chain configuration as the benchmark runs it (64 sequences x 32 heads, hint 5): the fused
    round stores the same bits as commit followed by verify."""
    w1 = wl.make_workload(1, seed=81)
    w2 = wl.make_workload(1, seed=82)
    two = _two_rounds(w1, w2, False, 5, 5)
    one = _two_rounds(w1, w2, True, 5, 5)
    for x, y, name in zip(two, one, ("S", "O", "U", "status")):
        assert torch.equal(x, y), name
    assert not one[3].any()


def test_fused_small_round_on_a_state_pool():
    """commit(r) + verify(r+1) of chains with the states scattered in a pool: bit for bit the plain call."""
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w1 = wl.make_workload(1, B=6, H_v=4, seed=91)
    w2 = wl.make_workload(1, B=6, H_v=4, seed=92)
    n_states = 9
    perm = torch.randperm(n_states, generator=torch.Generator().manual_seed(3))[: w1.B].to(torch.int32)
    d = lambda t: t.to(dev)

    def run(pool):
        status = torch.zeros(w1.B, dtype=torch.int32, device=dev)
        t1 = tw.Tree.empty(d(w1.node_offsets), d(w1.parent), w1.H_v, 5)
        t2 = tw.Tree.empty(d(w2.node_offsets), d(w2.parent), w2.H_v, 5)
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
                                         d(w2.beta), t2, w2.H_qk, O2, U2, True, status)
            torch.cuda.synchronize()
            assert torch.all(S[sorted(set(range(n_states)) - set(perm.tolist()))] == 0.25)
            S = S[idx.long()]
        else:
            S = d(w1.S0).clone()
            tw.treewy_verify(S, d(w1.q), d(w1.k), d(w1.v), d(w1.beta), t1, w1.H_qk, O1, U1, status)
            tw.treewy_commit_verify(S, U1, d(w1.k), t1, d(w1.accepted), d(w2.q), d(w2.k), d(w2.v), d(w2.beta), t2,
                                    w2.H_qk, O2, U2, True, status)
            torch.cuda.synchronize()
        return S.cpu(), O2.cpu(), U2.cpu(), status.cpu()

    a, b = run(False), run(True)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert not a[3].any() and not torch.equal(a[0], w1.S0)
