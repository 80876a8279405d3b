"""GPU parity tests: libtreewy (through its C ABI) against the fp64 CPU oracle, element by
element, on seeded inputs small enough for the oracle to finish in seconds yet spanning
several CTAs, shared q/k heads and ragged tails."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


SMALL = {  # config id -> overrides that keep the structure but shrink the batch
    0: {},
    1: dict(B=6, H_v=8),
    2: dict(B=5, H_v=8),
    3: dict(B=3, H_v=4),
    4: dict(B=21, H_v=4, prefix_tokens=32),
    5: dict(B=3, H_v=4),
}


# "generic": fp32 SIMT kernel; "general": tensor-core kernel for up to 64 nodes (no size hint);
# "hinted": the caller states max_nodes, so trees of up to 32 nodes take the tensor-core solve
@pytest.mark.parametrize("path", ["generic", "general", "hinted"])
@pytest.mark.parametrize("cid", sorted(SMALL))
def test_configs_match_oracle(oracle, cid, path):
    w = wl.make_workload(cid, **SMALL[cid])
    generic = path == "generic"
    hint = w.max_nodes if path == "hinted" else 0
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, generic=generic, max_nodes=hint)
    assert not gpu["status"].any()
    errs = pu.assert_parity(w, gpu, tree_ref, ref)
    print(f"config {cid} path={path}: worst (max-abs/rms, rel-fro) {errs}")
    if w.io_dtype == torch.bfloat16:
        gpu16 = pu.run_gpu(w, torch.bfloat16, generic=generic, max_nodes=hint)
        got, floor = pu.assert_bf16_outputs(w, gpu16, gpu, ref)
        print(f"   bf16 O: {got} against rounding floor {floor}")
        assert torch.equal(gpu16["S"], gpu["S"])


@pytest.mark.parametrize("generic", [True, False])
def test_fp32_inputs_bf16_heads_shared_by_four(oracle, generic):
    w = wl.make_workload(2, B=3, H_v=8, H_qk=2)
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, generic=generic)
    pu.assert_parity(w, gpu, tree_ref, ref)
    w32 = wl.make_workload(2, B=2, H_v=4, io_dtype=torch.float32)
    tree_ref, ref = pu.run_oracle(oracle, w32)
    gpu = pu.run_gpu(w32, torch.float32, generic=generic)
    pu.assert_parity(w32, gpu, tree_ref, ref)


def _custom(trees, H_v=2, H_qk=1, seed=1, dtype=torch.bfloat16, accepted=None):
    """A workload with hand-made topologies and config-2 value distributions."""
    base = wl.make_workload(2, B=1, H_v=H_v, H_qk=H_qk, seed=seed)
    g = torch.Generator().manual_seed(seed)
    off = [0]
    for t in trees:
        off.append(off[-1] + len(t))
    T, B = off[-1], len(trees)
    norm = lambda x: x / x.norm(dim=-1, keepdim=True)
    return wl.Workload(
        name="custom", config_id=-1, B=B, H_v=H_v, H_qk=H_qk, io_dtype=dtype,
        node_offsets=torch.tensor(off, dtype=torch.int32),
        parent=torch.tensor([p for t in trees for p in t], dtype=torch.int32),
        q=norm(torch.randn(T, H_qk, 128, generator=g)).to(dtype),
        k=norm(torch.randn(T, H_qk, 128, generator=g)).to(dtype),
        v=torch.randn(T, H_v, 128, generator=g).to(dtype),
        alpha=0.9 + 0.099 * torch.rand(T, H_v, generator=g),
        beta=0.1 + 0.8 * torch.rand(T, H_v, generator=g),
        S0=(0.05 * torch.randn(B, H_v, 128, 128, generator=g)).to(dtype),
        accepted=torch.tensor(accepted if accepted is not None else [len(t) - 1 for t in trees],
                              dtype=torch.int32), seed=seed)


@pytest.mark.parametrize("generic", [True, False])
def test_degenerate_topologies(oracle, generic):
    chain64 = [i - 1 for i in range(64)]
    star64 = [-1] + [0] * 63
    forest = [-1, -1, 0, 1, -1, 4, 5]
    single = [-1]
    trees = [chain64, star64, forest, single, [-1, 0], chain64[:33]]
    w = _custom(trees, H_v=4, H_qk=2, accepted=[63, 17, 6, 0, -1, 32])
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, generic=generic)
    assert not gpu["status"].any()
    pu.assert_parity(w, gpu, tree_ref, ref)
    # accepted = -1: the stored state is bit-identical to the input state
    assert torch.equal(gpu["S"][4], w.S0[4])


@pytest.mark.parametrize("generic", [True, False])
def test_malformed_sequences_are_skipped_not_trapped(oracle, generic):
    good = [-1, 0, 0, 2]
    bad_parent = [-1, 2, 0]               # parent[1] = 2 >= 1
    trees = [good, bad_parent, good, [-1, 0]]
    w = _custom(trees, H_v=2, H_qk=2, accepted=[3, 1, 9, 1])   # sequence 2: accepted out of range
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, generic=generic)
    from paper_2608_20961_b200 import binding as tw
    assert list(gpu["status"]) == [0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED, 0]
    assert list(ref.seq_status) == list(gpu["status"])
    pu.assert_parity(w, gpu, tree_ref, ref, skip_seqs=(1, 2))
    off = w.node_offsets.tolist()
    # skipped sequence: outputs untouched (canary), state untouched
    assert torch.all(gpu["O"][off[1]:off[2]] == gpu["canary"])
    assert torch.all(gpu["U"][off[1]:off[2]] == gpu["canary"])
    assert torch.equal(gpu["S"][1], w.S0[1]) and torch.equal(gpu["S"][2], w.S0[2])
    # bad accepted only stops the commit: verify outputs of sequence 2 are right
    sl = slice(off[2], off[3])
    np.testing.assert_allclose(gpu["O"][sl].double().numpy(), ref_O_of(oracle, w, 2), atol=1e-4)


def ref_O_of(oracle, w, b):
    one = w.select_sequences([b])
    one.accepted[:] = -1
    return pu.run_oracle(oracle, one)[1].O


def test_max_nodes_hint_flags_longer_sequences():
    from paper_2608_20961_b200 import binding as tw
    w = _custom([[-1, 0, 1], [i - 1 for i in range(20)]], H_v=2, H_qk=2)
    gpu = pu.run_gpu(w, torch.float32, max_nodes=16)
    assert list(gpu["status"]) == [0, tw.SEQ_TOO_MANY_NODES]


def test_empty_batch_is_a_no_op():
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    off = torch.zeros(1, dtype=torch.int32, device=dev)
    par = torch.zeros(4, dtype=torch.int32, device=dev)[:0]
    tree = tw.Tree.empty(off, par, 2)
    z = torch.zeros(4, 2, 128, device=dev)
    tw.treewy_tree_prepare(tree, z[:, :, 0], None)
    tw.treewy_verify(z, z, z, z, z[:, :, 0], tree, 2, z.clone(), z.clone(), None)
    tw.treewy_commit(z, z, z, tree, 2, off, None, None)
    torch.cuda.synchronize()


def test_metamorphic_commit_then_verify_on_gpu(oracle):
    # commit node a on the GPU, then verify a's subtree from the new state: outputs of those
    # nodes must reproduce the first verify (fp32 state hand-over keeps it tight)
    tree = [-1, 0, 1, 1, 3, 0, 2]
    w = _custom([tree], H_v=2, H_qk=1, dtype=torch.float32, accepted=[1])
    first = pu.run_gpu(w, torch.float32)
    sub = [2, 3, 4, 6]
    w2 = _custom([[-1, -1, 1, 0]], H_v=2, H_qk=1, dtype=torch.float32, accepted=[-1])
    idx = torch.tensor(sub)
    w2.q, w2.k, w2.v = w.q[idx], w.k[idx], w.v[idx]
    w2.alpha, w2.beta = w.alpha[idx], w.beta[idx]
    w2.S0 = first["S"]
    second = pu.run_gpu(w2, torch.float32)
    torch.testing.assert_close(second["O"], first["O"][idx], rtol=0, atol=2e-5)
    torch.testing.assert_close(second["U"], first["U"][idx], rtol=0, atol=2e-5)


@pytest.mark.parametrize("hint", [16, 32])
def test_small_trees_through_the_tensor_core_solve(oracle, hint):
    """Shapes that stress the up-to-32-node kernel: full chains (paths deeper than the eight
    ancestors its register path handles), stars, forests, single nodes, mixed in one batch."""
    n = hint
    chain = [i - 1 for i in range(n)]
    star = [-1] + [0] * (n - 1)
    forest = [-1, -1, 0, 1, -1, 4, 5]
    comb = [-1] + [max(0, i - 2) for i in range(1, n)]          # depth ~ n/2
    trees = [chain, star, forest, [-1], [-1, 0], comb, chain[:9], chain[:10]]
    w = _custom(trees, H_v=4, H_qk=2, accepted=[n - 1, 3, 6, 0, -1, n - 1, 8, 9])
    tree_ref, ref = pu.run_oracle(oracle, w)
    gpu = pu.run_gpu(w, torch.float32, max_nodes=hint)
    assert not gpu["status"].any()
    pu.assert_parity(w, gpu, tree_ref, ref)
    gpu16 = pu.run_gpu(w, torch.bfloat16, max_nodes=hint)
    assert torch.equal(gpu16["O"], gpu["O"].to(torch.bfloat16)) and torch.equal(gpu16["U"], gpu["U"])


def test_malformed_sequences_in_the_tensor_core_solve(oracle):
    from paper_2608_20961_b200 import binding as tw
    good = [-1, 0, 0, 2]
    trees = [good, [-1, 2, 0], good, [i - 1 for i in range(20)]]
    w = _custom(trees, H_v=2, H_qk=2, accepted=[3, 1, 9, 1])
    gpu = pu.run_gpu(w, torch.float32, max_nodes=16)
    assert list(gpu["status"]) == [0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED, tw.SEQ_TOO_MANY_NODES]
    tree_ref, ref = pu.run_oracle(oracle, w.select_sequences([0]))
    off = w.node_offsets.tolist()
    np.testing.assert_allclose(gpu["O"][:4].double().numpy(), ref.O, atol=1e-4)
    assert torch.all(gpu["O"][off[1]:off[2]] == gpu["canary"])
    assert torch.all(gpu["U"][off[3]:off[4]] == gpu["canary"])


def test_prepare_from_log_gates(oracle):
    """Gates given as logarithms: the tree outputs are those of the oracle run on exp(log alpha), the
    cumulative log-gate is the plain sum along the root path, and verify on top of it matches."""
    from paper_2608_20961_b200 import binding as tw
    w = wl.make_workload(5, B=4, H_v=4, seed=7)
    g = torch.log(w.alpha.double()).float()                      # what a GDN layer would hand over
    w.alpha = torch.exp(g.double()).float()
    tree_ref = oracle.prepare(w.node_offsets.numpy(), w.parent.numpy(), np.exp(g.double().numpy()))
    dev = torch.device("cuda:0")
    tree = tw.Tree.empty(w.node_offsets.to(dev), w.parent.to(dev), w.H_v, w.max_nodes)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    tw.treewy_tree_prepare_log(tree, g.to(dev), status)
    torch.cuda.synchronize()
    assert not status.any()
    np.testing.assert_array_equal(tree.depth.cpu().numpy(), tree_ref.depth)
    np.testing.assert_array_equal(tree.anc_mask.cpu().numpy().view(np.uint64), tree_ref.anc_mask)
    np.testing.assert_array_equal(tree.level_order.cpu().numpy(), tree_ref.level_order)
    np.testing.assert_allclose(tree.cum_log_gate.cpu().numpy(), tree_ref.cum_log_gate, rtol=0, atol=1e-5)
    lin = tw.Tree.empty(w.node_offsets.to(dev), w.parent.to(dev), w.H_v, w.max_nodes)
    tw.treewy_tree_prepare(lin, w.alpha.to(dev), status)
    torch.cuda.synchronize()
    np.testing.assert_allclose(tree.cum_log_gate.cpu().numpy(), lin.cum_log_gate.cpu().numpy(), rtol=0, atol=2e-6)


@pytest.mark.parametrize("H_v,H_qk", [(1, 1), (2, 1), (3, 3), (6, 1), (4, 2), (5, 1)])
def test_mixed_size_batches_across_head_layouts(oracle, H_v, H_qk):
    """A batch that holds trees on both sides of 32 nodes gets one launch per size class, each numbering
    the units of its class's sequences (one, several, an odd number of units per sequence; heads taken
    singly or in pairs): every sequence must be verified exactly once, whatever its place in the batch."""
    g = torch.Generator().manual_seed(100 + 7 * H_v + H_qk)
    sizes = [40, 3, 64, 17, 1, 33, 32, 8, 50, 20, 64, 2, 36]
    trees = [wl.random_parent_tree(g, n, 6) for n in sizes]
    w = _custom(trees, H_v=H_v, H_qk=H_qk, seed=9, accepted=[n // 2 for n in sizes])
    gpu = pu.run_gpu(w, torch.float32, max_nodes=64)
    assert not gpu["status"].any()
    assert not (gpu["U"] == gpu["canary"]).all(dim=-1).any()
    tree_ref, ref = pu.run_oracle(oracle, w)
    pu.assert_parity(w, gpu, tree_ref, ref)


def test_mixed_size_batch_larger_than_the_class_table(oracle):
    """More sequences than a class launch lists in shared memory (1024): both class launches walk the
    whole batch and drop the other class's sequences one by one."""
    g = torch.Generator().manual_seed(77)
    sizes = [1 + int(torch.randint(0, 3, (1,), generator=g)) for _ in range(1040)]
    for at, n in ((5, 64), (333, 40), (700, 33), (1030, 57)):
        sizes[at] = n
    trees = [wl.random_parent_tree(g, n, 5) for n in sizes]
    w = _custom(trees, H_v=1, H_qk=1, seed=12, accepted=[n - 1 for n in sizes])
    gpu = pu.run_gpu(w, torch.float32, max_nodes=64)
    assert not gpu["status"].any()
    assert not (gpu["U"] == gpu["canary"]).all(dim=-1).any()
    tree_ref, ref = pu.run_oracle(oracle, w)
    pu.assert_parity(w, gpu, tree_ref, ref)


def test_mixed_size_batch_with_many_heads_per_sequence():
    """More units than a class launch's 16-bit unit table can number (sequences x heads > 65536; here
    520 x 128 unpaired heads, 2 GB of states): both class launches walk the whole batch instead.  Checked
    against the SIMT kernel on the same inputs (every row written exactly where that kernel writes)."""
    g = torch.Generator().manual_seed(78)
    sizes = [1 + int(torch.randint(0, 2, (1,), generator=g)) for _ in range(520)]
    for at, n in ((7, 40), (519, 64)):
        sizes[at] = n
    trees = [wl.random_parent_tree(g, n, 4) for n in sizes]
    w = _custom(trees, H_v=128, H_qk=128, seed=13, accepted=[n - 1 for n in sizes])
    fast = pu.run_gpu(w, torch.float32, max_nodes=64, want_s32=False)
    slow = pu.run_gpu(w, torch.float32, max_nodes=64, want_s32=False, generic=True)
    assert not fast["status"].any() and not slow["status"].any()
    assert not (fast["U"] == fast["canary"]).all(dim=-1).any()
    for name in ("O", "U"):
        scale = float(slow[name].abs().max())
        assert float((fast[name] - slow[name]).abs().max()) <= 5e-5 * scale, name
    assert torch.equal(fast["S"], slow["S"]) or float((fast["S"].float() - slow["S"].float()).abs().max()) <= 2 ** -7 * float(slow["S"].float().abs().max())
