"""Wide draft trees (65..128 nodes): treewy_tree_prepare_wide / treewy_verify_wide /
treewy_commit_wide walk parent chains instead of 64-bit ancestor masks.  Same parity gates against
the oracle as the main calls (the oracle's node limit is raised to 128 for these tests), same status
and skip semantics; on trees of up to 64 nodes they agree with the main calls."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import _custom

pytestmark = pytest.mark.gpu


@pytest.fixture()
def wide_oracle(oracle):
    oracle.set_max_nodes(128)
    yield oracle
    oracle.set_max_nodes(64)


def run_wide(w, o_dtype=torch.float32, max_nodes=0):
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    d = lambda t: t.to(dev)
    tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, max_nodes)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    q, k, v, S = d(w.q), d(w.k), d(w.v), d(w.S0).clone()
    canary = 7.25
    O = torch.full((w.T, w.H_v, 128), canary, dtype=o_dtype, device=dev)
    U = torch.full((w.T, w.H_v, 128), canary, dtype=torch.float32, device=dev)
    S32 = torch.full(S.shape, canary, dtype=torch.float32, device=dev)
    tw.treewy_tree_prepare_wide(tree, d(w.alpha), status)
    tw.treewy_verify_wide(S, q, k, v, d(w.beta), tree, w.H_qk, O, U, status)
    tw.treewy_commit_wide(S, U, k, tree, w.H_qk, d(w.accepted), S32, status)
    torch.cuda.synchronize()
    return dict(depth=tree.depth.cpu().numpy(), anc_mask=None, cum_log_gate=tree.cum_log_gate.cpu().numpy(),
                level_order=tree.level_order.cpu().numpy(), O=O.cpu(), U=U.cpu(), S=S.cpu(), S32=S32.cpu(),
                status=status.cpu().numpy(), canary=canary)


def _trees():
    g = torch.Generator().manual_seed(5)
    chain = [i - 1 for i in range(128)]
    star = [-1] + [0] * 127
    comb = [-1] + [max(0, i - 2) for i in range(1, 100)]           # depth ~ 50
    return [chain, star, comb, wl.random_parent_tree(g, 128, 10), wl.random_parent_tree(g, 65, 6),
            wl.random_parent_tree(g, 97, 30), [-1, -1, 0, 1, -1, 4, 5], [-1]]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_wide_trees_match_the_oracle(wide_oracle, dtype):
    trees = _trees()
    w = _custom(trees, H_v=4, H_qk=2, seed=9, dtype=dtype, accepted=[127, 64, 99, 120, -1, 96, 6, 0])
    tree_ref, ref = pu.run_oracle(wide_oracle, w)
    gpu = run_wide(w)
    assert not gpu["status"].any() and not ref.seq_status.any()
    gpu["anc_mask"] = tree_ref.anc_mask        # (the wide calls write no masks: nothing to compare)
    errs = pu.assert_parity(w, gpu, tree_ref, ref)
    print(f"wide trees, {dtype}: {errs}")
    assert torch.equal(gpu["S"][4], w.S0[4])                       # accepted = -1
    if dtype == torch.bfloat16:
        low = run_wide(w, torch.bfloat16)
        assert torch.equal(low["O"], gpu["O"].to(torch.bfloat16)) and torch.equal(low["U"], gpu["U"])


def test_wide_calls_agree_with_the_main_calls_up_to_64_nodes():
    w = wl.make_workload(3, B=3, H_v=4, seed=17)                   # 64-node trees
    a = run_wide(w, max_nodes=64)
    b = pu.run_gpu(w, torch.float32, max_nodes=64)
    assert not a["status"].any() and not b["status"].any()
    np.testing.assert_array_equal(a["depth"], b["depth"])
    np.testing.assert_array_equal(a["level_order"], b["level_order"])
    assert np.array_equal(a["cum_log_gate"], b["cum_log_gate"])    # the same sums in the same order
    for name in ("O", "U", "S32"):
        scale = float(b[name].abs().max())
        assert float((a[name] - b[name]).abs().max()) <= 2e-5 * scale, name


def test_wide_malformed_sequences_are_skipped_not_trapped(wide_oracle):
    from paper_2608_20961_b200 import binding as tw
    good = [i - 1 for i in range(70)]
    bad_parent = list(good)
    bad_parent[40] = 41
    trees = [good, bad_parent, good, [i - 1 for i in range(129)], [-1, 0]]
    w = _custom(trees, H_v=2, H_qk=2, accepted=[69, 1, 70, 5, 1])   # sequence 2: accepted out of range
    gpu = run_wide(w)
    assert list(gpu["status"]) == [0, tw.SEQ_BAD_PARENT, tw.SEQ_BAD_ACCEPTED, tw.SEQ_TOO_MANY_NODES, 0]
    off = w.node_offsets.tolist()
    for b in (1, 3):
        assert torch.all(gpu["O"][off[b]:off[b + 1]] == gpu["canary"])
        assert torch.all(gpu["U"][off[b]:off[b + 1]] == gpu["canary"])
        assert torch.equal(gpu["S"][b], w.S0[b])
    assert torch.equal(gpu["S"][2], w.S0[2])
    _, ref = pu.run_oracle(wide_oracle, w.select_sequences([0, 4]))
    got = torch.cat([gpu["O"][off[0]:off[1]], gpu["O"][off[4]:off[5]]]).double().numpy()
    np.testing.assert_allclose(got, ref.O, atol=1e-4)


def test_wide_limits_are_checked_on_the_host():
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w = _custom([[-1, 0]], H_v=2, H_qk=2)
    tree = tw.Tree.empty(w.node_offsets.to(dev), w.parent.to(dev), w.H_v, 129)
    with pytest.raises(tw.TreewyError):
        tw.treewy_tree_prepare_wide(tree, w.alpha.to(dev), None)


@pytest.mark.parametrize("seed", range(6))
def test_random_wide_batches_shallow_and_deep_trees_side_by_side(wide_oracle, seed):
    """Random batches of trees of 1..128 nodes whose depth limit is drawn per tree, so that the
    tensor-core kernel (paths of up to 16 ancestors) and the SIMT kernel (deeper ones) each take their
    share of one call; heads shared by 1, 2 or 4 value heads."""
    g = torch.Generator().manual_seed(100 + seed)
    ri = lambda hi: int(torch.randint(0, hi, (1,), generator=g))
    trees = []
    for _ in range(6 + ri(10)):
        n = (1, 2, 17, 33, 64, 65, 96, 127, 128)[ri(9)]
        depth_cap = (1, 2, 5, 10, 16, 17, 40, 128)[ri(8)]
        kind = ri(4)
        if kind == 0:      # a chain: as deep as it gets (17 nodes = 16 ancestors is the tensor-core kernel's limit)
            n = (17, 18, 40, 128)[ri(4)]
            trees.append([i - 1 for i in range(n)])
        elif kind == 1:    # a chain with a bush of leaves at its end
            stem = (15, 16, 17, 30)[ri(4)]
            trees.append([i - 1 for i in range(stem)] + [stem - 1] * (min(n, 128 - stem)))
        else:
            trees.append(wl.random_parent_tree(g, n, depth_cap) if n > 1 else [-1])
    H_v, H_qk = ((4, 4), (4, 2), (4, 1))[seed % 3]
    acc = [ri(len(t) + 1) - 1 for t in trees]                   # -1 .. n-1
    w = _custom(trees, H_v=H_v, H_qk=H_qk, seed=200 + seed, accepted=acc)
    tree_ref, ref = pu.run_oracle(wide_oracle, w)
    gpu = run_wide(w)
    assert not gpu["status"].any()
    gpu["anc_mask"] = tree_ref.anc_mask
    errs = pu.assert_parity(w, gpu, tree_ref, ref)
    print(f"seed {seed}: {len(trees)} trees, {errs}")


def test_wide_calls_on_a_tiny_batch(wide_oracle):
    """Fewer packed nodes than one load box has rows (T = 4 against boxes of 128 rows): the loads read
    zeros past the arrays' end and nothing outside a sequence's rows is written."""
    w = _custom([[-1], [-1, 0, 0]], H_v=2, H_qk=1, seed=31, accepted=[0, 2])
    tree_ref, ref = pu.run_oracle(wide_oracle, w)
    gpu = run_wide(w)
    assert not gpu["status"].any()
    gpu["anc_mask"] = tree_ref.anc_mask
    pu.assert_parity(w, gpu, tree_ref, ref)
