"""The benchmark configurations at FULL size, in the launch configuration bench.py times: every
sequence of configurations 1-4 is compared with the oracle element by element (the oracle does a
whole configuration in a second or two), every node's tree outputs are also checked through
invariants, and every stored state is checked to be the rounding of the fp32 state.  Only the
128-node workload of the wide-tree calls is compared on sampled sequences."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cid", [1, 2, 3, 4])
def test_full_size_config(oracle, cid):
    w = wl.make_workload(cid, prefix_device="cuda:0")
    gpu = pu.run_gpu(w, torch.float32, max_nodes=w.max_nodes)
    assert not gpu["status"].any()
    pu.assert_tree_invariants(w, gpu)
    tree_ref, ref = pu.run_oracle(oracle, w)
    errs = pu.assert_parity(w, gpu, tree_ref, ref)         # the whole batch, every output
    print(f"config {cid} full size, all {w.B} sequences: {errs}")
    # stored state is RNE(fp32 state); finite everywhere; no row of O or U left at its canary value
    assert torch.equal(gpu["S"], gpu["S32"].to(gpu["S"].dtype))
    assert torch.isfinite(gpu["O"]).all() and torch.isfinite(gpu["U"]).all()
    assert not (gpu["U"] == gpu["canary"]).all(dim=-1).any()
    assert not (gpu["O"] == gpu["canary"]).all(dim=-1).any()


def test_full_size_bf16_outputs_match_rounded_fp32_outputs():
    w = wl.make_workload(2)
    a = pu.run_gpu(w, torch.float32, max_nodes=w.max_nodes, want_s32=False)
    b = pu.run_gpu(w, torch.bfloat16, max_nodes=w.max_nodes, want_s32=False)
    assert torch.equal(b["O"], a["O"].to(torch.bfloat16))
    assert torch.equal(b["U"], a["U"]) and torch.equal(b["S"], a["S"])


def test_tensor_core_and_simt_kernels_agree_at_full_size():
    w = wl.make_workload(2, B=64)
    a = pu.run_gpu(w, torch.float32, generic=False, want_s32=False)
    b = pu.run_gpu(w, torch.float32, generic=True, want_s32=False)
    # the tensor-core kernel's second product takes its operands as two-term bf16 splits and drops the
    # lo.lo term: 3 * 2^-18 = 1.1e-5 of |r_j| |T_ij| per product at worst, summed over a root path
    scale = float(b["O"].abs().max())
    assert float((a["O"] - b["O"]).abs().max()) <= 5e-5 * scale
    assert float((a["U"] - b["U"]).abs().max()) <= 5e-5 * float(b["U"].abs().max())


def test_full_size_half_u_is_the_rounded_u():
    """Workload 2 at full size through treewy_verify_half_u / treewy_commit_half_u: U16 = RNE(U32) and the
    same O, bit for bit; the committed state is the commit of the widened values."""
    from paper_2608_20961_b200 import binding as tw
    dev = torch.device("cuda:0")
    w = wl.make_workload(2)
    d = lambda t: t.to(dev)
    tree = tw.Tree.empty(d(w.node_offsets), d(w.parent), w.H_v, w.max_nodes)
    status = torch.zeros(w.B, dtype=torch.int32, device=dev)
    q, k, v, beta, acc = d(w.q), d(w.k), d(w.v), d(w.beta), d(w.accepted)
    tw.treewy_tree_prepare(tree, d(w.alpha), status)
    out = {}
    for half in (False, True):
        S = d(w.S0).clone()
        O = torch.empty((w.T, w.H_v, 128), dtype=torch.bfloat16, device=dev)
        U = torch.empty((w.T, w.H_v, 128), dtype=torch.float16 if half else torch.float32, device=dev)
        if half:
            tw.treewy_verify_half_u(S, q, k, v, beta, tree, w.H_qk, O, U, status)
            tw.treewy_commit_half_u(S, U, k, tree, w.H_qk, acc, None, status)
        else:
            tw.treewy_verify(S, q, k, v, beta, tree, w.H_qk, O, U, status)
            tw.treewy_commit(S, U.half().float(), k, tree, w.H_qk, acc, None, status)
        torch.cuda.synchronize()
        out[half] = (S, O, U)
    assert not status.any()
    assert torch.equal(out[True][1], out[False][1])
    assert torch.equal(out[True][2], out[False][2].half())
    assert torch.equal(out[True][0], out[False][0])


def test_full_size_wide_trees(oracle):
    """The 128-node workload through the wide-tree calls, every sequence against the oracle."""
    from tests.test_gpu_wide import run_wide
    w = wl.make_workload(6)
    gpu = run_wide(w, max_nodes=w.max_nodes)
    assert not gpu["status"].any()
    oracle.set_max_nodes(128)
    try:
        tree_ref, ref = pu.run_oracle(oracle, w)
    finally:
        oracle.set_max_nodes(64)
    gpu["anc_mask"] = tree_ref.anc_mask        # (the wide calls write no masks: nothing to compare)
    errs = pu.assert_parity(w, gpu, tree_ref, ref)
    print(f"workload 6 full size, all {w.B} sequences: {errs}")
    assert torch.isfinite(gpu["O"]).all() and torch.isfinite(gpu["U"]).all()
    assert not (gpu["U"] == gpu["canary"]).all(dim=-1).any() and not (gpu["O"] == gpu["canary"]).all(dim=-1).any()
