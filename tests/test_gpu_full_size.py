"""The benchmark configurations at FULL size, in the launch configuration bench.py times:
sampled sequences are compared with the oracle element by element, every node's tree outputs
are checked through invariants, and every stored state is checked to be the rounding of the
fp32 state."""
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
    g = np.random.default_rng(cid)
    seqs = sorted(set([0, w.B - 1] + g.integers(0, w.B, 4).tolist()))
    if cid == 4:   # make sure every tree size of the ragged mix is sampled
        sizes = (w.node_offsets[1:] - w.node_offsets[:-1]).tolist()
        seqs = sorted(set(seqs + [sizes.index(s) for s in (1, 8, 16, 32, 64) if s in sizes]))
    errs = pu.assert_parity_sampled(oracle, w, gpu, seqs)
    print(f"config {cid} full size, sequences {seqs}: {errs}")
    # whole batch: stored state is RNE(fp32 state); finite everywhere; untouched canaries none
    assert torch.equal(gpu["S"], gpu["S32"].to(gpu["S"].dtype))
    assert torch.isfinite(gpu["O"]).all() and torch.isfinite(gpu["U"]).all()
    assert not (gpu["U"] == gpu["canary"]).all(dim=-1).any()


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
    scale = float(b["O"].abs().max())
    assert float((a["O"] - b["O"]).abs().max()) <= 1e-5 * scale
    assert float((a["U"] - b["U"]).abs().max()) <= 1e-5 * float(b["U"].abs().max())
