"""Host-side arithmetic and input generators (no GPU, no oracle)."""
import os

import torch

from paper_2608_20961_b200 import footprint as fp
from paper_2608_20961_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_memory_arithmetic.txt")


def paper_numbers():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            key, val = line.split("=")
            out[key.strip()] = int(val)
    return out


def test_memory_arithmetic_matches_the_paper():
    p = paper_numbers()
    assert fp.kv_cache_bytes_per_token(10) == p["kv_bytes_per_token_35B"]
    assert fp.kv_cache_bytes_per_token(15) == p["kv_bytes_per_token_397B"]
    assert fp.gdn_state_bytes_per_seq(30, 32) == p["state_bytes_per_seq_35B"]
    assert fp.gdn_state_bytes_per_seq(45, 64) == p["state_bytes_per_seq_397B"]
    assert fp.snapshot_blocks(3) * fp.gdn_state_bytes_per_seq(30, 32) == p["snapshot_bytes_per_seq_35B_k3"]
    assert fp.snapshot_blocks(3) * fp.gdn_state_bytes_per_seq(45, 64) == p["snapshot_bytes_per_seq_397B_k3"]
    assert fp.pseudo_value_shrink() == p["pseudo_value_shrink"]
    for key, val in p.items():
        if key.startswith("widths_"):
            w = tuple(int(x) for x in key.split("_")[1:])
            assert fp.nodes_from_widths(w) == val
            assert len(wl.widths_tree(w)) == val
        if key.startswith("blocks_"):
            w = tuple(int(x) for x in key.split("_")[1:])
            assert fp.snapshot_blocks(fp.nodes_from_widths(w)) == val


def test_footprint_report_for_the_n32_tree():
    r = fp.footprint_report(32, 32, 16)
    assert r["U_bytes"] == 512 * 1024                     # fp32 U, 32 nodes x 32 heads x 128
    assert r["snapshot_bytes"] == 33 * 1024 * 1024        # 33 bf16 states of 1 MiB
    assert r["snapshot_over_U"] == 66 and r["snapshot_over_U_if_16bit"] == 132
    assert r["blocks_snapshotting"] == 33 and r["blocks_reconstruct"] == 1


def test_algorithmic_bytes_of_the_n32_tree():
    pb = fp.algorithmic_bytes([32] * 256, [4] * 256, 32, 16)
    per_seq_verify = pb.verify / 256 / 1024
    per_seq_commit = pb.commit / 256 / 1024
    # S0 1024 + q,k 256 + v 256 + O 256 + U 512 + gates/mask 8.25 KiB
    assert abs(per_seq_verify - 2312.25) < 1e-9
    assert 2125 < per_seq_commit < 2135                    # 2 x 1024 KiB of state + 4 path rows
    assert pb.tensor_flops == 256 * (32 * 2 * 64 * 128 * 128 + 16 * 2 * 64 * 32 * 128)


def check_tree(parent, max_depth=None):
    depth = wl.tree_depths(parent)
    assert parent[0] == -1 and all(-1 <= p < i for i, p in enumerate(parent))
    if max_depth is not None:
        assert max(depth) <= max_depth
    return depth


def test_workload_shapes_and_structure():
    w0 = wl.make_workload(0)
    assert (w0.B, w0.H_v, w0.H_qk, w0.T) == (1, 1, 1, 4) and w0.io_dtype == torch.float32
    assert w0.parent.tolist() == [-1, 0, 1, 2] and w0.accepted.tolist() == [2]

    w1 = wl.make_workload(1, B=4, H_v=4)
    assert w1.T == 20 and w1.H_qk == 4 and w1.q.dtype == torch.bfloat16
    assert all(0 <= a <= 4 for a in w1.accepted.tolist())

    w2 = wl.make_workload(2, B=6, H_v=4)
    assert w2.H_qk == 2 and w2.T == 6 * 32
    trees = [w2.parent[i * 32:(i + 1) * 32].tolist() for i in range(6)]
    for t in trees:
        check_tree(t, 6)
    assert trees[0] != trees[1]                            # a fresh tree per sequence

    w3 = wl.make_workload(3, B=3, H_v=2)
    for i in range(3):
        t = w3.parent[i * 64:(i + 1) * 64].tolist()
        d = check_tree(t, 4)
        assert [d[:57].count(x) for x in range(5)] == [1, 8, 16, 16, 16]
        assert int(w3.accepted[i]) in wl.tree_leaves(t)
    assert float(w3.alpha.min()) >= 0.95

    w4 = wl.make_workload(4, B=24, H_v=2, prefix_tokens=8)
    sizes = (w4.node_offsets[1:] - w4.node_offsets[:-1]).tolist()
    assert set(sizes) <= {1, 8, 16, 32, 64} and len(set(sizes)) > 2
    off = w4.node_offsets.tolist()
    for b in range(24):
        check_tree(w4.parent[off[b]:off[b + 1]].tolist(), 8)
        assert 0 <= int(w4.accepted[b]) < sizes[b]
    assert float(w4.S0.float().abs().max()) > 0            # the prefix recurrence wrote something

    w5 = wl.make_workload(5, B=2, H_v=2)
    assert w5.T == 80 and w5.H_qk == 1


def test_workloads_are_seeded_and_normalised():
    a = wl.make_workload(2, B=3, H_v=2)
    b = wl.make_workload(2, B=3, H_v=2)
    c = wl.make_workload(2, B=3, H_v=2, seed=5)
    assert torch.equal(a.q, b.q) and torch.equal(a.S0, b.S0) and torch.equal(a.parent, b.parent)
    assert not torch.equal(a.q, c.q)
    assert torch.allclose(a.k.float().norm(dim=-1), torch.ones(a.T, a.H_qk), atol=1e-2)
    assert 0.9 <= float(a.alpha.min()) and float(a.alpha.max()) <= 0.999
    assert 0.1 <= float(a.beta.min()) and float(a.beta.max()) <= 0.9


def test_select_sequences_repacks():
    w = wl.make_workload(4, B=10, H_v=2, prefix_tokens=2)
    s = w.select_sequences([7, 2])
    off = w.node_offsets.tolist()
    assert s.B == 2 and s.T == (off[8] - off[7]) + (off[3] - off[2])
    assert torch.equal(s.v[: off[8] - off[7]], w.v[off[7]:off[8]])
    assert torch.equal(s.S0[1], w.S0[2]) and int(s.accepted[0]) == int(w.accepted[7])
