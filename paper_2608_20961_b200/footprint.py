"""Byte and flop accounting for GDN draft-tree verify + commit (host arithmetic only).

Two uses: (1) the memory-footprint report -- what snapshotting holds per sequence
(Section 2, "The memory problem": n_GDN x n_vhead x d_v x d_k x 2 B per state, k+1 or
N+1 states) against the pseudo-value matrix of Section 3 ("Reconstruct on commit");
(2) the ALGORITHMIC bytes of one prepare + verify + commit pass, i.e. the bytes the
method itself must move once, which is the numerator of the HBM roofline fraction.
"""
from __future__ import annotations

from dataclasses import dataclass

D = 128


def kv_cache_bytes_per_token(n_softmax: int, n_kv_heads: int = 2, d_head: int = 256,
                             elem: int = 2) -> int:
    """2 (K,V) x softmax layers x KV heads x d_head x element size (Section 2)."""
    return 2 * n_softmax * n_kv_heads * d_head * elem


def gdn_state_bytes_per_seq(n_gdn: int, n_vhead: int, d_v: int = D, d_k: int = D,
                            elem: int = 2) -> int:
    """One committed recurrent state per GDN layer and value head (Section 2)."""
    return n_gdn * n_vhead * d_v * d_k * elem


def snapshot_blocks(n_draft_nodes: int) -> int:
    """Full-state snapshotting keeps the committed state plus one state per draft node."""
    return n_draft_nodes + 1


def nodes_from_widths(widths) -> int:
    """Draft nodes of a ``draft_tree_widths`` tree: w1 + w1 w2 + w1 w2 w3 + ..."""
    total, level = 0, 1
    for w in widths:
        level *= w
        total += level
    return total


def pseudo_value_shrink(d_k: int = D) -> int:
    """A pseudo-value row (d_v numbers) against a state (d_v x d_k) per node, same dtype."""
    return d_k


@dataclass
class PassBytes:
    prepare: int
    verify: int
    commit: int
    tensor_flops: int

    @property
    def total(self) -> int:
        return self.prepare + self.verify + self.commit


def algorithmic_bytes(nodes_per_seq, commit_path_len, H_v: int, H_qk: int, io_elem: int = 2,
                      o_elem: int = 2, u_elem: int = 4) -> PassBytes:
    """Bytes each call must move once, summed over the batch.

    nodes_per_seq[b]   N_b
    commit_path_len[b] depth(accepted)+1, or 0 when nothing is accepted (state untouched)

    prepare: parent in, alpha in, depth / mask / cumulative log-gate out.
    verify : S0, q, k, v, beta, log-gate, mask in; O and U out.
    commit : S0 in and out, and the accepted path's rows of U, k and the log-gate in.
    tensor_flops counts the dense contractions: [Q;K] S0^T per value head and
    [Q;K] K^T per q/k head (2 flops per multiply-add).
    """
    state = D * D * io_elem
    prep = ver = com = flops = 0
    for n, plen in zip(nodes_per_seq, commit_path_len):
        n, plen = int(n), int(plen)
        prep += n * (4 + 4 * H_v) + n * (4 + 8 + 4 * H_v)
        ver += H_v * state + 2 * n * H_qk * D * io_elem + n * H_v * D * io_elem
        ver += n * H_v * 8 + n * 8
        ver += n * H_v * D * (o_elem + u_elem)
        if plen > 0:
            com += 2 * H_v * state
            com += plen * (H_v * D * u_elem + H_qk * D * io_elem + 4 * H_v) + 8 + 4
        flops += H_v * 2 * (2 * n) * D * D + H_qk * 2 * (2 * n) * n * D
    return PassBytes(prep, ver, com, flops)


def footprint_report(n_nodes: int, H_v: int, H_qk: int, state_elem: int = 2,
                     u_elem: int = 4) -> dict:
    """Per sequence and layer: what commit needs kept (U, plus the k rows and log-gates it
    reads) against the N+1 states snapshotting keeps."""
    u = n_nodes * H_v * D * u_elem
    extra = n_nodes * H_qk * D * state_elem + n_nodes * H_v * 4
    one_state = H_v * D * D * state_elem
    snaps = snapshot_blocks(n_nodes) * one_state
    return {
        "U_bytes": u, "U_plus_k_and_gate_bytes": u + extra, "one_state_bytes": one_state,
        "snapshot_bytes": snaps, "snapshot_over_U": snaps / u,
        "snapshot_over_U_if_16bit": snaps / (u * 2 / u_elem),
        "blocks_snapshotting": snapshot_blocks(n_nodes), "blocks_reconstruct": 1,
    }
