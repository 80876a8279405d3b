"""Seeded synthetic inputs for GDN draft-tree verify + commit.

This module only DRAWS inputs: tree topologies, q/k/v rows, gates, committed
states and accepted nodes, with the shapes of Qwen3.5-35B-A3B / 397B-A17B GDN
layers (d_k = d_v = 128; 32 or 64 value heads; chains of a few drafts, trees of
up to 64 nodes).  It holds none of the verify / commit arithmetic and is imported
by the tests and the bench, never by the CUDA library or by the CPU oracle.

All random numbers come from one ``torch.Generator`` on the CPU, seeded with
``20260800 + config_id`` unless a seed is given, and are drawn in fp32 in the fixed
order  tree -> q -> k -> v -> alpha -> beta -> S0 -> accepted.  q and k are
L2-normalised in fp32 and only then rounded to the storage dtype, so every consumer
reads the same rounded bits.

The one place a recurrence appears is ``prefix_state`` (workload 4): the committed
state there is, by the workload's definition, what a GDN layer holds after 256
random prefix tokens; it is produced with plain torch ops and is an INPUT to both
the library and the oracle -- nothing is ever compared against it.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

D = 128  # d_k = d_v of both Qwen3.5 hybrids
MAX_NODES = 64
SEED_BASE = 20260800


@dataclass
class Workload:
    """One batch of draft trees with everything verify + commit read (CPU tensors)."""
    name: str
    config_id: int
    B: int
    H_v: int
    H_qk: int
    io_dtype: torch.dtype            # storage dtype of S0, q, k, v (and of O)
    node_offsets: torch.Tensor       # int32 [B+1]
    parent: torch.Tensor             # int32 [T], local index, -1 = hangs off S0
    q: torch.Tensor                  # [T, H_qk, 128]
    k: torch.Tensor                  # [T, H_qk, 128]
    v: torch.Tensor                  # [T, H_v, 128]
    alpha: torch.Tensor              # fp32 [T, H_v]
    beta: torch.Tensor               # fp32 [T, H_v]
    S0: torch.Tensor                 # [B, H_v, 128, 128], d_k contiguous
    accepted: torch.Tensor           # int32 [B]
    seed: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def T(self) -> int:
        return int(self.parent.numel())

    @property
    def max_nodes(self) -> int:
        off = self.node_offsets
        return int((off[1:] - off[:-1]).max()) if self.B > 0 else 0

    def select_sequences(self, seqs) -> "Workload":
        """The sub-batch made of the listed sequences (all heads), repacked."""
        seqs = [int(s) for s in seqs]
        off = self.node_offsets.tolist()
        rows = [i for s in seqs for i in range(off[s], off[s + 1])]
        new_off = [0]
        for s in seqs:
            new_off.append(new_off[-1] + off[s + 1] - off[s])
        idx = torch.tensor(rows, dtype=torch.long)
        sidx = torch.tensor(seqs, dtype=torch.long)
        return Workload(
            name=self.name + f"[{len(seqs)} seqs]", config_id=self.config_id, B=len(seqs),
            H_v=self.H_v, H_qk=self.H_qk, io_dtype=self.io_dtype,
            node_offsets=torch.tensor(new_off, dtype=torch.int32),
            parent=self.parent[idx].clone(), q=self.q[idx].clone(), k=self.k[idx].clone(),
            v=self.v[idx].clone(), alpha=self.alpha[idx].clone(), beta=self.beta[idx].clone(),
            S0=self.S0[sidx].clone(), accepted=self.accepted[sidx].clone(), seed=self.seed,
            meta=dict(self.meta))


# --------------------------------------------------------------------------- trees

def _randint(g: torch.Generator, n: int) -> int:
    return int(torch.randint(0, n, (1,), generator=g).item())


def chain_tree(n: int) -> list[int]:
    """parent[i] = i - 1: a draft chain whose first node hangs off the committed state."""
    return [i - 1 for i in range(n)]


def random_parent_tree(g: torch.Generator, n: int, parent_depth_below: int) -> list[int]:
    """Node 0 is the root; node i > 0 picks its parent uniformly among the earlier
    nodes whose depth is < ``parent_depth_below`` (so depths reach that bound at most)."""
    parent, depth = [-1], [0]
    for _ in range(1, n):
        cands = [j for j, dj in enumerate(depth) if dj < parent_depth_below]
        p = cands[_randint(g, len(cands))]
        parent.append(p)
        depth.append(depth[p] + 1)
    return parent


def wide_tree(g: torch.Generator, n: int = 64) -> list[int]:
    """Root -> 8 children -> 2 children each -> 1 child each down to depth 4 (57 nodes in
    level order), then extra leaves under uniformly random earlier nodes of depth < 4."""
    parent, depth = [-1], [0]
    level = [0]
    for fan in (8, 2, 1, 1):
        nxt = []
        for p in level:
            for _ in range(fan):
                parent.append(p)
                depth.append(depth[p] + 1)
                nxt.append(len(parent) - 1)
        level = nxt
    assert len(parent) == 57
    while len(parent) < n:
        cands = [j for j, dj in enumerate(depth) if dj < 4]
        p = cands[_randint(g, len(cands))]
        parent.append(p)
        depth.append(depth[p] + 1)
    return parent[:n]


def widths_tree(widths: tuple[int, ...]) -> list[int]:
    """``draft_tree_widths`` tree in DFS pre-order: every node at level l has widths[l]
    children, the first level hangs off the committed state (N = w1 + w1 w2 + ...)."""
    parent: list[int] = []

    def grow(p: int, level: int):
        if level == len(widths):
            return
        for _ in range(widths[level]):
            parent.append(p)
            grow(len(parent) - 1, level + 1)

    grow(-1, 0)
    return parent


def tree_depths(parent: list[int]) -> list[int]:
    depth: list[int] = []
    for p in parent:
        depth.append(0 if p < 0 else depth[p] + 1)
    return depth


def tree_leaves(parent: list[int]) -> list[int]:
    has_child = set(p for p in parent if p >= 0)
    return [i for i in range(len(parent)) if i not in has_child]


# --------------------------------------------------------------------------- values

def _normalised(g, shape) -> torch.Tensor:
    x = torch.randn(shape, generator=g, dtype=torch.float32)
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-12)


def _uniform(g, shape, lo: float, hi: float) -> torch.Tensor:
    return lo + (hi - lo) * torch.rand(shape, generator=g, dtype=torch.float32)


def prefix_state(g: torch.Generator, n_units: int, n_tokens: int, alpha_rng, beta_rng,
                 device: str = "cpu") -> torch.Tensor:
    """fp32 state [n_units, 128, 128] a GDN head holds after ``n_tokens`` random tokens,
    starting from zero (the gated delta rule, Eq. 1, one token at a time).  Token inputs
    are drawn on the CPU generator; the updates run on ``device``."""
    S = torch.zeros(n_units, D, D, dtype=torch.float32, device=device)
    for _ in range(n_tokens):
        k = _normalised(g, (n_units, D)).to(device)
        v = torch.randn((n_units, D), generator=g, dtype=torch.float32).to(device)
        a = _uniform(g, (n_units, 1), *alpha_rng).to(device)
        b = _uniform(g, (n_units, 1), *beta_rng).to(device)
        Sk = torch.bmm(S, k.unsqueeze(-1)).squeeze(-1)          # what the state predicts for k
        S.mul_(a.unsqueeze(-1))
        S.baddbmm_((b * (v - a * Sk)).unsqueeze(-1), k.unsqueeze(1))
    return S.cpu()


_DEFAULTS = {
    # id: (name, B, H_v, H_qk, dtype)
    0: ("tiny-chain-fp32", 1, 1, 1, torch.float32),
    1: ("35B-chain5", 64, 32, 32, torch.bfloat16),
    2: ("35B-tree32", 256, 32, 16, torch.bfloat16),
    3: ("397B-wide64", 128, 64, 64, torch.bfloat16),
    4: ("ragged-stress", 512, 32, 32, torch.bfloat16),
    5: ("widths-3-3-3", 64, 32, 16, torch.bfloat16),
    6: ("wide128", 64, 32, 32, torch.bfloat16),
}


def make_workload(config_id: int, seed: int | None = None, B: int | None = None,
                  H_v: int | None = None, H_qk: int | None = None,
                  io_dtype: torch.dtype | None = None, prefix_device: str = "cpu",
                  prefix_tokens: int = 256) -> Workload:
    """Workloads 0-4 are the five benchmark configurations; 5 is a paper-shaped extra
    (``draft_tree_widths = (3,3,3)`` under one root, N = 40); 6 has trees of 128 nodes (random
    parents of depth < 10) for the library's wide-tree calls.  ``B``, ``H_v``, ``H_qk``
    shrink a configuration for parity tests without changing its structure."""
    name, B0, Hv0, Hqk0, dt0 = _DEFAULTS[config_id]
    B = B0 if B is None else B
    H_v = Hv0 if H_v is None else H_v
    if H_qk is None:
        H_qk = max(1, H_v // (Hv0 // Hqk0))
    io_dtype = dt0 if io_dtype is None else io_dtype
    assert H_v % H_qk == 0
    seed = SEED_BASE + config_id if seed is None else seed
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)

    alpha_rng, beta_rng = (0.9, 0.999), (0.1, 0.9)
    if config_id == 3:
        alpha_rng, beta_rng = (0.95, 0.999), (0.05, 0.95)

    # ---- trees
    trees: list[list[int]] = []
    for _ in range(B):
        if config_id == 0:
            trees.append(chain_tree(4))
        elif config_id == 1:
            trees.append(chain_tree(5))
        elif config_id == 2:
            trees.append(random_parent_tree(g, 32, 6))
        elif config_id == 3:
            trees.append(wide_tree(g, 64))
        elif config_id == 4:
            n = (1, 8, 16, 32, 64)[_randint(g, 5)]
            trees.append(random_parent_tree(g, n, 8))
        elif config_id == 5:
            trees.append([-1] + [p + 1 for p in widths_tree((3, 3, 3))])
        elif config_id == 6:
            trees.append(random_parent_tree(g, 128, 10))
        else:
            raise ValueError(config_id)
    offsets = [0]
    for t in trees:
        offsets.append(offsets[-1] + len(t))
    T = offsets[-1]
    parent = torch.tensor([p for t in trees for p in t], dtype=torch.int32)

    # ---- values, fixed draw order
    q = _normalised(g, (T, H_qk, D)).to(io_dtype)
    k = _normalised(g, (T, H_qk, D)).to(io_dtype)
    v = torch.randn((T, H_v, D), generator=g, dtype=torch.float32).to(io_dtype)
    alpha = _uniform(g, (T, H_v), *alpha_rng)
    beta = _uniform(g, (T, H_v), *beta_rng)
    if config_id == 4:
        S0 = prefix_state(g, B * H_v, prefix_tokens, alpha_rng, beta_rng, prefix_device)
        S0 = S0.view(B, H_v, D, D).to(io_dtype)
    else:
        S0 = (0.05 * torch.randn((B, H_v, D, D), generator=g, dtype=torch.float32)).to(io_dtype)

    # ---- accepted node
    acc: list[int] = []
    for t in trees:
        if config_id == 0:
            acc.append(2)
        elif config_id == 1:
            acc.append(_randint(g, 5))          # chain: node index = accepted depth
        elif config_id == 3:
            leaves = tree_leaves(t)
            acc.append(leaves[_randint(g, len(leaves))])
        elif config_id == 5:
            deep = [i for i, dpt in enumerate(tree_depths(t)) if dpt >= 2]
            acc.append(deep[_randint(g, len(deep))])
        else:
            acc.append(_randint(g, len(t)))
    return Workload(name=name, config_id=config_id, B=B, H_v=H_v, H_qk=H_qk, io_dtype=io_dtype,
                    node_offsets=torch.tensor(offsets, dtype=torch.int32), parent=parent,
                    q=q, k=k, v=v, alpha=alpha, beta=beta, S0=S0,
                    accepted=torch.tensor(acc, dtype=torch.int32), seed=seed,
                    meta={"alpha_range": alpha_rng, "beta_range": beta_rng})
