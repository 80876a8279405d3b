"""Randomised batches: ragged tree sizes (so that every size class, the compacted work lists of
the class launches and the small-tree kernel are exercised), odd and even numbers of value heads
per q/k head (paired and unpaired walks), a few malformed sequences.  The tensor-core kernels must
agree with the fp32 SIMT kernel on the same inputs, flag the same sequences, leave the same rows
untouched, and match the oracle on sampled sequences."""
import numpy as np
import pytest
import torch

from paper_2608_20961_b200 import workloads as wl
from tests import parity_util as pu
from tests.test_gpu_parity import _custom

pytestmark = pytest.mark.gpu


def _batch(seed):
    g = torch.Generator().manual_seed(1000 + seed)
    r = lambda n: int(torch.randint(0, n, (1,), generator=g))
    hint = (8, 16, 32, 64, 64, 64)[seed % 6]
    B = 1 + r(40) if seed < 10 else 300 + r(300)      # the last two: several units per CTA in every class
    H_qk = 1 + r(3)
    H_v = H_qk * (1 + r(4))
    sizes = [1 + r(hint) if r(4) else (1, 8, 16, 32, 64)[r(5)] for _ in range(B)]
    sizes = [min(s, hint) for s in sizes]
    trees = [wl.random_parent_tree(g, s, 1 + r(12)) for s in sizes]
    accepted = [r(s + 1) - 1 for s in sizes]                       # -1 .. s-1
    bad = set()
    if B > 3:                                                     # one malformed parent, one bad accepted node
        b1, b2 = r(B), r(B)
        if len(trees[b1]) > 2:
            trees[b1][1] = 2
            bad.add(b1)
        if b2 not in bad:
            accepted[b2] = len(trees[b2]) + 3
            bad.add(b2)
    w = _custom(trees, H_v=H_v, H_qk=H_qk, seed=seed, accepted=accepted)
    return w, hint, bad


@pytest.mark.parametrize("seed", range(12))   # seeds 10, 11: hint 64, hundreds of sequences
def test_random_ragged_batches(oracle, seed):
    w, hint, bad = _batch(seed)
    fast = pu.run_gpu(w, torch.float32, max_nodes=hint)
    slow = pu.run_gpu(w, torch.float32, max_nodes=hint, generic=True)
    assert list(fast["status"]) == list(slow["status"])
    assert {b for b in range(w.B) if fast["status"][b]} == bad
    untouched = (slow["U"] == slow["canary"])
    assert torch.equal(fast["U"] == fast["canary"], untouched)
    assert torch.equal(fast["O"] == fast["canary"], slow["O"] == slow["canary"])
    for name in ("O", "U", "S32"):
        a, b = fast[name], slow[name]
        scale = float(b[b != slow["canary"]].abs().max()) if bool((b != slow["canary"]).any()) else 1.0
        assert float((a - b).abs().max()) <= 2e-5 * max(scale, 1.0), name
    good = [b for b in range(w.B) if b not in bad]
    if good:
        picks = sorted(set(good[:: max(1, len(good) // 3)]))[:4]
        pu.assert_parity_sampled(oracle, w, fast, picks)
