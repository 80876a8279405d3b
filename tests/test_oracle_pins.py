"""Pins for the fp64 CPU oracle: everything here is fixed by the paper or by mathematics,
and none of it re-uses the oracle's own formula.

  * Eq. 1 run with the LITERAL transition matrix  alpha (I - beta k k^T)  by numpy matmuls,
    on chains and along every enumerated root-to-node path of small trees (brute force);
  * closed forms: beta = 0 (pure decay), alpha = beta = 1 with orthonormal keys (exact
    overwrite S k_i = v_i), a 2x2 single-node case worked by hand;
  * the paper's closed form (Eq. 2 solve, read-out, Eq. 3 reconstruct) written with
    numpy.linalg.solve: the paper states it equals the recurrence to ~1e-15 in fp64 and
    ~1e-7 in fp32 (Section 4);
  * tree indexing against a parent-chain walk.
Non-square states (d_v != d_k) are used so that a transposed operand cannot pass.
"""
import numpy as np
import pytest


def rng(seed):
    return np.random.default_rng(seed)


def random_tree(r, n, forest=False):
    parent = [-1]
    for i in range(1, n):
        lo = -1 if forest else 0
        parent.append(int(r.integers(lo, i)))
    return parent


def path_to(parent, i):
    p = []
    while i >= 0:
        p.append(i)
        i = parent[i]
    return p[::-1]


def draw(r, trees, H_v, H_qk, d_k, d_v, normalise=True):
    off = np.cumsum([0] + [len(t) for t in trees]).astype(np.int32)
    T, B = int(off[-1]), len(trees)
    parent = np.array([p for t in trees for p in t], np.int32)
    q = r.standard_normal((T, H_qk, d_k))
    k = r.standard_normal((T, H_qk, d_k))
    if normalise:
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((T, H_v, d_v))
    alpha = r.uniform(0.9, 0.999, (T, H_v))
    beta = r.uniform(0.1, 0.9, (T, H_v))
    S0 = 0.5 * r.standard_normal((B, H_v, d_v, d_k))
    accepted = np.array([int(r.integers(-1, len(t))) for t in trees], np.int32)
    return dict(node_offsets=off, parent=parent, S0=S0, q=q, k=k, v=v, alpha=alpha, beta=beta,
                accepted=accepted)


def literal_chain(S, ks, vs, qs, alphas, betas):
    """Eq. 1 with the transition matrix formed explicitly; returns states and outputs."""
    d_k = S.shape[1]
    states, outs = [], []
    for k, v, q, a, b in zip(ks, vs, qs, alphas, betas):
        M = a * (np.eye(d_k) - b * np.outer(k, k))
        S = S @ M + b * np.outer(v, k)
        states.append(S)
        outs.append(S @ q)
    return states, outs


# ------------------------------------------------------------------ worked by hand

def test_single_node_by_hand(oracle):
    # S0 = [[1,2],[3,4]], k = e1, v = (5,6), alpha = beta = 1/2, q = (1,1)
    # S0 (I - k k^T / 2) = [[.5,2],[1.5,4]];  * alpha = [[.25,1],[.75,2]];  + beta v k^T = [[2.5,0],[3,0]]
    S0 = np.array([[[[1.0, 2.0], [3.0, 4.0]]]])
    res = oracle.verify_commit([0, 1], [-1], S0, [[[1.0, 1.0]]], [[[1.0, 0.0]]], [[[5.0, 6.0]]],
                               [[0.5]], [[0.5]], [0])
    np.testing.assert_allclose(res.S_commit[0, 0], [[2.75, 1.0], [3.75, 2.0]], rtol=0, atol=1e-15)
    np.testing.assert_allclose(res.O[0, 0], [3.75, 5.75], rtol=0, atol=1e-15)
    # pseudo-value: beta (v - alpha S0 k) = .5 ((5,6) - .5 (1,3))
    np.testing.assert_allclose(res.U[0, 0], [2.25, 2.25], rtol=0, atol=1e-15)
    # accepted = -1 keeps the committed state
    res = oracle.verify_commit([0, 1], [-1], S0, [[[1.0, 1.0]]], [[[1.0, 0.0]]], [[[5.0, 6.0]]],
                               [[0.5]], [[0.5]], [-1])
    np.testing.assert_array_equal(res.S_commit, S0)


# ------------------------------------------------------------------ chain == Eq. 1

@pytest.mark.parametrize("n,d_k,d_v", [(4, 128, 128), (9, 6, 4), (64, 16, 8)])
def test_chain_equals_literal_recurrence(oracle, n, d_k, d_v):
    r = rng(10 + n)
    w = draw(r, [[i - 1 for i in range(n)]], 1, 1, d_k, d_v)
    w["accepted"][:] = n - 2 if n > 1 else 0
    res = oracle.verify_commit(**w, want_snapshots=True)
    states, outs = literal_chain(w["S0"][0, 0], w["k"][:, 0], w["v"][:, 0], w["q"][:, 0],
                                 w["alpha"][:, 0], w["beta"][:, 0])
    for i in range(n):
        np.testing.assert_allclose(res.Snap[i, 0], states[i], rtol=0, atol=1e-13)
        np.testing.assert_allclose(res.O[i, 0], outs[i], rtol=0, atol=1e-13)
    np.testing.assert_allclose(res.S_commit[0, 0], states[int(w["accepted"][0])], rtol=0, atol=1e-13)


# ------------------------------------------------------------------ brute force over paths

@pytest.mark.parametrize("seed", range(6))
def test_tiny_trees_by_path_enumeration(oracle, seed):
    r = rng(100 + seed)
    H_v, H_qk, d_k, d_v = 4, 2, 5, 3
    trees = [random_tree(r, int(r.integers(1, 8)), forest=(seed % 2 == 1)) for _ in range(3)]
    w = draw(r, trees, H_v, H_qk, d_k, d_v)
    res = oracle.verify_commit(**w, want_snapshots=True)
    off = w["node_offsets"]
    for b, tree in enumerate(trees):
        for h in range(H_v):
            hq = h // (H_v // H_qk)
            for i in range(len(tree)):
                rows = [off[b] + j for j in path_to(tree, i)]
                states, outs = literal_chain(w["S0"][b, h], w["k"][rows, hq], w["v"][rows, h],
                                             w["q"][rows, hq], w["alpha"][rows, h],
                                             w["beta"][rows, h])
                np.testing.assert_allclose(res.Snap[off[b] + i, h], states[-1], rtol=0, atol=1e-13)
                np.testing.assert_allclose(res.O[off[b] + i, h], outs[-1], rtol=0, atol=1e-13)
                # pseudo-value against the state BEFORE the node, from the literal walk
                S_prev = w["S0"][b, h] if len(states) == 1 else states[-2]
                t = rows[-1]
                u = w["beta"][t, h] * (w["v"][t, h] - w["alpha"][t, h] * S_prev @ w["k"][t, hq])
                np.testing.assert_allclose(res.U[t, h], u, rtol=0, atol=1e-13)
            a = int(w["accepted"][b])
            if a < 0:
                np.testing.assert_array_equal(res.S_commit[b, h], w["S0"][b, h])
            else:
                np.testing.assert_array_equal(res.S_commit[b, h], res.Snap[off[b] + a, h])


# ------------------------------------------------------------------ closed forms

def test_beta_zero_is_pure_decay(oracle):
    r = rng(7)
    trees = [random_tree(r, 12), random_tree(r, 5)]
    w = draw(r, trees, 2, 2, 8, 6)
    w["beta"][:] = 0.0
    res = oracle.verify_commit(**w, want_snapshots=True)
    off = w["node_offsets"]
    for b, tree in enumerate(trees):
        for h in range(2):
            for i in range(len(tree)):
                g = np.prod([w["alpha"][off[b] + j, h] for j in path_to(tree, i)])
                np.testing.assert_allclose(res.Snap[off[b] + i, h], g * w["S0"][b, h], rtol=1e-14)
                np.testing.assert_allclose(res.O[off[b] + i, h],
                                           g * w["S0"][b, h] @ w["q"][off[b] + i, h], rtol=0,
                                           atol=1e-14)
    assert np.all(res.U == 0.0)


def test_orthonormal_keys_overwrite_exactly(oracle):
    # alpha = beta = 1, keys orthonormal along every path: the delta rule stores v_j under
    # k_j without disturbing the others, so S_a k_j = v_j for every j on the path, and with
    # G = 0 the pseudo-values are V - K S0^T.
    r = rng(8)
    n, d_k, d_v = 10, 16, 7
    tree = random_tree(r, n)
    w = draw(r, [tree], 1, 1, d_k, d_v)
    Q, _ = np.linalg.qr(r.standard_normal((d_k, d_k)))
    w["k"][:, 0] = Q[:n]                       # all n keys mutually orthonormal
    w["alpha"][:] = 1.0
    w["beta"][:] = 1.0
    res = oracle.verify_commit(**w, want_snapshots=True)
    for i in range(n):
        for j in path_to(tree, i):
            np.testing.assert_allclose(res.Snap[i, 0] @ w["k"][j, 0], w["v"][j, 0], rtol=0,
                                       atol=1e-13)
    np.testing.assert_allclose(res.U[:, 0], w["v"][:, 0] - w["k"][:, 0] @ w["S0"][0, 0].T, rtol=0,
                               atol=1e-13)


# ------------------------------------------------------------------ the paper's closed form

def closed_form(w, b, h, H_v, H_qk, dtype=np.float64):
    """Eq. 2 (solve), the read-out, and Eq. 3 (reconstruct), with dense numpy algebra."""
    off = w["node_offsets"]
    lo, hi = int(off[b]), int(off[b + 1])
    n = hi - lo
    hq = h // (H_v // H_qk)
    parent = w["parent"][lo:hi]
    K = w["k"][lo:hi, hq].astype(dtype)
    Q = w["q"][lo:hi, hq].astype(dtype)
    V = w["v"][lo:hi, h].astype(dtype)
    al = w["alpha"][lo:hi, h].astype(dtype)
    be = w["beta"][lo:hi, h].astype(dtype)
    S0 = w["S0"][b, h].astype(dtype)
    anc = np.zeros((n, n), bool)               # anc[t, i] = i is ancestor-or-self of t
    g = np.zeros(n, dtype)
    for t in range(n):
        p = int(parent[t])
        if p >= 0:
            anc[t] = anc[p]
        anc[t, t] = True
        g[t] = al[t] * (g[p] if p >= 0 else 1.0)
    strict = anc & ~np.eye(n, dtype=bool)
    ratio = g[:, None] / g[None, :]
    G = ratio * (K @ K.T) * strict
    R = be[:, None] * V - (be * g)[:, None] * (K @ S0.T)
    Ut = np.linalg.solve(np.eye(n, dtype=dtype) + be[:, None] * G, R)
    O = g[:, None] * (Q @ S0.T) + (ratio * (Q @ K.T) * anc) @ Ut
    a = int(w["accepted"][b])
    if a < 0:
        Sa = S0
    else:
        wgt = np.where(anc[a], g[a] / g, 0).astype(dtype)
        Sa = g[a] * S0 + (wgt[:, None] * Ut).T @ K
    return Ut, O, Sa


@pytest.mark.parametrize("seed,n,d", [(0, 32, 128), (1, 64, 128), (2, 17, 24)])
def test_closed_form_matches_recurrence(oracle, seed, n, d):
    r = rng(200 + seed)
    H_v, H_qk = 2, 1
    trees = [random_tree(r, n), [i - 1 for i in range(n)]]
    w = draw(r, trees, H_v, H_qk, d, d)
    res = oracle.verify_commit(**w)
    off = w["node_offsets"]
    for b in range(2):
        for h in range(H_v):
            Ut, O, Sa = closed_form(w, b, h, H_v, H_qk)
            sl = slice(int(off[b]), int(off[b + 1]))
            np.testing.assert_allclose(res.U[sl, h], Ut, rtol=0, atol=1e-12)
            np.testing.assert_allclose(res.O[sl, h], O, rtol=0, atol=1e-12)
            np.testing.assert_allclose(res.S_commit[b, h], Sa, rtol=0, atol=1e-12)
            # the paper's fp32 figure (~1e-7) for the same closed form
            U32, O32, S32 = closed_form(w, b, h, H_v, H_qk, np.float32)
            for got, ref in ((U32, res.U[sl, h]), (O32, res.O[sl, h]), (S32, res.S_commit[b, h])):
                rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
                assert rel < 5e-6


# ------------------------------------------------------------------ invariants

def test_shared_qk_heads_equal_replicated(oracle):
    r = rng(9)
    trees = [random_tree(r, 9), random_tree(r, 3)]
    w = draw(r, trees, 4, 2, 6, 5)
    shared = oracle.verify_commit(**w)
    w2 = dict(w)
    w2["q"] = np.repeat(w["q"], 2, axis=1)
    w2["k"] = np.repeat(w["k"], 2, axis=1)
    repl = oracle.verify_commit(**w2)
    np.testing.assert_array_equal(shared.O, repl.O)
    np.testing.assert_array_equal(shared.S_commit, repl.S_commit)


def test_subtree_independence(oracle):
    # deleting a branch that is not on a node's path leaves that node untouched
    r = rng(11)
    tree = [-1, 0, 0, 1, 1, 2, 5]             # node 2's subtree: {2, 5, 6}
    w = draw(r, [tree], 1, 1, 6, 6)
    w["accepted"][:] = 4
    full = oracle.verify_commit(**w)
    keep = [0, 1, 3, 4]
    w2 = {key: (val[keep] if key in ("q", "k", "v", "alpha", "beta") else val) for key, val in w.items()}
    w2["parent"] = np.array([-1, 0, 1, 1], np.int32)
    w2["node_offsets"] = np.array([0, 4], np.int32)
    w2["accepted"] = np.array([3], np.int32)
    cut = oracle.verify_commit(**w2)
    np.testing.assert_array_equal(full.O[keep], cut.O)
    np.testing.assert_array_equal(full.U[keep], cut.U)
    np.testing.assert_array_equal(full.S_commit, cut.S_commit)


def test_commit_then_verify_composes(oracle):
    # committing node a and verifying a's subtree from S_a reproduces the original outputs
    r = rng(12)
    tree = [-1, 0, 1, 1, 3, 0]
    w = draw(r, [tree], 1, 1, 8, 5)
    w["accepted"][:] = 1
    full = oracle.verify_commit(**w)
    sub = [2, 3, 4]
    w2 = {key: (val[sub] if key in ("q", "k", "v", "alpha", "beta") else val) for key, val in w.items()}
    w2["parent"] = np.array([-1, -1, 1], np.int32)   # a forest hanging off the new state
    w2["node_offsets"] = np.array([0, 3], np.int32)
    w2["accepted"] = np.array([-1], np.int32)
    w2["S0"] = full.S_commit
    again = oracle.verify_commit(**w2)
    np.testing.assert_allclose(again.O, full.O[sub], rtol=0, atol=1e-13)
    np.testing.assert_allclose(again.U, full.U[sub], rtol=0, atol=1e-13)


# ------------------------------------------------------------------ tree indexing

@pytest.mark.parametrize("seed", range(4))
def test_prepare_against_parent_walk(oracle, seed):
    r = rng(300 + seed)
    trees = [random_tree(r, int(r.integers(1, 65)), forest=bool(seed % 2)) for _ in range(7)]
    trees += [[i - 1 for i in range(64)], [-1] * 64, [-1]]
    off = np.cumsum([0] + [len(t) for t in trees]).astype(np.int32)
    parent = np.array([p for t in trees for p in t], np.int32)
    alpha = r.uniform(0.5, 0.999, (int(off[-1]), 3))
    tr = oracle.prepare(off, parent, alpha)
    assert not tr.seq_status.any()
    for b, tree in enumerate(trees):
        depths = [len(path_to(tree, i)) - 1 for i in range(len(tree))]
        want = sorted(range(len(tree)), key=lambda i: (depths[i], i))
        assert list(tr.level_order[off[b]:off[b + 1]]) == want
        for i in range(len(tree)):
            path = path_to(tree, i)
            t = off[b] + i
            assert tr.depth[t] == len(path) - 1
            assert int(tr.anc_mask[t]) == sum(1 << j for j in path)
            assert bin(int(tr.anc_mask[t])).count("1") == tr.depth[t] + 1
            for h in range(3):
                g = np.prod([alpha[off[b] + j, h] for j in path])
                assert abs(np.exp(tr.cum_log_gate[t, h]) - g) < 1e-14


def test_malformed_sequences_are_flagged_and_skipped(oracle):
    r = rng(13)
    trees = [[-1, 0, 1], [-1, 1, 0], [-1, 0]]          # sequence 1 has parent[1] = 1 >= 1
    w = draw(r, trees, 1, 1, 4, 4)
    w["accepted"] = np.array([1, 0, 5], np.int32)     # sequence 2: accepted out of range
    res = oracle.verify_commit(**w)
    assert list(res.seq_status) == [0, oracle.SEQ_BAD_PARENT, oracle.SEQ_BAD_ACCEPTED]
    assert np.all(res.O[3:] == 0) and np.all(res.S_commit[1:] == 0) and np.any(res.O[:3] != 0)
    tr = oracle.prepare(w["node_offsets"], w["parent"], w["alpha"])
    assert list(tr.seq_status) == [0, oracle.SEQ_BAD_PARENT, 0]
    off = np.array([0, 65], np.int32)
    tr = oracle.prepare(off, np.full(65, -1, np.int32), np.full((65, 1), 0.9))
    assert list(tr.seq_status) == [oracle.SEQ_TOO_MANY_NODES]


def test_node_ranges_outside_the_packed_arrays_are_flagged_and_skipped(oracle):
    """The packed layout's own rule (the paper packs nothing): a sequence whose range of node_offsets is
    negative, runs backwards or ends past the T packed nodes the tree declares is malformed; the
    sequences around it are computed as if it were not there."""
    r = rng(17)
    trees = [[-1, 0, 1], [-1, 0, 0, 1], [-1, 0]]
    w = draw(r, trees, 1, 1, 4, 4)
    good = oracle.verify_commit(**w)
    cut = oracle.verify_commit(**w, T_declared=8)              # sequence 2 = [7, 9) sticks out of 8 nodes
    assert list(cut.seq_status) == [0, 0, oracle.SEQ_BAD_OFFSETS]
    assert np.array_equal(cut.O[:7], good.O[:7]) and np.all(cut.O[7:] == 0) and np.all(cut.S_commit[2] == 0)
    assert np.array_equal(cut.S_commit[:2], good.S_commit[:2])
    tr = oracle.prepare(w["node_offsets"], w["parent"], w["alpha"], T_declared=8)
    assert list(tr.seq_status) == [0, 0, oracle.SEQ_BAD_OFFSETS] and np.all(tr.depth[7:] == -1)
    back = dict(w, node_offsets=np.array([0, 3, 2, 9], np.int32))   # sequence 1 runs backwards
    res = oracle.verify_commit(**back)
    assert res.seq_status[1] == oracle.SEQ_BAD_OFFSETS and res.seq_status[0] == 0
    assert np.array_equal(res.O[:3], good.O[:3])
    neg = dict(w, node_offsets=np.array([-1, 3, 7, 9], np.int32))
    assert oracle.verify_commit(**neg).seq_status[0] == oracle.SEQ_BAD_OFFSETS


# ------------------------------------------------------------------ trees of more than 64 nodes

def test_wide_trees_chain_and_closed_form(oracle):
    """With the node limit raised to 128 (what the tests of the library's wide-tree calls do) the
    oracle is still the literal recurrence on a chain and the closed form on a tree; a sequence of
    129 nodes is flagged; the 64-bit masks keep the bits of the first 64 nodes only."""
    oracle.set_max_nodes(128)
    try:
        r = rng(77)
        n = 100
        w = draw(r, [[i - 1 for i in range(n)]], 1, 1, 6, 5)
        w["accepted"][:] = n - 3
        res = oracle.verify_commit(**w, want_snapshots=True)
        states, outs = literal_chain(w["S0"][0, 0], w["k"][:, 0], w["v"][:, 0], w["q"][:, 0],
                                     w["alpha"][:, 0], w["beta"][:, 0])
        for i in (0, 63, 64, 65, n - 1):
            np.testing.assert_allclose(res.Snap[i, 0], states[i], rtol=0, atol=1e-12)
            np.testing.assert_allclose(res.O[i, 0], outs[i], rtol=0, atol=1e-12)
        np.testing.assert_allclose(res.S_commit[0, 0], states[n - 3], rtol=0, atol=1e-12)

        trees = [random_tree(r, 128), random_tree(r, 70)]
        w = draw(r, trees, 2, 1, 8, 8)
        res = oracle.verify_commit(**w)
        off = w["node_offsets"]
        for b in range(2):
            for h in range(2):
                Ut, O, Sa = closed_form(w, b, h, 2, 1)
                sl = slice(int(off[b]), int(off[b + 1]))
                np.testing.assert_allclose(res.U[sl, h], Ut, rtol=0, atol=1e-11)
                np.testing.assert_allclose(res.O[sl, h], O, rtol=0, atol=1e-11)
                np.testing.assert_allclose(res.S_commit[b, h], Sa, rtol=0, atol=1e-11)
        tree = oracle.prepare(w["node_offsets"], w["parent"], w["alpha"])
        par = w["parent"]
        for i in (0, 5, 63, 64, 100, 127):                       # depth and log-gate by walking up
            d, p, acc = 0, int(par[i]), [i]
            while p >= 0:
                d, acc, p = d + 1, acc + [p], int(par[p])
            assert int(tree.depth[i]) == d
            np.testing.assert_allclose(tree.cum_log_gate[i, 0], sum(np.log(w["alpha"][j, 0]) for j in sorted(acc)),
                                       rtol=0, atol=1e-12)
            assert int(tree.anc_mask[i]) == sum(1 << j for j in acc if j < 64)

        w = draw(r, [[i - 1 for i in range(129)]], 1, 1, 4, 4)
        res = oracle.verify_commit(**w)
        assert list(res.seq_status) == [2]
    finally:
        oracle.set_max_nodes(64)
