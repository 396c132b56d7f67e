"""Pins for the oracle's token-tree verification (Algorithm 1 in full; CPU only).

  * a chain-shaped tree is the chain case: same decisions, tokens and uniforms as oracle.verify;
  * losslessness with several children per node drawn independently from q (Sec. 3, last
    paragraph; Algorithm 1's residual update): the first emitted token follows the target
    distribution of the root, and the token emitted after an accepted node follows that node's;
  * the probability that some child of the root is accepted, in closed form for two children:
    a + (1 - a) * sum_v min(p'_v, q_v) with a = sum_v min(p_v, q_v), p' = norm((p - q)+);
  * temperature 0: the walk follows the target's arg-max as long as a child carries it;
  * bookkeeping: the path is a root-to-node path of the tree and out_tokens spells it.
"""
import numpy as np
import pytest
from scipy import stats

import oracle
import synth


def _softmax(z):
    z = z - z.max(-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(-1, keepdims=True)


def _depths(parent):
    d = np.zeros(len(parent), np.int64)
    for i, p in enumerate(parent):
        d[i] = 0 if p < 0 else d[p] + 1
    return d


def test_chain_shaped_tree_is_the_chain_case(oracle_mod):
    B, n, V = 300, 4, 50
    target = synth.gauss_logits(3, "tc", (B, n + 1, V))
    draft = synth.noisy_draft_logits(3, "tc", target[:, :n], 0.7)
    toks = synth.sample_from_logits(3, "tc", draft)
    parent = np.arange(-1, n - 1)
    for T in (1.0, 0.5, 0.0):
        want = oracle.verify(toks, draft, target, T, seed=5, offset=2)
        got = oracle.verify_tree(parent, toks, draft, target, T, seed=5, offset=2)
        assert np.array_equal(got["accept_len"], want["accept_len"])
        assert np.array_equal(got["n_out"], want["n_out"])
        assert np.array_equal(got["out_tokens"], want["out_tokens"])
        assert want["accept_len"].min() < n and want["accept_len"].max() >= 1
        for b in range(B):
            a = got["accept_len"][b]
            assert list(got["path"][b, :a]) == list(range(a)) and (got["path"][b, a:] == -1).all()


def _mc_tree(B, V=16, seed=21):
    # root -> 3 children (nodes 0..2), each with 2 children (nodes 3..8)
    parent = np.array([-1, -1, -1, 0, 0, 1, 1, 2, 2])
    rng = np.random.default_rng(seed)
    t = rng.normal(0, 1.5, size=(len(parent) + 1, V)).astype(np.float32)       # a row per node
    d = (t[[0, 1]] * 0.6 + rng.normal(0, 1.0, size=(2, V))).astype(np.float32)  # q_0, q_1
    target = np.broadcast_to(t, (B,) + t.shape).copy()
    draft = np.broadcast_to(d, (B,) + d.shape).copy()
    depth = _depths(parent)
    # every node's token is an independent draw from the q of its depth
    per_node = np.broadcast_to(d[depth], (B, len(parent), V)).copy()
    toks = synth.sample_from_logits(seed, "mct", per_node)
    return parent, t, d, target, draft, toks


def test_monte_carlo_losslessness_with_several_children(oracle_mod):
    B, V = 600_000, 16
    parent, t, d, target, draft, toks = _mc_tree(B, V)
    p, q = _softmax(t.astype(np.float64)), _softmax(d.astype(np.float64))
    res = oracle.verify_tree(parent, toks, draft, target, 1.0, seed=3, offset=1)
    first = res["out_tokens"][:, 0]
    assert stats.chisquare(np.bincount(first, minlength=V), p[0] * B).pvalue > 1e-3
    # after an accepted child c of the root the next emitted token follows the row of node c
    for c in range(3):
        sel = res["path"][:, 0] == c
        assert sel.sum() > 20_000
        second = res["out_tokens"][sel, 1]
        assert stats.chisquare(np.bincount(second, minlength=V), p[1 + c] * sel.sum()).pvalue > 1e-3
    # more children accept more often than one child would: 1 - TV is the one-child rate
    one_child = np.minimum(p[0], q[0]).sum()
    assert (res["accept_len"] >= 1).mean() > one_child + 0.02
    # bookkeeping
    assert (res["n_out"] == res["accept_len"] + 1).all() and res["accept_len"].max() == 2
    for b in range(0, B, 997):
        a = res["accept_len"][b]
        prev = -1
        for j in range(a):
            node = res["path"][b, j]
            assert parent[node] == prev and res["out_tokens"][b, j] == toks[b, node]
            prev = node
        assert (res["path"][b, a:] == -1).all() and (res["out_tokens"][b, a + 1:] == -1).all()
        assert 0 <= res["out_tokens"][b, a] < V


def test_acceptance_probability_with_two_children(oracle_mod):
    B, V = 400_000, 16
    rng = np.random.default_rng(8)
    t = rng.normal(0, 1.5, size=(3, V)).astype(np.float32)
    d = (t[:1] * 0.5 + rng.normal(0, 1.0, size=(1, V))).astype(np.float32)
    parent = np.array([-1, -1])
    target = np.broadcast_to(t, (B, 3, V)).copy()
    draft = np.broadcast_to(d, (B, 1, V)).copy()
    toks = synth.sample_from_logits(8, "two", np.broadcast_to(d, (B, 2, V)).copy())
    res = oracle.verify_tree(parent, toks, draft, target, 1.0, seed=4, offset=0)
    p, q = _softmax(t[0].astype(np.float64)), _softmax(d[0].astype(np.float64))
    a1 = np.minimum(p, q).sum()
    resid = np.maximum(p - q, 0.0)
    resid /= resid.sum()
    want = a1 + (1 - a1) * np.minimum(resid, q).sum()
    got = (res["accept_len"] >= 1).mean()
    assert abs(got - want) < 5 * np.sqrt(want * (1 - want) / B)
    first_child = (res["path"][:, 0] == 0).mean()
    assert abs(first_child - a1) < 5 * np.sqrt(a1 * (1 - a1) / B)
    # the emitted token is distributed as p whatever happened on the way
    first = res["out_tokens"][:, 0]
    assert stats.chisquare(np.bincount(first, minlength=V), p * B).pvalue > 1e-3


def test_greedy_walk_follows_the_targets_argmax(oracle_mod):
    B, V = 40, 30
    parent = np.array([-1, -1, 0, 0, 1, 3])          # depths 0 0 1 1 1 2
    n = len(parent)
    target = synth.gauss_logits(9, "gt", (B, n + 1, V))
    am = target.argmax(-1)
    rng = np.random.default_rng(1)
    toks = rng.integers(0, V, size=(B, n)).astype(np.int32)
    want_len = np.zeros(B, np.int64)
    for b in range(B):
        # plant a path of random length: root -> 0 -> 3 -> 5
        L = rng.integers(0, 4)
        chain = [0, 3, 5][:L]
        u = 0
        for node in chain:
            toks[b, node] = am[b, u]
            u = node + 1
        # make sure no other child accidentally matches
        u, depth_ok = 0, 0
        for node in chain:
            depth_ok += 1
            u = node + 1
        kids = [i for i in range(n) if parent[i] == u - 1]
        for kid in kids:
            if kid not in chain and toks[b, kid] == am[b, u]:
                toks[b, kid] = (am[b, u] + 1) % V
        # siblings tried before a planted node must not match either
        u = 0
        for node in chain:
            for kid in [i for i in range(n) if parent[i] == u - 1 and i < node]:
                if toks[b, kid] == am[b, u]:
                    toks[b, kid] = (am[b, u] + 1) % V
            u = node + 1
        want_len[b] = L
    res = oracle.verify_tree(parent, toks, None, target, 0.0, seed=1, offset=0, max_depth=3)
    assert np.array_equal(res["accept_len"], want_len)
    for b in range(B):
        a = res["accept_len"][b]
        u = 0 if a == 0 else res["path"][b, a - 1] + 1
        assert res["out_tokens"][b, a] == am[b, u]


def test_malformed_trees_are_rejected(oracle_mod):
    V = 8
    target = np.zeros((1, 3, V), np.float32)
    draft = np.zeros((1, 1, V), np.float32)
    toks = np.zeros((1, 2), np.int32)
    with pytest.raises(ValueError):
        oracle.verify_tree(np.array([1, -1]), toks, draft, target, 1.0, 1, 0)      # parent after child
    with pytest.raises(ValueError):
        oracle.verify_tree(np.array([-1, 0]), toks, draft, target, 1.0, 1, 0)      # depth 1 needs 2 rows of q


def _full_tree(fan):
    """parent / rank lists of the tree whose nodes at depth t are all combinations of ranks
    below fan[t] (breadth-first node ids), and each node's tuple of ranks from the root."""
    parent, rank, ranks_of = [], [], []
    level = [(-1, ())]
    for f in fan:
        nxt = []
        for pid, pr in level:
            for r in range(f):
                parent.append(pid)
                rank.append(r)
                ranks_of.append(pr + (r,))
                nxt.append((len(parent) - 1, pr + (r,)))
        level = nxt
    return parent, rank, ranks_of


def test_build_tree_paths_are_the_product_of_the_top_lists(oracle_mod):
    """Drafting the tree (Algorithm 1; appendix "Token Tree Verification"): with one draft
    distribution per depth, the root-to-leaf token paths of the tree with fan-out fan[t] at depth t
    are exactly the Cartesian product of the depths' top-fan[t] lists, written here with
    itertools; a chain of rank 0 is the arg-max chain."""
    import itertools
    rng = np.random.default_rng(5)
    B, R, top_n, V = 3, 4, 4, 50
    top = np.stack([np.stack([rng.permutation(V)[:top_n] for _ in range(R)]) for _ in range(B)]).astype(np.int32)
    fan = (3, 2, 2)
    parent, rank, ranks_of = _full_tree(fan)
    toks = oracle.build_tree(parent, rank, top)
    leaves = [i for i in range(len(parent)) if i not in set(parent)]
    for b in range(B):
        paths = set()
        for leaf in leaves:
            path, i = [], leaf
            while i >= 0:
                path.append(int(toks[b, i]))
                i = parent[i]
            paths.add(tuple(reversed(path)))
        want = set(itertools.product(*[top[b, t, :fan[t]].tolist() for t in range(len(fan))]))
        assert paths == want
    chain = oracle.build_tree([-1, 0, 1, 2], [0, 0, 0, 0], top)
    assert np.array_equal(chain, top[:, :, 0])
    with pytest.raises(ValueError):
        oracle.build_tree([-1, 0, 1, 2, 3], [0] * 5, top)          # deeper than the R rows
    with pytest.raises(ValueError):
        oracle.build_tree([-1, 0], [0, top_n], top)                # rank beyond the list


def test_build_tree_with_sampled_tokens_keeps_siblings_distinct(oracle_mod):
    rng = np.random.default_rng(6)
    B, R, top_n, V = 64, 3, 4, 12
    top = np.stack([np.stack([rng.permutation(V)[:top_n] for _ in range(R)]) for _ in range(B)]).astype(np.int32)
    sampled = rng.integers(0, V, size=(B, R)).astype(np.int32)
    sampled[::2] = top[::2, :, 2]                                    # often one of the listed tokens
    parent, rank, ranks_of = _full_tree((4, 3))
    toks = oracle.build_tree(parent, rank, top, sampled)
    for b in range(B):
        for i in range(len(parent)):
            t = len(ranks_of[i]) - 1
            if rank[i] == 0:
                assert toks[b, i] == sampled[b, t]
        for p in set(parent):
            kids = [i for i in range(len(parent)) if parent[i] == p]
            assert len({int(toks[b, i]) for i in kids}) == len(kids)   # no token twice among siblings


def test_greedy_tree_round_accepts_while_the_target_token_is_listed(oracle_mod):
    """build_tree + verify_tree at temperature 0 against a closed form: with the full tree of
    fan-out n, the walk goes on exactly as long as the target's arg-max after the accepted path
    is among the drafter's n most likely tokens of that depth."""
    rng = np.random.default_rng(7)
    B, R, top_n, V = 40, 3, 3, 30
    fan = (3, 3, 3)
    parent, rank, ranks_of = _full_tree(fan)
    n = len(parent)
    top = np.stack([np.stack([rng.permutation(V)[:top_n] for _ in range(R)]) for _ in range(B)]).astype(np.int32)
    toks = oracle.build_tree(parent, rank, top)
    tl = rng.normal(0, 1, size=(B, n + 1, V)).astype(np.float32)
    # make the target's arg-max a listed token with probability ~2/3 at every decision row
    for b in range(B):
        for u in range(n + 1):
            t = 0 if u == 0 else len(ranks_of[u - 1])
            if t < R and rng.random() < 0.67:
                tl[b, u, top[b, t, rng.integers(0, top_n)]] = 9.0
    res = oracle.verify_tree(parent, toks, None, tl, 0.0, 1, 0, max_depth=len(fan))
    for b in range(B):
        u, acc = 0, 0
        while acc < len(fan):
            star = int(tl[b, u].argmax())
            kids = [i for i in range(n) if parent[i] == u - 1]
            hit = [i for i in kids if toks[b, i] == star]
            if not hit:
                break
            u, acc = hit[0] + 1, acc + 1
        assert res["accept_len"][b] == acc
        assert res["out_tokens"][b, acc] == int(tl[b, u].argmax())
    assert res["accept_len"].max() == len(fan) and res["accept_len"].min() == 0
