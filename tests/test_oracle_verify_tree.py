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
