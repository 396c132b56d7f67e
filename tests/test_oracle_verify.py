"""Pins for the oracle's verify path and random stream (CPU only).

  * Philox-4x32-10 against published known-answer vectors (tests/golden), plus uniformity
    and serial-correlation statistics of the 24-bit uniforms it feeds to the acceptance test;
  * Eq. 1 closed forms: P(accept) = sum_v min(p_v, q_v) = 1 - TV(p, q);
  * losslessness (Sec. 3, last paragraph; Sec. 4.2): the first emitted token follows p_0 and,
    given that x_0 was accepted, the second follows p_1 -- Monte Carlo on a 16-token vocabulary;
  * special cases whose answer is known without running the algorithm: p = q, disjoint
    supports, temperature 0, and the 1 <= n_out <= gamma+1 bound of Sec. 3.
"""
import os

import numpy as np
import pytest
from scipy import stats

import oracle
import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _softmax(z):
    z = z - z.max(-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(-1, keepdims=True)


def test_philox_known_answers(oracle_mod):
    n = 0
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.replace("->", " ").split()]
        out = oracle.philox4x32(w[4:6], w[0:4])
        assert [int(x) for x in out] == w[6:10]
        n += 1
    assert n >= 3


def test_uniforms_layout_and_statistics(oracle_mod):
    # counter = (i, b, offset_lo, offset_hi), key = (seed_lo, seed_hi); word 0 -> r, word 1 -> u2
    seed, off = (7 << 32) | 5, (3 << 32) | 9
    w = oracle.philox4x32([5, 7], [2, 11, 9, 3])
    r, u2 = oracle.uniforms(seed, off, 11, 2)
    assert r == (int(w[0]) >> 8) / 2 ** 24 and u2 == (int(w[1]) >> 8) / 2 ** 24
    us = np.array([oracle.uniforms(1, 0, b, i) for b in range(4000) for i in range(5)])
    assert us.min() >= 0.0 and us.max() < 1.0
    for col in (0, 1):
        u = us[:, col]
        hist, _ = np.histogram(u, bins=64, range=(0, 1))
        assert stats.chisquare(hist).pvalue > 1e-4
        lag1 = np.corrcoef(u[:-1], u[1:])[0, 1]
        assert abs(lag1) < 4 / np.sqrt(len(u))
    assert abs(np.corrcoef(us[:, 0], us[:, 1])[0, 1]) < 4 / np.sqrt(len(us))


def _mc_inputs(B, V=16, n=2, seed=11):
    rng = np.random.default_rng(seed)
    t = rng.normal(0, 1.5, size=(n + 1, V)).astype(np.float32)
    d = (t[:n] + rng.normal(0, 1.0, size=(n, V))).astype(np.float32)
    target = np.broadcast_to(t, (B, n + 1, V)).copy()
    draft = np.broadcast_to(d, (B, n, V)).copy()
    return t, d, target, draft


def test_monte_carlo_losslessness_and_acceptance_rate(oracle_mod):
    B, V, n = 1_000_000, 16, 2
    t, d, target, draft = _mc_inputs(B, V, n)
    p, q = _softmax(t.astype(np.float64)), _softmax(d.astype(np.float64))
    toks = synth.sample_from_logits(3, "mc", draft)             # x_i ~ q_i, drawn on the host
    res = oracle.verify(toks, draft, target, 1.0, seed=1, offset=0)
    first = res["out_tokens"][:, 0]
    assert stats.chisquare(np.bincount(first, minlength=V), p[0] * B).pvalue > 1e-3
    # Eq. 1: acceptance probability of position 0 is sum_v min(p, q)
    acc0 = (res["accept_len"] >= 1).mean()
    want = np.minimum(p[0], q[0]).sum()
    assert abs(acc0 - want) < 5 * np.sqrt(want * (1 - want) / B)
    # given x_0 accepted, the second emitted token follows p_1
    sel = res["accept_len"] >= 1
    second = res["out_tokens"][sel, 1]
    assert stats.chisquare(np.bincount(second, minlength=V), p[1] * sel.sum()).pvalue > 1e-3
    acc1 = (res["accept_len"][sel] >= 2).mean()
    want1 = np.minimum(p[1], q[1]).sum()
    assert abs(acc1 - want1) < 5 * np.sqrt(want1 * (1 - want1) / sel.sum())
    # all accepted -> one extra token from p_2 (n_target = n_draft + 1)
    full = res["accept_len"] == n
    assert (res["n_out"][full] == n + 1).all()
    third = res["out_tokens"][full, n]
    assert stats.chisquare(np.bincount(third, minlength=V), p[2] * full.sum()).pvalue > 1e-3
    # bounds and bookkeeping
    assert res["n_out"].min() >= 1 and res["n_out"].max() <= n + 1
    assert (res["n_out"] == res["accept_len"] + 1).all()
    for a in range(n + 1):
        rows = res["accept_len"] == a
        assert np.array_equal(res["out_tokens"][rows, :a], toks[rows, :a])
        assert (res["out_tokens"][rows, a + 1:] == -1).all()


def test_monte_carlo_point_mass_drafts(oracle_mod):
    # deterministic drafts with q = point mass: accept w.p. p(x); the residual is p without x
    B, V, n = 400_000, 16, 2
    t, _, target, _ = _mc_inputs(B, V, n, seed=5)
    p = _softmax(t.astype(np.float64))
    toks = np.broadcast_to(np.array([p[0].argmax(), 3], np.int32), (B, n)).copy()
    res = oracle.verify(toks, None, target, 1.0, seed=9, offset=4)
    first = res["out_tokens"][:, 0]
    assert stats.chisquare(np.bincount(first, minlength=V), p[0] * B).pvalue > 1e-3
    acc = (res["accept_len"] >= 1).mean()
    px = p[0].max()
    assert abs(acc - px) < 5 * np.sqrt(px * (1 - px) / B)


def test_temperature_scales_both_distributions(oracle_mod):
    B, V, n = 300_000, 16, 1
    t, d, target, draft = _mc_inputs(B, V, n, seed=2)
    T = 0.7
    p, q = _softmax(t.astype(np.float64) / T), _softmax(d.astype(np.float64) / T)
    toks = synth.sample_from_logits(4, "mcT", draft, temperature=T)
    res = oracle.verify(toks, draft, target, T, seed=2, offset=1)
    first = res["out_tokens"][:, 0]
    assert stats.chisquare(np.bincount(first, minlength=V), p[0] * B).pvalue > 1e-3
    want = np.minimum(p[0], q[0]).sum()
    assert abs((res["accept_len"] >= 1).mean() - want) < 5 * np.sqrt(want * (1 - want) / B)


def test_identical_distributions_accept_everything(oracle_mod):
    B, n, V = 64, 4, 100
    target = synth.gauss_logits(1, "same", (B, n + 1, V))
    draft = target[:, :n].copy()
    toks = synth.sample_from_logits(1, "same", draft)
    for n_target in (n, n + 1):
        res = oracle.verify(toks, draft, target[:, :n_target], 1.0, 1, 0)
        assert (res["accept_len"] == n).all()
        assert (res["n_out"] == n_target).all()
        assert np.array_equal(res["out_tokens"][:, :n], toks)


def test_disjoint_supports_reject_and_resample_from_target(oracle_mod):
    B, V = 200_000, 16
    t = np.full(V, -np.inf, np.float32)
    d = np.full(V, -np.inf, np.float32)
    t[:8] = np.linspace(0, 2, 8)
    d[8:] = np.linspace(0, 1, 8)
    target = np.broadcast_to(t, (B, 2, V)).copy()
    draft = np.broadcast_to(d, (B, 1, V)).copy()
    toks = synth.sample_from_logits(2, "dis", draft)
    assert toks.min() >= 8
    res = oracle.verify(toks, draft, target, 1.0, 3, 0)
    assert (res["accept_len"] == 0).all() and (res["n_out"] == 1).all()
    p = _softmax(t.astype(np.float64))
    first = res["out_tokens"][:, 0]
    assert first.max() < 8
    assert stats.chisquare(np.bincount(first, minlength=V)[:8], p[:8] * B).pvalue > 1e-3
    # q(x) = 0 under the draft but p(x) > 0: always accepted
    toks2 = np.zeros((B, 1), np.int32)
    res2 = oracle.verify(toks2[:100], draft[:100], target[:100], 1.0, 3, 0)
    assert (res2["accept_len"] == 1).all()


def test_greedy_accepts_common_prefix(oracle_mod):
    B, n, V = 50, 5, 40
    target = synth.gauss_logits(4, "g", (B, n + 1, V))
    am = target.argmax(-1).astype(np.int32)
    rng = np.random.default_rng(0)
    toks = am[:, :n].copy()
    first_bad = rng.integers(0, n + 1, size=B)
    for b in range(B):
        if first_bad[b] < n:
            toks[b, first_bad[b]] = (am[b, first_bad[b]] + 1) % V
            toks[b, first_bad[b] + 1:] = rng.integers(0, V, size=n - first_bad[b] - 1)
    res = oracle.verify(toks, None, target, 0.0, 1, 0)
    assert np.array_equal(res["accept_len"], first_bad)
    for b in range(B):
        a = first_bad[b]
        assert res["out_tokens"][b, a] == am[b, a]        # the target's own token follows
        assert res["n_out"][b] == a + 1
    # without a bonus row nothing is emitted after a fully accepted chain
    res = oracle.verify(am[:, :n], None, target[:, :n], 0.0, 1, 0)
    assert (res["n_out"] == n).all() and (res["accept_len"] == n).all()
    # ties in the target row resolve to the lower id
    tie = np.zeros((1, 1, V), np.float32)
    tie[0, 0, [5, 9]] = 3.0
    assert oracle.verify(np.array([[9]], np.int32), None, tie, 0.0, 1, 0)["out_tokens"][0, 0] == 5


def test_margins_and_nonfinite(oracle_mod):
    B, n, V = 32, 3, 64
    target = synth.gauss_logits(6, "m", (B, n + 1, V))
    draft = synth.noisy_draft_logits(6, "m", target[:, :n], 0.5)
    toks = synth.sample_from_logits(6, "m", draft)
    res = oracle.verify(toks, draft, target, 1.0, 1, 0)
    p, q = _softmax(target.astype(np.float64)), _softmax(draft.astype(np.float64))
    for b in range(B):
        for i in range(min(res["accept_len"][b] + 1, n)):
            r, _ = oracle.uniforms(1, 0, b, i)
            ratio = min(1.0, p[b, i, toks[b, i]] / q[b, i, toks[b, i]])
            assert abs(res["margin_accept"][b, i] - abs(r - ratio)) < 1e-12
        assert np.isinf(res["margin_accept"][b, res["accept_len"][b] + 1:]).all()
        assert 0.0 <= res["margin_cdf"][b] <= 1.0
    bad = target.copy()
    bad[3, 0, 10] = np.nan
    res = oracle.verify(toks, draft, bad, 1.0, 1, 0)
    assert res["nonfinite"][3] == 1 and res["accept_len"][3] == 0 and res["nonfinite"].sum() == 1
    # reading R17: the poisoned position is rejected and the arg-max over the row's non-NaN
    # target logits is emitted (NaN counts as -inf, ties to the lower id)
    row = bad[3, 0].astype(np.float64)
    row[np.isnan(row)] = -np.inf
    assert res["out_tokens"][3, 0] == int(np.argmax(row)) and res["n_out"][3] == 1
    assert (res["out_tokens"][3, 1:] == -1).all()
    bad2 = target.copy()
    bad2[5, 0, :] = -1.0
    bad2[5, 0, 0] = np.nan                       # NaN at id 0 must not win the tie among the rest
    bad2[5, 0, [7, 9]] = 2.5
    res = oracle.verify(toks, draft, bad2, 1.0, 1, 0)
    assert res["nonfinite"][5] == 1 and res["out_tokens"][5, 0] == 7
    # a poisoned DRAFT row rejects too and emits the target row's arg-max
    badd = draft.copy()
    badd[6, 0, 3] = np.inf
    res = oracle.verify(toks, badd, target, 1.0, 1, 0)
    assert res["nonfinite"][6] == 1 and res["accept_len"][6] == 0
    assert res["out_tokens"][6, 0] == int(target[6, 0].argmax())
    with pytest.raises(ValueError):
        oracle.verify(toks, draft, target[:, :2], 1.0, 1, 0)


def test_cdf_neighbours_are_the_adjacent_positive_weight_tokens(oracle_mod):
    """The verify routines report, beside the sampled token, the positive-weight tokens on either
    side of it in the running sum -- the only tokens a draw on a CDF boundary may turn into.
    Checked by brute force on a residual with many zero-weight tokens."""
    B, V = 200, 48
    target = synth.gauss_logits(8, "nb", (B, 2, V))
    draft = synth.noisy_draft_logits(8, "nb", target[:, :1], 1.5)
    toks = synth.sample_from_logits(8, "nb", draft)
    res = oracle.verify(toks, draft, target, 1.0, 4, 0)
    p, q = _softmax(target.astype(np.float64)), _softmax(draft.astype(np.float64))
    seen_zero_gap = 0
    for b in range(B):
        a = int(res["accept_len"][b])
        w = np.maximum(p[b, 0] - q[b, 0], 0.0) if a == 0 else p[b, 1]
        tok = int(res["out_tokens"][b, a])
        assert w[tok] > 0.0
        pos = np.flatnonzero(w > 0.0)
        k = int(np.searchsorted(pos, tok))
        lo = int(pos[k - 1]) if k > 0 else -1
        hi = int(pos[k + 1]) if k + 1 < len(pos) else -1
        assert list(res["neighbours"][b]) == [lo, hi], (b, tok, lo, hi, res["neighbours"][b])
        seen_zero_gap += (lo >= 0 and tok - lo > 1) or (hi >= 0 and hi - tok > 1)
    assert seen_zero_gap > 10      # the zero-weight gaps were really skipped
    # a draw at the very end of the running sum has no successor
    t1 = np.full((1, 1, V), -np.inf, np.float32)
    t1[0, 0, 5] = 0.0
    r1 = oracle.verify(np.array([[3]], np.int32), None, t1, 1.0, 1, 0)
    assert r1["out_tokens"][0, 0] == 5 and list(r1["neighbours"][0]) == [-1, -1]
