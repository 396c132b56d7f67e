"""Parity of ps_verify_tree (Algorithm 1 in full) with the CPU oracle (needs a B200).

Paths, accept lengths and emitted tokens must equal the oracle's exactly, except where the
oracle itself reports that a decision sat on a boundary: some |r - min(1,p/q)| < 1e-6 on the
way, or the sampling point within 1e-5 of the total weight from a CDF step.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from test_gpu_verify import ACCEPT_BAND, CDF_BAND, _ctx

pytestmark = pytest.mark.gpu

# a 26-node tree of the shape tree drafters use: 4 children of the root, fewer further down
TREE26 = [-1, -1, -1, -1, 0, 0, 0, 1, 1, 2, 4, 4, 5, 7, 10, 10, 11, 12, 13, 14, 14, 16, 18, 19, 21, 22]


def _depths(parent):
    d = []
    for p in parent:
        d.append(0 if p < 0 else d[p] + 1)
    return np.array(d)


def _case(parent, B, V, seed, sigma=0.6, T=1.0):
    n = len(parent)
    depth = _depths(parent)
    D = int(depth.max()) + 1
    tl = synth.gauss_logits(seed, ("tt", V), (B, n + 1, V))
    # q_t: a noisy copy of the root's target row, one per depth
    dl = synth.noisy_draft_logits(seed, ("td", V), np.repeat(tl[:, :1], D, axis=1), sigma)
    toks = synth.sample_from_logits(seed, ("tx", V), dl[:, depth], temperature=max(T, 0.5))
    # make the target rows of the nodes resemble q of the next depth, so that deep paths occur
    for i in range(n):
        if depth[i] + 1 < D:
            tl[:, 1 + i] = dl[:, depth[i] + 1] + 0.5 * tl[:, 1 + i]
    return toks.astype(np.int32), dl, tl


def _run_both(g, parent, toks, dl, tl, T, seed, offset):
    import paper_2410_05589_b200 as ps
    D = int(_depths(parent).max()) + 1
    want = oracle.verify_tree(parent, toks, dl, tl, T, seed, offset, max_depth=D)
    got = g.verify_tree(list(parent), ps.to_device(toks), ps.to_device(dl) if dl is not None else None,
                        ps.to_device(tl), T, seed, offset)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in got.items()}, want


def _assert_same(got, want):
    B = len(want["n_out"])
    excused = 0
    for b in range(B):
        same = all(np.array_equal(got[k][b], want[k][b]) for k in ("accept_len", "n_out", "out_tokens", "path"))
        if same:
            continue
        if np.array_equal(got["path"][b], want["path"][b]):
            # same walk, another emitted token: only the neighbouring positive-weight token of the
            # oracle's running sum is acceptable, and only when the draw sat on a CDF step
            assert want["margin_cdf"][b] < CDF_BAND, (b, want["margin_cdf"][b])
            a = int(want["accept_len"][b])
            assert got["accept_len"][b] == a and got["n_out"][b] == want["n_out"][b]
            assert np.array_equal(got["out_tokens"][b, :a], want["out_tokens"][b, :a])
            nb = [int(x) for x in want["neighbours"][b] if x >= 0]
            assert int(got["out_tokens"][b, a]) in nb, (b, got["out_tokens"][b, a], nb)
        else:
            assert want["margin_accept"][b] < ACCEPT_BAND, (b, want["margin_accept"][b])
        excused += 1
    assert excused <= max(1, B // 100), excused


@pytest.mark.parametrize("V", [1000, 32000, 128256])
@pytest.mark.parametrize("T", [1.0, 0.6])
def test_tree_verify_matches_oracle(V, T):
    B = 64 if V < 20000 else (16 if V < 100000 else 4)
    g = _ctx(V)
    toks, dl, tl = _case(TREE26, B, V, seed=2, T=T)
    got, want = _run_both(g, TREE26, toks, dl, tl, T, seed=1, offset=3)
    _assert_same(got, want)
    if B >= 16:
        assert want["accept_len"].max() >= 2 and want["accept_len"].min() == 0   # deep and empty paths
        assert (want["path"][:, 0] > 0).any()                                   # a later sibling was taken
    # second call, new offset: the scratch (tickets) was left clean by the first
    got, want = _run_both(g, TREE26, toks, dl, tl, T, seed=1, offset=4)
    _assert_same(got, want)
    assert g.poll() == 0


def test_chain_shaped_tree_equals_ps_verify():
    import paper_2410_05589_b200 as ps
    V, B, n = 5000, 48, 5
    g = _ctx(V)
    tl = synth.gauss_logits(4, "cc", (B, n + 1, V))
    dl = synth.noisy_draft_logits(4, "cc", tl[:, :n], 0.5)
    toks = synth.sample_from_logits(4, "cc", dl)
    parent = list(range(-1, n - 1))
    for T in (1.0, 0.0):
        chain = g.verify(ps.to_device(toks), ps.to_device(dl), ps.to_device(tl), T, 7, 1)
        tree = g.verify_tree(parent, ps.to_device(toks), ps.to_device(dl), ps.to_device(tl), T, 7, 1)
        torch.cuda.synchronize()
        for k in ("accept_len", "n_out", "out_tokens"):
            assert torch.equal(chain[k], tree[k]), (T, k)


def test_greedy_tree_and_wide_fanout():
    V, B = 2000, 32
    g = _ctx(V)
    parent = [-1] * 8 + [0, 0, 3, 3]          # 8 children of the root
    toks, dl, tl = _case(parent, B, V, seed=6, sigma=1.5)
    got, want = _run_both(g, parent, toks, None, tl, 0.0, seed=1, offset=0)
    _assert_same(got, want)
    got, want = _run_both(g, parent, toks, dl, tl, 1.0, seed=1, offset=0)   # up to 8 rejections per row
    _assert_same(got, want)


def test_tree_argument_errors_and_nonfinite():
    import paper_2410_05589_b200 as ps
    V, B = 1000, 4
    g = _ctx(V)
    toks, dl, tl = _case([-1, 0, 0], B, V, seed=8)
    with pytest.raises(ps.PsError):
        g.verify_tree([0, -1, 0], ps.to_device(toks), ps.to_device(dl), ps.to_device(tl), 1.0, 1, 0)
    with pytest.raises(ps.PsError):   # draft logits are needed at T > 0
        g.verify_tree([-1, 0, 0], ps.to_device(toks), None, ps.to_device(tl), 1.0, 1, 0)
    bad = tl.copy()
    bad[2, 0, 17] = np.nan
    got, want = _run_both(g, [-1, 0, 0], toks, dl, bad, 1.0, seed=1, offset=0)
    _assert_same(got, want)
    assert want["nonfinite"][2] == 1 and got["accept_len"][2] == 0
    assert g.poll() == -6   # PS_ERR_NONFINITE


@pytest.mark.parametrize("sampled", [False, True])
def test_draft_step_build_tree_verify_tree_chain(sampled):
    """A whole tree round with nothing on the host (Algorithm 1): ps_draft_step (top-4 per row) ->
    ps_build_tree (static 26-node shape, rank = position among the siblings) -> target logits ->
    ps_verify_tree.  The top-n lists are checked against the oracle's draft step, the tree tokens
    against the oracle's build_tree bit for bit, the walk against the oracle's verify_tree on the
    kernel's draft logits, at temperatures 1 and 0."""
    import paper_2410_05589_b200 as ps
    from harness import Pair, check_top
    s = synth.CONFIGS["mini"].with_(k_masks=5)
    B = 3
    p = Pair(s, B, lens=[21, 60, 5])
    parent = TREE26
    depth = _depths(parent)
    rank = []
    for i, par in enumerate(parent):
        rank.append(sum(1 for j in range(i) if parent[j] == par))
    D = int(depth.max()) + 1
    assert D <= s.rows and max(rank) < 4
    hl, tl_ = p.to_device(p.hidden_last), p.to_device(p.token_last)
    if sampled:
        out = p.g.draft_step_sampled(list(range(B)), hl, tl_, 1.0, 5, 2, top_n=4)
    else:
        out = p.g.draft_step(list(range(B)), hl, tl_, top_n=4)
    toks_d = p.g.build_tree(parent, rank, out["top_ids"], out["sampled"] if sampled else None)
    torch.cuda.synchronize()
    top_ids = out["top_ids"].cpu().numpy()
    for b in range(B):
        want = p.oracle_step(b)
        for j in range(s.rows):
            check_top(top_ids[b, j], out["top_logit"][b, j].cpu().numpy(), want["logits"][j], s.dtype)
    toks = toks_d.cpu().numpy()
    smp = out["sampled"].cpu().numpy() if sampled else None
    assert np.array_equal(toks, oracle.build_tree(parent, rank, top_ids, smp))
    for b in range(B):          # siblings carry distinct tokens
        for par in set(parent):
            kids = [i for i in range(len(parent)) if parent[i] == par]
            assert len({int(toks[b, i]) for i in kids}) == len(kids)
    dl = out["logits"][:, :D].contiguous()
    dl_np = dl.cpu().numpy()
    # target rows: the drafter's row of the node's depth plus noise, so that deep paths occur
    tgt = synth.gauss_logits(9, "chain_t", (B, len(parent) + 1, s.vocab), sigma=1.0)
    tgt[:, 0] += dl_np[:, 0]
    for i in range(len(parent)):
        if depth[i] + 1 < D:
            tgt[:, 1 + i] += dl_np[:, depth[i] + 1]
    hits = 0
    for T in (1.0, 0.0):
        for off in range(4):
            got = p.g.verify_tree(parent, toks_d, dl, ps.to_device(tgt), T, 3, off)
            torch.cuda.synchronize()
            got = {k: v.cpu().numpy() for k, v in got.items()}
            want = oracle.verify_tree(parent, toks, dl_np, tgt, T, 3, off, max_depth=D)
            _assert_same(got, want)
            hits += int(want["accept_len"].sum())
    assert hits > 0
    # malformed requests come back as a status
    with pytest.raises(ps.PsError):
        p.g.build_tree([-1, -1], [0, 0], out["top_ids"])            # two siblings of one rank
    with pytest.raises(ps.PsError):
        p.g.build_tree([-1, 0], [0, 4], out["top_ids"])             # rank beyond top_n
    with pytest.raises(ps.PsError):
        p.g.build_tree(list(range(-1, 6)), [0] * 7, out["top_ids"])  # deeper than k+1 rows
    assert p.g.poll() == 0
