"""Parity of ps_verify (and the device Philox stream) with the CPU oracle (needs a B200).

Accept lengths and emitted tokens must equal the oracle's exactly, except where the oracle
itself reports that the decision sat on a boundary: |r - min(1,p/q)| < 1e-6 for an acceptance
test, or the sampling point within 1e-5 of the total weight from a CDF step.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from harness import ACCEPT_BAND, CDF_BAND, assert_verify_same

pytestmark = pytest.mark.gpu


def _ctx(V, max_batch=128):
    """A minimal context whose only job is to own the verify scratch (tiny drafter, vocab V)."""
    import paper_2410_05589_b200 as ps
    s = synth.CONFIGS["tiny"].with_(vocab=V, hidden=64, n_heads=1, n_kv_heads=1, ffn=64, k_masks=1)
    W = synth.weights(s)
    return ps.drafter_from_shape(s, W, max_batch=max_batch, max_ctx=8)


def _run_both(g, toks, dl, tl, T, seed, offset):
    import paper_2410_05589_b200 as ps
    want = oracle.verify(toks, dl, tl, T, seed, offset)
    got = g.verify(ps.to_device(toks), ps.to_device(dl) if dl is not None else None,
                   ps.to_device(tl), T, seed, offset)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in got.items()}
    return got, want


def _assert_same(got, want, n_draft):
    return assert_verify_same(got, want)


def test_device_philox_equals_oracle_words():
    import paper_2410_05589_b200 as ps
    rng = np.random.default_rng(0)
    n = 100_000
    ctr = rng.integers(0, 2 ** 32, size=(n, 4), dtype=np.uint64).astype(np.uint32)
    ctr[:3] = [[0, 0, 0, 0], [0xFFFFFFFF] * 4, [0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344]]
    key = [0xA4093822, 0x299F31D0]
    out = ps.philox_fill(key, torch.from_numpy(ctr.view(np.int32)).cuda()).cpu().numpy().view(np.uint32)
    assert [hex(x) for x in out[2]] == ["0xd16cfe09", "0x94fdcceb", "0x5001e420", "0x24126ea1"]
    for i in list(range(64)) + list(rng.integers(0, n, 400)):
        assert np.array_equal(out[i], oracle.philox4x32(key, ctr[i]))
    zero = ps.philox_fill([0, 0], torch.zeros((1, 4), dtype=torch.int32, device="cuda")).cpu().numpy().view(np.uint32)
    assert [hex(x) for x in zero[0]] == ["0x6627e8d5", "0xe169c58d", "0xbc57ac4c", "0x9b00dbd8"]


@pytest.mark.parametrize("V,n_draft,bonus", [(1000, 16, 0), (32000, 15, 1), (1000, 5, 0), (1000, 4, 1), (5003, 3, 1), (130, 1, 0),
                                            (32000, 4, 1), (65536, 2, 1), (8, 1, 1), (65540, 1, 1), (128256, 2, 1),
                                            (131070, 1, 1)])
@pytest.mark.parametrize("T", [1.0, 0.6])
def test_stochastic_verify_matches_oracle(V, n_draft, bonus, T):
    # vocabularies that are a multiple of 4 take the cluster kernel (8 blocks per row up to 65536,
    # 16 up to 131072; 4 blocks up to 32768 when the batch's 8-block clusters exceed the SMs, as
    # these batches do), the rest the one-block-per-row kernel
    B = 96 if V < 20000 else 24
    g = _ctx(V)
    tl = synth.gauss_logits(1, ("t", V), (B, n_draft + bonus, V))
    dl = synth.noisy_draft_logits(1, ("d", V), tl[:, :n_draft], 0.6)
    toks = synth.sample_from_logits(1, ("x", V), dl, temperature=T)
    got, want = _run_both(g, toks, dl, tl, T, seed=1, offset=7)
    _assert_same(got, want, n_draft)
    assert want["accept_len"].min() < n_draft and want["accept_len"].max() >= 1   # both branches hit
    # second call, new offset: scratch (tickets) was left clean by the first
    got, want = _run_both(g, toks, dl, tl, T, seed=1, offset=8)
    _assert_same(got, want, n_draft)
    assert g.poll() == 0


def test_point_mass_drafts_and_greedy():
    V, B, n = 2000, 64, 5
    g = _ctx(V)
    tl = synth.zipf_logits(2, "pm", B, n + 1, V)
    toks = tl[:, :n].argmax(-1).astype(np.int32)
    toks[::3, 2] = 7
    got, want = _run_both(g, toks, None, tl, 1.0, seed=5, offset=0)
    _assert_same(got, want, n)
    for nt in (n, n + 1):
        got, want = _run_both(g, toks, None, tl[:, :nt], 0.0, seed=5, offset=0)
        for k in ("accept_len", "n_out", "out_tokens"):
            assert np.array_equal(got[k], want[k])
    # ties resolve to the lower id on both sides
    tie = np.zeros((1, 1, V), np.float32)
    tie[0, 0, [40, 1500]] = 2.0
    got, want = _run_both(g, np.array([[1500]], np.int32), None, tie, 0.0, 1, 0)
    assert got["out_tokens"][0, 0] == want["out_tokens"][0, 0] == 40


def test_identical_and_disjoint_distributions():
    V, B, n = 512, 32, 4
    g = _ctx(V)
    tl = synth.gauss_logits(3, "same", (B, n + 1, V))
    dl = tl[:, :n].copy()
    toks = synth.sample_from_logits(3, "same", dl)
    got, want = _run_both(g, toks, dl, tl, 1.0, 2, 0)
    assert (got["accept_len"] == n).all() and (got["n_out"] == n + 1).all()
    _assert_same(got, want, n)
    t = np.full((B, 2, V), -np.inf, np.float32)
    d = np.full((B, 1, V), -np.inf, np.float32)
    t[:, :, :100] = synth.gauss_logits(3, "dj", (B, 2, 100))
    d[:, :, 100:] = synth.gauss_logits(3, "dk", (B, 1, V - 100))
    toks = synth.sample_from_logits(3, "dj", d)
    got, want = _run_both(g, toks, d, t, 1.0, 2, 0)
    assert (got["accept_len"] == 0).all() and (got["out_tokens"][:, 0] < 100).all()
    _assert_same(got, want, 1)
    assert g.poll() == 0


def test_nonfinite_logits_set_status_not_a_fault():
    V, B, n = 300, 8, 3
    g = _ctx(V)
    tl = synth.gauss_logits(4, "nf", (B, n, V))
    dl = synth.noisy_draft_logits(4, "nf", tl, 0.3)
    toks = synth.sample_from_logits(4, "nf", dl)
    tl[2, 0, 17] = np.nan
    got, want = _run_both(g, toks, dl, tl, 1.0, 1, 0)
    assert want["nonfinite"][2] == 1
    for k in ("accept_len", "n_out"):
        assert got[k][2] == want[k][2]
    assert got["out_tokens"][2, 0] == want["out_tokens"][2, 0]
    assert g.poll() == -6          # PS_ERR_NONFINITE, reported once
    assert g.poll() == 0
    import paper_2410_05589_b200 as ps
    with pytest.raises(ps.PsError):
        g.verify(ps.to_device(toks), None, ps.to_device(tl[:, :1]), 1.0, 1, 0)


def test_monte_carlo_losslessness_on_device():
    """Sec. 3 / Sec. 4.2: the emitted token follows the target distribution (16-token vocabulary)."""
    from scipy import stats
    import paper_2410_05589_b200 as ps
    V, n, B, reps = 16, 2, 128, 400
    g = _ctx(V)
    rng = np.random.default_rng(11)
    t = rng.normal(0, 1.5, size=(n + 1, V)).astype(np.float32)
    d = (t[:n] + rng.normal(0, 1.0, size=(n, V))).astype(np.float32)
    p = np.exp(t[0].astype(np.float64)); p /= p.sum()
    tl = ps.to_device(np.broadcast_to(t, (B, n + 1, V)).copy())
    dl_np = np.broadcast_to(d, (B, n, V)).copy()
    dl = ps.to_device(dl_np)
    counts = np.zeros(V)
    for r in range(reps):
        toks = synth.sample_from_logits(5, ("mc", r), dl_np)
        out = g.verify(ps.to_device(toks), dl, tl, 1.0, seed=3, offset=r)
        counts += np.bincount(out["out_tokens"][:, 0].cpu().numpy(), minlength=V)
    assert stats.chisquare(counts, p * B * reps).pvalue > 1e-3
