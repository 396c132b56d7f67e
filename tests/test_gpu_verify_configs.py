"""ps_verify at the verify shapes of the five benchmark workloads, against the CPU oracle
(needs a B200): [1,5,1000] N(0,4) logits (tiny), [1,5,32000] Zipf-biased logits at temperatures
0 and 1 (the 7B- and 13B-shaped batch-1 workloads), [B,k+1,32000] for points of the 13B batch
sweep up to [64,9,32000], and [16,9,32000] (the 33B-class workload).  Each in both modes of
Algorithm 1's chain case: n_draft = n_target = k+1, and n_draft = k with the extra target row
(the bonus token).  Draft logits are the target's plus Gaussian noise (sigma 0.4: about 3.5
tokens a round at k = 4, the acceptance lengths of Table 1) and the drafts are drawn
from q, so acceptances, rejections with a residual draw and the bonus draw all occur; a single
sequence is run over several inputs and Philox offsets for the same reason.  Bit-exact, with
the two boundary exceptions enforced by harness.assert_verify_same.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from harness import assert_verify_same
from test_gpu_verify import _ctx

pytestmark = pytest.mark.gpu


def _target(kind, seed, stream, B, P, V):
    if kind == "zipf":
        return synth.zipf_logits(seed, stream, B, P, V)
    return synth.gauss_logits(seed, stream, (B, P, V))


def _run(g, toks, dl, tl, T, seed, offset):
    import paper_2410_05589_b200 as ps
    want = oracle.verify(toks, dl, tl, T, seed, offset)
    got = g.verify(ps.to_device(toks), ps.to_device(dl) if dl is not None else None, ps.to_device(tl), T, seed, offset)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in got.items()}, want


CASES = [
    # name, B, k, V, logits kind, input seed, temperatures, sigma of the draft noise
    ("tiny", 1, 4, 1000, "gauss", 0, (1.0, 0.0), 0.5),
    ("7b", 1, 4, 32000, "zipf", 2000, (1.0, 0.0), 0.4),
    ("13b", 1, 4, 32000, "zipf", 3000, (1.0, 0.0), 0.4),
    ("13b_sweep_b1_k2", 1, 2, 32000, "zipf", 4000, (1.0,), 0.4),
    ("13b_sweep_b4_k8", 4, 8, 32000, "zipf", 4000, (1.0,), 0.4),
    ("13b_sweep_b16_k4", 16, 4, 32000, "zipf", 4000, (1.0, 0.0), 0.4),
    ("13b_sweep_b64_k8", 64, 8, 32000, "zipf", 4000, (1.0,), 0.4),
    ("33b", 16, 8, 32000, "zipf", 5000, (1.0,), 0.4),
]


@pytest.mark.parametrize("mode", ["A", "B"])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_verify_at_workload_shapes(case, mode):
    name, B, k, V, kind, in_seed, temps, sigma = case
    n_target = k + 1
    n_draft = k + 1 if mode == "A" else k
    g = _ctx(V, max_batch=max(B, 2))
    reps = 12 if B == 1 else (6 if B <= 4 else 1)
    for T in temps:
        hit_reject = hit_accept = hit_full = 0
        excused = 0
        for rep in range(reps):
            tl = _target(kind, in_seed, ("vt", name, rep), B, n_target, V)
            dl = synth.noisy_draft_logits(in_seed, ("vd", name, rep), tl[:, :n_draft], sigma)
            if T > 0:
                toks = synth.sample_from_logits(in_seed, ("vx", name, rep), dl, temperature=T)
            else:
                toks = dl.argmax(-1).astype(np.int32)      # greedy drafts
            # the workloads' Philox seed is 1, the offset the iteration index
            got, want = _run(g, toks, dl if T > 0 else None, tl, T, 1, rep)
            excused += assert_verify_same(got, want, max_excused=1)
            hit_reject += int((want["accept_len"] < n_draft).sum())
            hit_accept += int((want["accept_len"] >= 1).sum())
            hit_full += int((want["accept_len"] == n_draft).sum())
            assert (want["n_out"] >= (1 if n_target > n_draft else 0)).all() and (want["n_out"] <= n_draft + 1).all()
        assert excused <= 1
        # both branches ran, and (mode B) a fully accepted chain drew its bonus token
        assert hit_reject > 0 and hit_accept > 0, (T, hit_reject, hit_accept)
        if B * reps >= 12 and T > 0:
            assert hit_full > 0, "no fully accepted chain in the sample"
    assert g.poll() == 0


def test_draft_step_then_verify_on_the_13b_shape():
    """The headline chain: ps_draft_step at the 13B shape (batch 1, k = 4, 1024 cached positions),
    its own logits and arg-max drafts handed to ps_verify with Zipf-biased target logits, the
    result compared with the oracle's verify on the kernel's logits (Eq. 1, Algorithm 1 chain
    case), at temperatures 1 and 0, both modes.  A second set of target logits is the kernel's
    logits plus noise, so that drafts are accepted."""
    import paper_2410_05589_b200 as ps
    s = synth.CONFIGS["13b"]
    W = synth.weights(s)
    L, R, V = 1024, s.rows, s.vocab
    g = ps.drafter_from_shape(s, W, max_batch=1, max_ctx=L + R)
    K, Vv = synth.kv_rows(s, ("kv", 0), L)
    g.kv_import(0, ps.to_device(K), ps.to_device(Vv))
    hl, tl_ = synth.hidden_states(s, "last", 1), synth.token_ids(s, "last", 1)
    out = g.draft_step([0], ps.to_device(hl), ps.to_device(tl_), top_n=1)
    torch.cuda.synchronize()
    logits = out["logits"].cpu().numpy()            # [1][R][V]
    toks = out["top_ids"][:, :, 0].contiguous()
    assert np.array_equal(toks.cpu().numpy(), logits.argmax(-1))
    zipf = synth.zipf_logits(s.seed, "tgt0", 1, R, V)
    near = synth.noisy_draft_logits(s.seed, "near", logits, 0.5)
    accepted = 0
    for tgt in (zipf, near):
        for T in (1.0, 0.0):
            for n_draft in (R, R - 1):
                for offset in range(4):
                    dt = toks[:, :n_draft].contiguous()
                    dlg = out["logits"][:, :n_draft].contiguous()
                    res = g.verify(dt, dlg if T > 0 else None, ps.to_device(tgt), T, 1, offset)
                    torch.cuda.synchronize()
                    got = {k2: v.cpu().numpy() for k2, v in res.items()}
                    want = oracle.verify(dt.cpu().numpy(), logits[:, :n_draft] if T > 0 else None, tgt, T, 1, offset)
                    assert_verify_same(got, want, max_excused=1)
                    accepted += int(want["accept_len"][0])
    assert accepted > 0
    assert g.poll() == 0
