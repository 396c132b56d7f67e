"""Shared set-up for the parity tests: one oracle and one CUDA drafter on the same inputs."""
from __future__ import annotations

import numpy as np
import torch

import synth
from oracle import Oracle, OracleConfig


def oracle_for(s, W, max_batch, max_ctx, no_fc=False):
    return Oracle(OracleConfig(s.dtype, s.hidden, s.n_heads, s.n_kv_heads, s.head_dim, s.ffn,
                               s.vocab, s.k_masks, max_batch, max_ctx, s.rope_base, s.rms_eps, no_fc), W)


def as_f64(a, dtype):
    return (a if dtype == 0 else synth.bf16_bits_to_f32(a)).astype(np.float64)


class Pair:
    """Oracle + CUDA drafter with identical weights and identical caches."""

    def __init__(self, s, B, with_bias=False, context="append", lens=None, flags=0, oracle_seqs=None,
                 extra_ctx=0, weights=None):
        import paper_2410_05589_b200 as ps

        self.s, self.B = s, B
        self.W = synth.weights(s, with_bias=with_bias) if weights is None else weights
        self.lens = synth.ctx_lengths(s, B) if lens is None else np.asarray(lens, np.int32)
        max_ctx = int(self.lens.max()) + s.k_masks + 1 + extra_ctx
        self.oracle_seqs = list(range(B)) if oracle_seqs is None else list(oracle_seqs)
        self.o = oracle_for(s, self.W, B, max_ctx, no_fc=bool(flags & 8))   # 8 = PS_FLAG_NO_FC
        self.g = ps.drafter_from_shape(s, self.W, max_batch=B, max_ctx=max_ctx, flags=flags)
        self.to_device = ps.to_device
        hid, tok = [], []
        for b in range(B):
            L = int(self.lens[b])
            if context == "append":
                h, t = synth.hidden_states(s, ("ctx", b), L), synth.token_ids(s, ("ctx", b), L)
                hid.append(h)
                tok.append(t)
                if b in self.oracle_seqs:
                    assert self.o.kv_append(b, h, t) == 0
            else:
                K, V = synth.kv_rows(s, ("kv", b), L)
                if b in self.oracle_seqs:
                    self.o.kv_import(b, as_f64(K, s.dtype), as_f64(V, s.dtype))
                self.g.kv_import(b, ps.to_device(K), ps.to_device(V))
        if context == "append" and self.lens.sum() > 0:
            self.g.kv_append(list(range(B)), [int(x) for x in self.lens],
                             ps.to_device(np.concatenate(hid)), ps.to_device(np.concatenate(tok)))
        self.hidden_last = synth.hidden_states(s, "last", B)
        self.token_last = synth.token_ids(s, "last", B)

    def gpu_step(self, top_n=4, want_logits=True, want_feat=True):
        out = self.g.draft_step(list(range(self.B)), self.to_device(self.hidden_last),
                                self.to_device(self.token_last), top_n=top_n,
                                want_logits=want_logits, want_feat=want_feat)
        torch.cuda.synchronize()
        return {k: (v.cpu().numpy() if v is not None else None) for k, v in out.items()}

    def oracle_step(self, b, **kw):
        return self.o.draft_step(b, self.hidden_last[b:b + 1], int(self.token_last[b]), **kw)


def logits_close(got, want, dtype):
    """The tolerance of the logits gate: fp32 1e-4 relative (to max(|o|, row rms)); bf16
    1e-2 absolute + 2e-2 relative.  Returns the worst ratio error/bound (<= 1 passes)."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    if dtype == 0:
        rms = np.sqrt((want ** 2).mean(-1, keepdims=True))
        bound = 1e-4 * np.maximum(np.abs(want), rms)
    else:
        bound = 1e-2 + 2e-2 * np.abs(want)
    return float((np.abs(got - want) / bound).max())


def check_top(ids, vals, want_logits, dtype):
    """Top-n ids must equal the oracle's ranking unless the oracle's own gap between the
    ranks involved is inside the logits tolerance; values must match within tolerance."""
    order = np.argsort(-want_logits, kind="stable")
    n = ids.shape[-1]
    tol = (lambda x: 1e-4 * max(abs(x), float(np.sqrt((want_logits ** 2).mean())))) if dtype == 0 \
        else (lambda x: 1e-2 + 2e-2 * abs(x))
    for t in range(n):
        w = want_logits[order[t]]
        assert abs(vals[t] - w) <= 2 * tol(w), (t, vals[t], w)
        if ids[t] != order[t]:
            # allowed only when the oracle's logits of the two candidates are within tolerance
            assert abs(want_logits[ids[t]] - w) <= 2 * tol(w), (t, ids[t], order[t])


ACCEPT_BAND = 1e-6   # |r - min(1, p/q)| below which an acceptance decision may flip (the stated exception to bit-exactness)
CDF_BAND = 1e-5      # distance of the sampling point to a CDF step (fraction of the total weight) below
                     # which the emitted token may be the neighbouring positive-weight token


def assert_verify_same(got, want, max_excused=None):
    """Chain verify: accept_len / n_out / out_tokens equal the oracle's bit for bit, except where
    the oracle reports a decision on a boundary.  A differing accept length needs the first
    differing acceptance test inside ACCEPT_BAND; a differing emitted token needs the sampling
    point inside CDF_BAND AND the GPU token to be one of the two positive-weight tokens next to
    the oracle's in the running sum.  Returns the number of excused sequences."""
    B = len(want["n_out"])
    excused = 0
    for b in range(B):
        same = (got["accept_len"][b] == want["accept_len"][b] and got["n_out"][b] == want["n_out"][b]
                and np.array_equal(got["out_tokens"][b], want["out_tokens"][b]))
        if same:
            continue
        a_o, a_g = int(want["accept_len"][b]), int(got["accept_len"][b])
        if a_o != a_g:
            i = min(a_o, a_g)          # the first decision that differs
            assert want["margin_accept"][b, i] < ACCEPT_BAND, (b, i, want["margin_accept"][b, i])
            assert np.array_equal(got["out_tokens"][b, :i], want["out_tokens"][b, :i])
        else:
            assert want["margin_cdf"][b] < CDF_BAND, (b, want["margin_cdf"][b])
            assert got["n_out"][b] == want["n_out"][b]
            assert np.array_equal(got["out_tokens"][b, :a_o], want["out_tokens"][b, :a_o])
            nb = [int(x) for x in want["neighbours"][b] if x >= 0]
            assert int(got["out_tokens"][b, a_o]) in nb, (b, got["out_tokens"][b, a_o], want["out_tokens"][b, a_o], nb)
            assert (got["out_tokens"][b, a_o + 1:] == -1).all()
        excused += 1
    limit = max(1, B // 100) if max_excused is None else max_excused
    assert excused <= limit, excused
    return excused
