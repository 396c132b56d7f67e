"""Pins for the oracle's draft path (CPU only).

The oracle is checked against things other than itself:
  * a library Llama decoder layer (transformers) run WITHOUT any parallel-draft mask over
    context + rows 0..j: the masked single pass must give the same row j (Sec. 4.1: a row
    sees the real context and the masks of its own group only), and with no masks at all it
    must equal an ordinary one-token decoder step;
  * the parameter count printed in Sec. 5.1 "Models" (202M / 317M);
  * textbook identities of RoPE and RMSNorm observed through the oracle's taps;
  * structural invariants: a draft step does not change the cache, rows 0..j do not depend on
    how many masks follow.
"""
import numpy as np
import pytest
import torch

import synth
from oracle import Oracle, OracleConfig, row_stats


def _cfg(s, max_batch=None, max_ctx=None):
    return OracleConfig(s.dtype, s.hidden, s.n_heads, s.n_kv_heads, s.head_dim, s.ffn, s.vocab,
                        s.k_masks, max_batch or s.batch, max_ctx or (s.ctx_hi + s.k_masks + 1),
                        s.rope_base, s.rms_eps)


def _as_f64(a, dtype):
    return (a if dtype == 0 else synth.bf16_bits_to_f32(a)).astype(np.float64)


def _library_forward(s, W, x_in_rows):
    """fc -> transformers.LlamaDecoderLayer (plain causal mask) -> final norm -> LM head.

    x_in_rows: [n][2H] float64 inputs of the fc layer.  Returns logits [n][V], hdn [n][H].
    """
    from transformers import LlamaConfig
    from transformers.models.llama.modeling_llama import (LlamaDecoderLayer, LlamaRMSNorm,
                                                          LlamaRotaryEmbedding)

    cfg = LlamaConfig(hidden_size=s.hidden, num_attention_heads=s.n_heads,
                      num_key_value_heads=s.n_kv_heads, intermediate_size=s.ffn,
                      vocab_size=s.vocab, rms_norm_eps=s.rms_eps, rope_theta=s.rope_base,
                      head_dim=s.head_dim, attention_bias=False, mlp_bias=False,
                      num_hidden_layers=1)
    cfg._attn_implementation = "eager"
    layer = LlamaDecoderLayer(cfg, 0).double()
    t = lambda n: torch.from_numpy(_as_f64(W[n], s.dtype))
    with torch.no_grad():
        layer.self_attn.q_proj.weight.copy_(t("w_q"))
        layer.self_attn.k_proj.weight.copy_(t("w_k"))
        layer.self_attn.v_proj.weight.copy_(t("w_v"))
        layer.self_attn.o_proj.weight.copy_(t("w_o"))
        layer.mlp.gate_proj.weight.copy_(t("w_gate"))
        layer.mlp.up_proj.weight.copy_(t("w_up"))
        layer.mlp.down_proj.weight.copy_(t("w_down"))
        layer.input_layernorm.weight.copy_(t("g_in"))
        layer.post_attention_layernorm.weight.copy_(t("g_post"))
        final = LlamaRMSNorm(s.hidden, eps=s.rms_eps).double()
        final.weight.copy_(t("g_final"))
        n = x_in_rows.shape[0]
        x0 = torch.from_numpy(x_in_rows) @ t("w_fc").T
        if W.get("b_fc") is not None:
            x0 = x0 + t("b_fc")
        x0 = x0[None]
        pos = torch.arange(n)[None]
        cos, sin = LlamaRotaryEmbedding(cfg)(x0, pos)
        mask = torch.full((n, n), float("-inf"), dtype=torch.float64).triu(1)[None, None]
        hdn = layer(x0, attention_mask=mask, position_ids=pos, position_embeddings=(cos, sin))
        hdn = hdn[0] if isinstance(hdn, tuple) else hdn
        logits = final(hdn) @ t("w_lm").T
    return logits[0].numpy(), hdn[0].numpy()


def _inputs(s, W, ctx_hidden, ctx_tok, hid_last, tok_last, n_masks):
    """fc inputs of the unmasked sequence: context reals, last real, masks 1..n_masks."""
    E = _as_f64(W["embed"], s.dtype)
    rows = [np.concatenate([E[t], h]) for t, h in zip(ctx_tok, _as_f64(ctx_hidden, s.dtype))]
    rows.append(np.concatenate([E[tok_last], _as_f64(hid_last, s.dtype)[0]]))
    me, mf = _as_f64(W["mask_embed"], s.dtype), _as_f64(W["mask_feat"], s.dtype)
    for j in range(n_masks):
        rows.append(np.concatenate([me[j], mf[j]]))
    return np.stack(rows)


@pytest.mark.parametrize("bias", [False, True])
def test_masked_pass_equals_unmasked_library_layer(oracle_mod, bias):
    s = synth.CONFIGS["tiny"].with_(ctx_lo=11, ctx_hi=11)
    W = synth.weights(s, with_bias=bias)
    L = 11
    ctx_h, ctx_t = synth.hidden_states(s, "ctx", L), synth.token_ids(s, "ctx", L)
    hl, tl = synth.hidden_states(s, "last", 1), int(synth.token_ids(s, "last", 1)[0])
    o = Oracle(_cfg(s), W)
    assert o.kv_append(0, ctx_h, ctx_t) == 0
    got = o.draft_step(0, hl, tl)
    for j in range(s.k_masks + 1):
        # brute force: the last position of a plain causal forward over context + rows 0..j
        ref_logits, ref_hdn = _library_forward(s, W, _inputs(s, W, ctx_h, ctx_t, hl, tl, j))
        scale = np.abs(ref_logits[-1]).max()
        np.testing.assert_allclose(got["logits"][j], ref_logits[-1], rtol=0, atol=2e-5 * scale)
        np.testing.assert_allclose(got["feat"][j], ref_hdn[-1], rtol=0,
                                   atol=2e-5 * np.abs(ref_hdn[-1]).max())
    # a mistake in the mask rule is visible at this tolerance: letting row 1 miss row 0
    # (or see row 2) moves the logits by far more than 2e-5 of their scale
    assert np.abs(got["logits"][1] - got["logits"][2]).max() > 1e-3 * scale


def test_no_masks_is_an_ordinary_decoder_step(oracle_mod):
    s = synth.CONFIGS["mini32"].with_(ctx_lo=9, ctx_hi=9)
    W = synth.weights(s)
    ctx_h, ctx_t = synth.hidden_states(s, "c", 9), synth.token_ids(s, "c", 9)
    hl, tl = synth.hidden_states(s, "l", 1), int(synth.token_ids(s, "l", 1)[0])
    o = Oracle(_cfg(s), W)
    o.kv_append(0, ctx_h, ctx_t)
    k0 = o.draft_step(0, hl, tl, k_use=0)
    ref_logits, _ = _library_forward(s, W, _inputs(s, W, ctx_h, ctx_t, hl, tl, 0))
    np.testing.assert_allclose(k0["logits"][0], ref_logits[-1], rtol=0,
                               atol=2e-5 * np.abs(ref_logits).max())
    # rows 0..j of a k-mask run equal the rows of a j-mask run exactly
    full = o.draft_step(0, hl, tl)
    for j in range(s.k_masks + 1):
        part = o.draft_step(0, hl, tl, k_use=j)
        assert np.array_equal(part["logits"], full["logits"][: j + 1])


def test_gqa_against_library_layer(oracle_mod):
    s = synth.CONFIGS["mini32"].with_(n_heads=6, n_kv_heads=2, head_dim=32, hidden=192, ffn=400,
                                      vocab=300, ctx_lo=6, ctx_hi=6)
    W = synth.weights(s)
    ctx_h, ctx_t = synth.hidden_states(s, "c", 6), synth.token_ids(s, "c", 6)
    hl, tl = synth.hidden_states(s, "l", 1), int(synth.token_ids(s, "l", 1)[0])
    o = Oracle(_cfg(s), W)
    o.kv_append(0, ctx_h, ctx_t)
    got = o.draft_step(0, hl, tl)
    j = s.k_masks
    ref_logits, _ = _library_forward(s, W, _inputs(s, W, ctx_h, ctx_t, hl, tl, j))
    np.testing.assert_allclose(got["logits"][j], ref_logits[-1], rtol=0,
                               atol=2e-5 * np.abs(ref_logits).max())


def test_append_in_pieces_and_step_leaves_cache_alone(oracle_mod):
    s = synth.CONFIGS["tiny"]
    W = synth.weights(s)
    h, t = synth.hidden_states(s, "c", 10), synth.token_ids(s, "c", 10)
    hl, tl = synth.hidden_states(s, "l", 1), 3
    a = Oracle(_cfg(s, max_batch=2), W)
    a.kv_append(0, h, t)
    a.kv_append(1, h[:4], t[:4])
    a.kv_append(1, h[4:], t[4:])
    K0, V0 = a.kv_export(0)
    K1, V1 = a.kv_export(1)
    assert np.array_equal(K0, K1) and np.array_equal(V0, V1)
    r1 = a.draft_step(0, hl, tl)
    assert a.kv_len(0) == 10
    r2 = a.draft_step(0, hl, tl)               # idempotent: masks are never cached
    assert np.array_equal(r1["logits"], r2["logits"])
    Ka, Va = a.kv_export(0)
    assert np.array_equal(K0, Ka) and np.array_equal(V0, Va)
    assert a.kv_append(0, synth.hidden_states(s, "x", 60), synth.token_ids(s, "x", 60)) == -3


def test_parameter_count_matches_paper():
    # Sec. 5.1 "Models": one layer with the target's hyper-parameters is a 202M drafter for 7B
    # targets and a 317M one for 13B targets.  That is exactly q,k,v,o (4 H^2) + gate,up,down
    # (3 H F); the shared embedding / LM head and the fc layer are not part of the count.
    for name, millions in (("7b", 202), ("13b", 317)):
        s = synth.CONFIGS[name]
        W_shapes = dict(w_q=(s.hidden, s.hidden), w_k=(s.hidden, s.hidden), w_v=(s.hidden, s.hidden),
                        w_o=(s.hidden, s.hidden), w_gate=(s.ffn, s.hidden), w_up=(s.ffn, s.hidden),
                        w_down=(s.hidden, s.ffn))
        n = sum(a * b for a, b in W_shapes.values())
        assert round(n / 1e6) == millions
    # the generator produces exactly those shapes
    s = synth.CONFIGS["tiny"]
    W = synth.weights(s)
    assert W["w_gate"].shape == (s.ffn, s.hidden) and W["w_down"].shape == (s.hidden, s.ffn)
    assert W["w_fc"].shape == (s.hidden, 2 * s.hidden)


def test_rope_and_rmsnorm_identities_through_taps(oracle_mod):
    s = synth.CONFIGS["tiny"]
    W = synth.weights(s)
    # identity fc: W_fc = [I 0] so x0 = embedding; unit gains
    H = s.hidden
    W["w_fc"] = np.concatenate([np.eye(H, dtype=np.float32), np.zeros((H, H), np.float32)], 1)
    for g in ("g_in", "g_post", "g_final"):
        W[g] = np.ones(H, np.float32)
    o = Oracle(_cfg(s), W)
    hl = synth.hidden_states(s, "l", 1)
    out = o.draft_step(0, hl, 5, taps=True)
    x0, xn = out["x0"], out["xn"]
    np.testing.assert_allclose(x0[0], W["embed"][5].astype(np.float64), atol=1e-12)
    # RMSNorm: unit gains -> mean(xn^2) = ms/(ms+eps)
    ms = (x0 ** 2).mean(1)
    np.testing.assert_allclose((xn ** 2).mean(1), ms / (ms + s.rms_eps), rtol=1e-12)
    # RoPE keeps norms, head by head: |q_rot| = |W_q xn| ; row j sits at position L + j = j
    Wq = W["w_q"].astype(np.float64)
    d = s.head_dim
    for j in range(s.rows):
        plain = (Wq @ xn[j]).reshape(s.n_heads, d)
        rot = out["q"][j].reshape(s.n_heads, d)
        np.testing.assert_allclose(np.linalg.norm(rot, axis=1), np.linalg.norm(plain, axis=1), rtol=1e-12)
        if j == 0:
            np.testing.assert_allclose(rot, plain, atol=1e-14)      # position 0: no rotation
        # pairing (i, i+d/2) and the angle j * base^(-2i/d), written as complex rotation
        i = np.arange(d // 2)
        ang = j * s.rope_base ** (-2.0 * i / d)
        z = (plain[:, : d // 2] + 1j * plain[:, d // 2:]) * np.exp(1j * ang)
        np.testing.assert_allclose(rot[:, : d // 2], z.real, atol=1e-12)
        np.testing.assert_allclose(rot[:, d // 2:], z.imag, atol=1e-12)
    # relative-position property: <rope(q,m), rope(k,n)> depends on m-n only.  Row 1 attends
    # to row 0 at distance 1 whatever the context length is: same scores after shifting by L.
    o2 = Oracle(_cfg(s), W)
    ctx_h, ctx_t = synth.hidden_states(s, "c", 7), synth.token_ids(s, "c", 7)
    o2.kv_append(0, ctx_h, ctx_t)
    out2 = o2.draft_step(0, hl, 5, taps=True)
    q1a, k0a = out["q"][1].reshape(-1, d), out["k_new"][0].reshape(-1, d)
    q1b, k0b = out2["q"][1].reshape(-1, d), out2["k_new"][0].reshape(-1, d)
    np.testing.assert_allclose((q1a * k0a).sum(1), (q1b * k0b).sum(1), atol=1e-9)


def test_bf16_cache_rows_are_bf16_values(oracle_mod):
    s = synth.CONFIGS["mini"].with_(hidden=256, n_heads=2, n_kv_heads=2, ffn=512, vocab=300)
    W = synth.weights(s)
    o = Oracle(_cfg(s), W)
    o.kv_append(0, synth.hidden_states(s, "c", 5), synth.token_ids(s, "c", 5))
    K, V = o.kv_export(0)
    for a in (K, V):
        f = a.astype(np.float32)
        assert np.array_equal(f.astype(np.float64), a)
        assert np.all((f.view(np.uint32) & 0xFFFF) == 0)
    out = o.draft_step(0, synth.hidden_states(s, "l", 1), 1)
    assert np.isfinite(out["logits"]).all()


def test_bf16_storage_against_library_layer(oracle_mod):
    """The bf16 storage branch (weights, hidden states and cache given as bf16 bit patterns) against
    the library layer fed the same values widened to float64.  The fc output involves no rounding
    on either side, so it must agree to fp64 accuracy: a wrong widening of the bit patterns or a
    wrong index in the bf16 matrix product fails here.  The logits differ only by the bf16
    rounding of the k / v rows (relative 2^-9 per entry, Sec. 5.1 shapes use bf16 caches)."""
    s = synth.CONFIGS["mini"].with_(hidden=256, n_heads=2, n_kv_heads=1, ffn=520, vocab=400, k_masks=3,
                                    ctx_lo=9, ctx_hi=9)
    W = synth.weights(s)
    assert W["w_fc"].dtype == np.uint16
    L = 9
    ctx_h, ctx_t = synth.hidden_states(s, "c", L), synth.token_ids(s, "c", L)
    hl, tl = synth.hidden_states(s, "l", 1), int(synth.token_ids(s, "l", 1)[0])
    o = Oracle(_cfg(s), W)
    assert o.kv_append(0, ctx_h, ctx_t) == 0
    got = o.draft_step(0, hl, tl, taps=True)
    x_in = _inputs(s, W, ctx_h, ctx_t, hl, tl, s.k_masks)
    # (a) exact part: x_in rows and x0 = W_fc x_in of the k+1 new rows
    np.testing.assert_array_equal(got["x_in"], x_in[L:])
    x0 = x_in[L:] @ _as_f64(W["w_fc"], 1).T
    np.testing.assert_allclose(got["x0"], x0, rtol=1e-12, atol=1e-13)
    ms = (x0 ** 2).mean(1, keepdims=True)
    np.testing.assert_allclose(got["xn"], x0 / np.sqrt(ms + s.rms_eps) * _as_f64(W["g_in"], 1), rtol=1e-12)
    # (b) the whole layer: equal up to the bf16 rounding of cached k / v
    for j in (0, s.k_masks):
        ref_logits, ref_hdn = _library_forward(s, W, x_in[: L + 1 + j])
        scale = np.abs(ref_logits[-1]).max()
        err = np.abs(got["logits"][j] - ref_logits[-1]).max()
        assert err < 4e-3 * scale, (j, err, scale)
        assert err > 0.0                      # the cache really is rounded
    # (c) the new rows' k / v are what a bf16 cache slot would hold
    for name in ("k_new", "v_new"):
        f = got[name].astype(np.float32)
        assert np.array_equal(f.astype(np.float64), got[name])
        assert np.all((f.view(np.uint32) & 0xFFFF) == 0)


def test_bf16_cache_rounding_is_nearest_even(oracle_mod):
    """Values stored in a bf16 cache are rounded to nearest, ties to even (R14: the cache is a
    bf16 data structure).  Checked on exact halfway points and their fp32 neighbours, which
    truncation, round-half-up and round-half-away each get wrong somewhere."""
    s = synth.CONFIGS["mini"].with_(hidden=128, n_heads=1, n_kv_heads=1, head_dim=64, ffn=128, vocab=64)
    o = Oracle(_cfg(s, max_batch=1, max_ctx=16), synth.weights(s))
    cases = []   # (fp32 bits, expected bf16 bits)
    for hi in (0x3F80, 0x3F81, 0x4049, 0x404A, 0xC2F6, 0xC2F7, 0x0080, 0x7F7E):
        up = hi + 1
        cases += [((hi << 16) | 0x8000, hi if hi % 2 == 0 else up),   # tie: to the even neighbour
                  ((hi << 16) | 0x8001, up), ((hi << 16) | 0x7FFF, hi),
                  ((hi << 16) | 0x0001, hi), ((hi << 16) | 0xFFFF, up), (hi << 16, hi)]
    bits = np.array([c[0] for c in cases], np.uint32)
    want = (np.array([c[1] for c in cases], np.uint32) << 16).view(np.float32).astype(np.float64)
    vals = bits.view(np.float32).astype(np.float64)
    w = s.n_kv_heads * s.head_dim
    n = -(-len(vals) // w)
    K = np.zeros((n, w)); V = np.zeros((n, w))
    K.flat[: len(vals)] = vals
    V.flat[: len(vals)] = -vals
    o.kv_import(0, K, V)
    Ke, Ve = o.kv_export(0)
    np.testing.assert_array_equal(Ke.flat[: len(vals)], want)
    np.testing.assert_array_equal(Ve.flat[: len(vals)], -want)


def test_row_stats():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(3, 50))
    x[1, 7] = x[1, 9] = x[1].max() + 1.0           # a tie: the lower id comes first
    mx, lse, ids, vals = row_stats(x, 4)
    np.testing.assert_allclose(mx, x.max(1))
    np.testing.assert_allclose(lse, np.log(np.exp(x).sum(1)), rtol=1e-13)
    order = np.argsort(-x, axis=1, kind="stable")[:, :4]
    assert np.array_equal(ids, order)
    assert ids[1, 0] == 7 and ids[1, 1] == 9
    np.testing.assert_array_equal(vals, np.take_along_axis(x, order, 1))


def test_embedding_only_input_is_the_identity_fc(oracle_mod):
    """The embedding-only drafter of the Medusa integration (Sec. 4.3: shared embedding and LM
    head, no target feature) is the pinned layer with fc = [I 0]: same logits, bit for bit."""
    from oracle import Oracle, OracleConfig
    s = synth.CONFIGS["mini32"].with_(k_masks=3)
    W = synth.weights(s)
    H = s.hidden
    W_id = dict(W)
    W_id["w_fc"] = np.concatenate([np.eye(H, dtype=np.float32), np.zeros((H, H), np.float32)], 1)
    cfg = lambda no_fc: OracleConfig(s.dtype, s.hidden, s.n_heads, s.n_kv_heads, s.head_dim, s.ffn, s.vocab,
                                     s.k_masks, 1, 64, s.rope_base, s.rms_eps, no_fc)
    a, b = Oracle(cfg(True), W), Oracle(cfg(False), W_id)
    h, t = synth.hidden_states(s, "c", 20), synth.token_ids(s, "c", 20)
    assert a.kv_append(0, h, t) == 0 and b.kv_append(0, h, t) == 0
    hl, tl = synth.hidden_states(s, "l", 1), synth.token_ids(s, "l", 1)
    ra, rb = a.draft_step(0, hl, int(tl[0])), b.draft_step(0, hl, int(tl[0]))
    assert np.array_equal(ra["logits"], rb["logits"]) and np.array_equal(ra["feat"], rb["feat"])
    # and the target feature really is ignored
    rc = a.draft_step(0, hl * 3 + 1, int(tl[0]))
    assert np.array_equal(ra["logits"], rc["logits"])


def test_group_wise_training_forward_equals_inference_at_every_prefix(oracle_mod):
    """Sec. 4.1 "Group-wise Parallel Training": the parallel-group layout with its mask and
    position indices makes the drafter behave in training as in inference: group t of the one
    batched forward equals the inference draft step taken after t real tokens."""
    from oracle import Oracle, OracleConfig
    s = synth.CONFIGS["mini32"].with_(k_masks=3)
    W = synth.weights(s)
    cfg = OracleConfig(s.dtype, s.hidden, s.n_heads, s.n_kv_heads, s.head_dim, s.ffn, s.vocab, s.k_masks,
                       1, 64, s.rope_base, s.rms_eps)
    n, L0 = 9, 6
    hp, tp = synth.hidden_states(s, "pre", L0), synth.token_ids(s, "pre", L0)
    h, t = synth.hidden_states(s, "grp", n), synth.token_ids(s, "grp", n)
    a = Oracle(cfg, W)
    assert a.kv_append(0, hp, tp) == 0
    got = a.group_forward(0, h, t)
    assert a.kv_len(0) == L0                      # forward only: the cache is as it was
    b = Oracle(cfg, W)
    assert b.kv_append(0, hp, tp) == 0
    for g in range(n):
        want = b.draft_step(0, h[g:g + 1], int(t[g]))
        np.testing.assert_allclose(got["logits"][g], want["logits"], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(got["feat"][g], want["feat"], rtol=1e-12, atol=1e-12)
        assert b.kv_append(0, h[g:g + 1], t[g:g + 1]) == 0
    # a [MASK] row of another group is never seen: changing group 2's learned rows' inputs
    # (here: its real pair) leaves the [MASK] rows of group 1 untouched but moves group 3
    h2 = h.copy()
    h2[2] = synth.hidden_states(s, "other", 1)[0]
    got2 = a.group_forward(0, h2, t)
    assert np.array_equal(got2["logits"][:2], got["logits"][:2])
    assert not np.allclose(got2["logits"][3], got["logits"][3])
