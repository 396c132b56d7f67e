"""Parity of ps_draft_step / ps_kv_append with the CPU oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import synth
from harness import Pair, as_f64, check_top, logits_close

pytestmark = pytest.mark.gpu


def _compare_step(p, top_n=4, seqs=None):
    got = p.gpu_step(top_n=top_n)
    s = p.s
    worst = 0.0
    for b in (p.oracle_seqs if seqs is None else seqs):
        want = p.oracle_step(b)
        e = logits_close(got["logits"][b], want["logits"], s.dtype)
        worst = max(worst, e)
        assert e <= 1.0, (b, e)
        ef = logits_close(got["feat"][b], want["feat"], s.dtype)
        assert ef <= 1.0, (b, "feat", ef)
        for j in range(s.rows):
            wl = want["logits"][j]
            m = wl.max()
            lse = m + np.log(np.exp(wl - m).sum())
            tol = 1e-4 * max(abs(m), 1.0) if s.dtype == 0 else 1e-2 + 2e-2 * abs(m)
            assert abs(got["row_max"][b, j] - m) <= tol
            assert abs(got["row_lse"][b, j] - lse) <= tol + 2e-2 * (s.dtype == 1)
            # statistics are those of the logits the kernel itself produced
            gl = got["logits"][b, j].astype(np.float64)
            assert abs(got["row_max"][b, j] - gl.max()) <= 1e-6 * max(1.0, abs(gl.max()))
            assert abs(got["row_lse"][b, j] - (gl.max() + np.log(np.exp(gl - gl.max()).sum()))) <= 1e-4
            check_top(got["top_ids"][b, j], got["top_logit"][b, j], wl, s.dtype)
            # internal consistency: exact ranking of the kernel's own logits
            order = np.lexsort((np.arange(s.vocab), -got["logits"][b, j]))[:top_n]
            assert np.array_equal(got["top_ids"][b, j], order)
    return worst


def test_tiny_fp32_config():
    p = Pair(synth.CONFIGS["tiny"], 1)
    _compare_step(p)


def test_tiny_fp32_with_bias_and_no_context():
    p = Pair(synth.CONFIGS["tiny"], 1, with_bias=True, lens=[0])
    _compare_step(p)


def test_mini32_ragged_batch():
    s = synth.CONFIGS["mini32"]
    p = Pair(s, 3, lens=[5, 77, 0])
    _compare_step(p, top_n=8)


@pytest.mark.parametrize("flags", [0, 16, 2, 4], ids=["tcgen05", "stage_launches", "unfused", "mma_sync"])
def test_mini_bf16_ragged_batch(flags):
    """The bf16 shape on each of the kernel sets the library holds: the tcgen05 GEMMs with the
    stages on either side of the attention chained into one launch each (15 rows: some CTAs of a
    chain have no unit in a stage) or launched one by one (PS_FLAG_STAGE_LAUNCHES), the plain
    one-kernel-per-stage path (PS_FLAG_UNFUSED_KERNELS) and the mma.sync weight-streaming
    GEMMs (PS_FLAG_MMA_SYNC_GEMM); contexts built by ps_kv_append on the same path."""
    s = synth.CONFIGS["mini"]
    p = Pair(s, s.batch, flags=flags)
    _compare_step(p, top_n=8)
    assert p.g.poll() == 0


@pytest.mark.parametrize("flags", [2, 4], ids=["unfused", "mma_sync"])
def test_fallback_kernels_more_rows_gqa_and_bias(flags):
    """The two fall-back kernel sets beyond their single-launch sizes: 7 sequences x 3 rows (the
    mma.sync GEMMs take 16 rows a launch), grouped-query attention, fc bias, top-1 only."""
    s = synth.CONFIGS["mini"].with_(k_masks=2, n_kv_heads=2, batch=7, ctx_lo=3, ctx_hi=150)
    p = Pair(s, 7, flags=flags, with_bias=True)
    _compare_step(p, top_n=1)
    assert p.g.poll() == 0


def test_mini_bf16_more_masks_and_gqa():
    s = synth.CONFIGS["mini"].with_(k_masks=8, n_kv_heads=2, batch=2, ctx_lo=130, ctx_hi=300)
    p = Pair(s, 2)
    _compare_step(p, top_n=1)


def test_mini_bf16_batch_beyond_one_launch():
    """More rows than one tensor-core launch takes (30 sequences x 5 rows = 150 > 128): the
    batch runs as groups of whole sequences; every sequence is checked, and each equals what
    the same sequence gives when it runs alone."""
    s = synth.CONFIGS["mini"]
    B = 30
    rng = np.random.default_rng(3)
    p = Pair(s, B, lens=[int(x) for x in rng.integers(0, 90, B)])
    _compare_step(p, top_n=8)
    got = p.gpu_step(top_n=2)
    for b in (0, 14, 15, 29):
        one = p.g.draft_step([b], p.to_device(p.hidden_last[b:b + 1]), p.to_device(p.token_last[b:b + 1]), top_n=2)
        torch.cuda.synchronize()
        assert np.abs(one["logits"][0].cpu().numpy() - got["logits"][b]).max() <= 1e-3
    assert p.g.poll() == 0


def test_kv_append_matches_oracle_cache_and_is_incremental():
    s = synth.CONFIGS["mini"]
    p = Pair(s, 2, lens=[40, 9])
    for b in range(2):
        Ko, Vo = p.o.kv_export(b)
        Kg, Vg = p.g.kv_export(b)
        Kg, Vg = Kg.float().cpu().numpy(), Vg.float().cpu().numpy()
        # bf16 cache: a one-ulp difference (2^-8 relative) is a rounding-boundary flip
        assert np.abs(Kg - Ko).max() <= 2e-2 * np.abs(Ko).max()
        assert (np.abs(Kg - Ko) <= 2.0 ** -7 * np.abs(Ko) + 1e-3).all()
        assert (np.abs(Vg - Vo) <= 2.0 ** -7 * np.abs(Vo) + 1e-3).all()
    # appending in two calls gives the same cache as one call, up to single rounding-boundary
    # flips of the bf16 rows: the GEMM's summation order depends on the rows of a launch
    import paper_2410_05589_b200 as ps
    g2 = ps.drafter_from_shape(s, p.W, max_batch=1, max_ctx=64)
    h, t = synth.hidden_states(s, ("ctx", 0), 40), synth.token_ids(s, ("ctx", 0), 40)
    g2.kv_append([0], [17], ps.to_device(h[:17]), ps.to_device(t[:17]))
    g2.kv_append([0], [23], ps.to_device(h[17:]), ps.to_device(t[17:]))
    K2, V2 = g2.kv_export(0)
    K1, V1 = p.g.kv_export(0)
    for A, Bt in ((K1, K2), (V1, V2)):
        A, Bt = A.float(), Bt.float()
        assert (torch.abs(A - Bt) <= 2.0 ** -7 * torch.abs(A) + 1e-4).all()
        assert (A != Bt).float().mean().item() < 0.01
    # the same split of the rows into calls gives the same bits
    g3 = ps.drafter_from_shape(s, p.W, max_batch=1, max_ctx=64)
    g3.kv_append([0], [17], ps.to_device(h[:17]), ps.to_device(t[:17]))
    g3.kv_append([0], [23], ps.to_device(h[17:]), ps.to_device(t[17:]))
    K3, V3 = g3.kv_export(0)
    assert torch.equal(K2, K3) and torch.equal(V2, V3)
    assert g2.kv_len(0) == 40


def test_step_is_idempotent_and_prefix_invariant_in_batch():
    s = synth.CONFIGS["mini"]
    p = Pair(s, 3)
    a = p.gpu_step()
    b = p.gpu_step()
    for k in ("logits", "feat", "top_ids", "row_lse"):
        assert np.array_equal(a[k], b[k])
    assert [p.g.kv_len(i) for i in range(3)] == [int(x) for x in p.lens]
    # a sequence's result does not depend on its batch neighbours or its slot order
    out = p.g.draft_step([2, 0], p.to_device(p.hidden_last[[2, 0]]), p.to_device(p.token_last[[2, 0]]),
                         top_n=1)
    torch.cuda.synchronize()
    lg = out["logits"].cpu().numpy()
    # (up to re-association in fp32 and in the hi/lo split of the activations: the k range is
    # split differently for different row counts; the bound is 100x below the logits tolerance)
    np.testing.assert_allclose(lg[0], a["logits"][2], rtol=0, atol=1e-4)
    np.testing.assert_allclose(lg[1], a["logits"][0], rtol=0, atol=1e-4)


def test_argument_errors_return_status():
    import paper_2410_05589_b200 as ps
    s = synth.CONFIGS["mini32"]
    p = Pair(s, 2, lens=[3, 4])
    g = p.g
    hl, tl = p.to_device(p.hidden_last), p.to_device(p.token_last)
    with pytest.raises(ps.PsError) as e:
        g.draft_step([0, 0], hl, tl)
    assert e.value.status == -1
    with pytest.raises(ps.PsError) as e:
        g.draft_step([0, 5], hl, tl)
    assert e.value.status == -1
    with pytest.raises(ps.PsError) as e:
        g.draft_step([0, 1], hl, tl, top_n=9)
    assert e.value.status == -1
    big = 200
    with pytest.raises(ps.PsError) as e:
        g.kv_append([0], [big], p.to_device(synth.hidden_states(s, "x", big)),
                    p.to_device(synth.token_ids(s, "x", big)))
    assert e.value.status == -3
    assert g.kv_len(0) == 3
    # the context is still usable
    assert np.isfinite(p.gpu_step()["logits"]).all()
    with pytest.raises(ps.PsError):
        ps.Drafter(dtype=1, hidden=100, n_heads=2, n_kv_heads=2, head_dim=50, ffn=64, vocab=10,
                   k_masks=1, max_batch=1, max_ctx=8, weights={})


@pytest.mark.parametrize("name", ["7b", "13b", "llama3_8b"])
def test_full_size_batch1(name):
    """The 7B-, 13B- and Llama-3-8B-shaped (grouped-query attention, 128k vocabulary) batch-1
    workloads at full size; context built by ps_kv_append on
    the GPU and imported into the oracle (appends are checked above), oracle rows one by one."""
    s = synth.CONFIGS[name]
    p = Pair(s, 1, context="import", extra_ctx=8)
    _compare_step(p, top_n=1)
    # the last 8 context rows again, this time produced by ps_kv_append at full size
    L = int(p.lens[0])
    h, t = synth.hidden_states(s, "tail", 8), synth.token_ids(s, "tail", 8)
    p.g.kv_append([0], [8], p.to_device(h), p.to_device(t))
    assert p.o.kv_append(0, h, t) == 0
    Ko, Vo = p.o.kv_export(0)
    Kg, Vg = p.g.kv_export(0)
    Kg, Vg = Kg.float().cpu().numpy(), Vg.float().cpu().numpy()
    assert (np.abs(Kg[L:] - Ko[L:]) <= 2.0 ** -7 * np.abs(Ko[L:]) + 1e-2).all()
    assert (np.abs(Vg[L:] - Vo[L:]) <= 2.0 ** -7 * np.abs(Vo[L:]) + 1e-2).all()


@pytest.mark.parametrize("name,B", [("mini", 3), ("7b", 1)])
def test_chained_stages_equal_stage_launches(name, B):
    """Up to 16 rows the GEMM stages before and after the attention share a launch.  The sums are
    the same sums in the same order as with one launch per stage (PS_FLAG_STAGE_LAUNCHES), so
    every output is equal bit for bit; forty chained steps in a row leave the stage counters
    as they found them (equal outputs every time, no expired wait)."""
    import paper_2410_05589_b200 as ps
    s = synth.CONFIGS[name]
    W = synth.weights(s)
    lens = synth.ctx_lengths(s, B)
    outs = []
    for flags in (0, 16):
        g = ps.drafter_from_shape(s, W, max_batch=B, max_ctx=int(lens.max()) + s.rows + 1, flags=flags)
        for b in range(B):
            K, V = synth.kv_rows(s, ("kv", b), int(lens[b]))
            g.kv_import(b, ps.to_device(K), ps.to_device(V))
        hl, tl = ps.to_device(synth.hidden_states(s, "last", B)), ps.to_device(synth.token_ids(s, "last", B))
        first = None
        for it in range(40 if flags == 0 else 1):
            o = g.draft_step(list(range(B)), hl, tl, top_n=4, want_logits=True, want_feat=True)
            cur = {k: o[k].cpu().numpy().copy() for k in ("logits", "feat", "top_ids", "top_logit", "row_max", "row_lse")}
            if first is None:
                first = cur
            else:
                for k in cur:
                    assert np.array_equal(cur[k], first[k]), (it, k)
        assert g.poll() == 0
        outs.append(first)
    for k in outs[0]:
        assert np.array_equal(outs[0][k], outs[1][k]), k


def test_stage_timers_and_launch_timers():
    """ps_profile(ctx, 1) times every stage (a launch per GEMM stage), ps_profile(ctx, 2) every launch
    (the chained stages stay chained); the outputs do not depend on the mode."""
    s = synth.CONFIGS["mini"]
    p = Pair(s, s.batch)
    ref = p.gpu_step(top_n=2)
    seen = {}
    for mode in (1, 2):
        p.g.profile(mode)
        got = p.gpu_step(top_n=2)
        torch.cuda.synchronize()
        seen[mode] = p.g.profile_read()
        p.g.profile(0)
        assert np.array_equal(got["logits"], ref["logits"]) and np.array_equal(got["top_ids"], ref["top_ids"])
    for name in ("fc_norm", "qkv_rope", "attention", "o_proj", "ffn_gate_up", "ffn_down", "lm_head"):
        assert name in seen[1] and seen[1][name][1] >= 1, (name, seen[1])
    assert "chain_fc_qkv" in seen[2] and "chain_o_ffn_lm" in seen[2] and "attention" in seen[2], seen[2]
    assert "ffn_down" not in seen[2] and "o_proj" not in seen[2], seen[2]
    assert p.g.poll() == 0


_W13 = {}


def _weights_13b_sweep():
    if "w" not in _W13:
        _W13["w"] = synth.weights(synth.CONFIGS["13b_sweep"])
    return _W13["w"]


@pytest.mark.parametrize("B,k", [(1, 2), (4, 8), (16, 2), (16, 4), (64, 4), (64, 8)])
def test_13b_batch_sweep_sampled_sequences(B, k):
    """Points of the 13B-shaped batch / mask-count sweep at full size (ragged contexts of 256 to
    2048 positions, imported): every sequence runs on the GPU, the oracle recomputes three of
    them (the shortest, the longest and the last) row by row."""
    s = synth.CONFIGS["13b_sweep"].with_(batch=B, k_masks=k)
    lens = synth.ctx_lengths(s, B)
    seqs = sorted({int(np.argmin(lens)), int(np.argmax(lens)), B - 1})
    p = Pair(s, B, context="import", oracle_seqs=seqs, weights=_weights_13b_sweep())
    _compare_step(p, top_n=1)
    assert p.g.poll() == 0


def test_33b_batch16_k8_sampled_sequences():
    """The 33B-class shape at B=16, k=8, contexts of 1024 to 4096 positions: the oracle
    recomputes the sequence with the longest context."""
    s = synth.CONFIGS["33b"]
    lens = synth.ctx_lengths(s, s.batch)
    p = Pair(s, s.batch, context="import", oracle_seqs=[int(np.argmax(lens))])
    _compare_step(p, top_n=1)
    assert p.g.poll() == 0


@pytest.mark.parametrize("name,B", [("mini", 3), ("mini", 1), ("tiny", 1)])
def test_embedding_only_drafter(name, B):
    """PS_FLAG_NO_FC: the drafter of the Medusa integration (Sec. 4.3), no fc and no target
    feature; contexts built by ps_kv_append, the tensor-core path (mini) and the plain one."""
    s = synth.CONFIGS[name]
    p = Pair(s, B, flags=8)
    _compare_step(p, top_n=2)
    # the feature argument is not read: NULL is accepted
    out = p.g.draft_step(list(range(B)), None, p.to_device(p.token_last), top_n=2)
    torch.cuda.synchronize()
    ref = p.gpu_step(top_n=2)
    assert np.array_equal(out["logits"].cpu().numpy(), ref["logits"])
    assert p.g.poll() == 0


@pytest.mark.parametrize("name,n,max_batch", [("mini", 11, 3), ("mini", 7, 16), ("tiny", 9, 4), ("mini32", 5, 1)])
def test_group_wise_training_forward(name, n, max_batch):
    """ps_group_forward (Sec. 4.1 "Group-wise Parallel Training", Fig. 3) against the oracle's
    forward over the whole group layout; groups run in chunks of max_batch on the tensor-core
    path (a few groups) or the plain kernels, after a committed prefix."""
    import paper_2410_05589_b200 as ps
    s = synth.CONFIGS[name]
    p = Pair(s, max_batch, lens=[13] + [0] * (max_batch - 1), oracle_seqs=[0], extra_ctx=n + 4)
    h, t = synth.hidden_states(s, "grp", n), synth.token_ids(s, "grp", n)
    want = p.o.group_forward(0, h, t)
    out = p.g.group_forward(0, p.to_device(h), p.to_device(t), top_n=1, want_feat=True)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in out.items()}
    for g in range(n):
        assert logits_close(got["logits"][g], want["logits"][g], s.dtype) <= 1.0, g
        assert logits_close(got["feat"][g], want["feat"][g], s.dtype) <= 1.0, g
        for j in range(s.rows):
            check_top(got["top_ids"][g, j], got["top_logit"][g, j], want["logits"][g, j], s.dtype)
    # forward only: the context is as it was, and an ordinary draft step still agrees
    assert p.g.kv_len(0) == 13
    step = p.g.draft_step([0], p.to_device(p.hidden_last[:1]), p.to_device(p.token_last[:1]), top_n=1)
    torch.cuda.synchronize()
    ref = p.oracle_step(0)
    assert logits_close(step["logits"][0].cpu().numpy(), ref["logits"], s.dtype) <= 1.0
    assert p.g.poll() == 0


def test_bounded_device_wait_reports_timeout():
    """Every device-side wait is bounded; when one runs out the kernel raises the status word and
    returns.  A test kernel waits (2 ms at most) on a barrier nothing completes: ps_poll reports
    PS_ERR_TIMEOUT once, the context keeps working."""
    s = synth.CONFIGS["mini"]
    p = Pair(s, 1, lens=[12])
    before = p.gpu_step(top_n=1)
    p.g.debug_wait_expires(4_000_000)
    assert p.g.poll() == -5          # PS_ERR_TIMEOUT
    assert p.g.poll() == 0
    after = p.gpu_step(top_n=1)
    assert np.array_equal(before["logits"], after["logits"])


def test_workspace_guard_words_stay_intact():
    """Every slice of the workspace is followed by guard words; after appends, draft steps on both
    kernel sets' shapes, sampling, verify and the tree calls none of them has been touched.  The
    detector itself is checked by overwriting one guard byte from the host side."""
    import ctypes as C
    import paper_2410_05589_b200 as ps
    s = synth.CONFIGS["mini"]
    p = Pair(s, 3, extra_ctx=8)
    g = p.g
    out = p.g.draft_step_sampled([0, 1, 2], p.to_device(p.hidden_last), p.to_device(p.token_last), 1.0, 3, 1, top_n=4)
    tgt = ps.to_device(synth.gauss_logits(1, "gw", (3, s.rows, s.vocab)))
    g.verify(out["sampled"], out["logits"], tgt, 1.0, 1, 0)
    parent, rank = [-1, -1, 0, 0, 1], [0, 1, 0, 1, 0]
    toks = g.build_tree(parent, rank, out["top_ids"])
    g.verify_tree(parent, toks, out["logits"][:, :2].contiguous(), ps.to_device(synth.gauss_logits(1, "gt", (3, 6, s.vocab))), 1.0, 1, 0)
    g.group_forward(0, p.to_device(synth.hidden_states(s, "grp", 3)), p.to_device(synth.token_ids(s, "grp", 3)), top_n=1)
    assert g.check_guards() == 0
    ptr, nbytes = C.c_void_p(), C.c_size_t()
    assert g.lib.ps_debug_buffer(g.h, b"a", C.byref(ptr), C.byref(nbytes)) == 0
    off = ptr.value - g.workspace.data_ptr() + ((nbytes.value + 255) // 256) * 256   # first guard byte behind "a"
    g.workspace[off + 7] = 0
    assert g.check_guards() == 1
    g.workspace[off + 7] = 0x5A
    assert g.check_guards() == 0
    assert g.poll() == 0


@pytest.mark.parametrize("k,B", [(0, 1), (0, 5), (15, 1), (15, 3)])
def test_mask_count_extremes(k, B):
    """No [MASK] position at all (the step is an ordinary one-token drafter step) and the most the
    library takes (15: 16 rows per sequence), one sequence and a ragged batch."""
    s = synth.CONFIGS["mini"].with_(k_masks=k, batch=B, ctx_lo=0, ctx_hi=120)
    p = Pair(s, B)
    _compare_step(p, top_n=2)
    assert p.g.poll() == 0
