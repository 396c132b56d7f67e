"""ps_verify_static against ps_verify (needs a B200).  Collected last on purpose.

ps_verify_static serves callers that may not allocate device memory at all -- a serving
process whose memory was handed to a pool at start-up, a plugin living under someone else's
allocator -- and therefore cannot own the workspace a context needs.  Its scratch is a fixed
array inside the library.  The test checks that, through the C ABI, it returns exactly what the
context-based entry point returns (the outputs are integers, so the tolerance is equality), on
two calls in a row: the second call finds the first call's leftovers in the shared array.
"""
import numpy as np
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu


def _case(V, B, n_draft, bonus, T, seed):
    tl = synth.gauss_logits(seed, ("zt", V), (B, n_draft + bonus, V))
    dl = synth.noisy_draft_logits(seed, ("zd", V), tl[:, :n_draft], 0.6)
    toks = synth.sample_from_logits(seed, ("zx", V), dl, temperature=max(T, 0.5))
    return toks, dl, tl


def test_static_scratch_verify_equals_context_verify_twice():
    import paper_2410_05589_b200 as ps

    V, B, n_draft = 3001, 40, 4
    s = synth.CONFIGS["tiny"].with_(vocab=V, hidden=64, n_heads=1, n_kv_heads=1, ffn=64, k_masks=1)
    g = ps.drafter_from_shape(s, synth.weights(s), max_batch=B, max_ctx=8)
    out = {"accept_len": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
           "out_tokens": torch.full((B, n_draft + 1), -7, dtype=torch.int32, device="cuda"),
           "n_out": torch.full((B,), -7, dtype=torch.int32, device="cuda")}
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    for call, (bonus, T, with_q) in enumerate([(1, 1.0, True), (0, 0.7, True), (1, 0.0, False)]):
        toks, dl, tl = _case(V, B, n_draft, bonus, T, seed=20 + call)
        d_toks, d_tl = ps.to_device(toks), ps.to_device(tl)
        d_dl = ps.to_device(dl) if with_q else None
        want = g.verify(d_toks, d_dl, d_tl, T, seed=9, offset=call)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        got = ps.verify_static(d_toks, d_dl, d_tl, T, seed=9, offset=call, out=out, nonfinite_flag=flag)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        for k in ("accept_len", "n_out", "out_tokens"):
            assert torch.equal(got[k], want[k]), (call, k)
        assert want["accept_len"].min().item() >= 0
    assert flag.item() == 0
    # a non-finite logit is reported through the caller's flag
    toks, dl, tl = _case(V, B, n_draft, 0, 1.0, seed=30)
    tl[0, 0, 5] = np.nan
    ps.verify_static(ps.to_device(toks), ps.to_device(dl), ps.to_device(tl), 1.0, 1, 0, out=out,
                     nonfinite_flag=flag)
    torch.cuda.synchronize()
    assert flag.item() == 1


def test_static_scratch_limits_are_reported():
    import paper_2410_05589_b200 as ps

    out = {"accept_len": torch.zeros(129, dtype=torch.int32, device="cuda"),
           "out_tokens": torch.zeros((129, 3), dtype=torch.int32, device="cuda"),
           "n_out": torch.zeros(129, dtype=torch.int32, device="cuda")}
    toks = torch.zeros((129, 2), dtype=torch.int32, device="cuda")
    tl = torch.zeros((129, 2, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(ps.PsError) as e:
        ps.verify_static(toks, None, tl, 1.0, 1, 0, out=out)
    assert e.value.status == -3 and "PS_STATIC_MAX_BATCH" in str(e.value)
    toks17 = torch.zeros((2, 17), dtype=torch.int32, device="cuda")
    tl17 = torch.zeros((2, 17, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(ps.PsError) as e:
        ps.verify_static(toks17, None, tl17, 1.0, 1, 0, out=out)
    assert e.value.status == -3
