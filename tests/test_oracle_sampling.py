"""Pins for the oracle's draft sampler (Algorithm 1: the tree is drafted "by sampling from the
parallel draft model"; CPU only).

The Gumbel-max rule is exact: argmax_v (z_v / T + G_v) with G = -ln(-ln u) follows softmax(z / T).
  * Monte Carlo over the offset counter on a 16-token row, at two temperatures (chi-square);
  * rows with different row ids draw independently (no correlation of the picks);
  * a tiny temperature gives the arg-max; the uniforms never reach 0 or 1 (finite noise).
"""
import numpy as np
from scipy import stats

import oracle


def _softmax(z):
    z = z - z.max(-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(-1, keepdims=True)


def test_gumbel_max_follows_softmax(oracle_mod):
    V, n = 16, 120_000
    z = np.random.default_rng(5).normal(0, 1.5, size=V)
    for T in (1.0, 0.5):
        p = _softmax(z / T)
        picks = np.empty(n, np.int64)
        rows = np.broadcast_to(z, (256, V)).copy()
        ids = np.arange(256, dtype=np.int32)            # 256 independent row ids per offset
        for off in range(n // 256 + 1):
            t, _ = oracle.gumbel_sample(rows, T, seed=11, offset=off, row_id=ids)
            picks[off * 256:(off + 1) * 256] = t[:max(0, min(256, n - off * 256))]
        assert stats.chisquare(np.bincount(picks, minlength=V), p * n).pvalue > 1e-3


def test_rows_draw_independently(oracle_mod):
    V, n = 8, 40_000
    rows = np.zeros((2, V))                              # uniform rows: picks are uniform on 0..7
    a = np.empty(n, np.int64)
    b = np.empty(n, np.int64)
    for off in range(n):
        t, _ = oracle.gumbel_sample(rows, 1.0, seed=3, offset=off, row_id=np.array([0, 1 << 8], np.int32))
        a[off], b[off] = t
    table = np.zeros((V, V))
    np.add.at(table, (a, b), 1)
    assert stats.chi2_contingency(table)[1] > 1e-3
    # another seed, another stream
    t1, _ = oracle.gumbel_sample(np.zeros((64, 50)), 1.0, 3, 0, np.arange(64, dtype=np.int32))
    t2, _ = oracle.gumbel_sample(np.zeros((64, 50)), 1.0, 4, 0, np.arange(64, dtype=np.int32))
    assert (t1 != t2).mean() > 0.8


def test_small_temperature_is_argmax_and_noise_is_finite(oracle_mod):
    rng = np.random.default_rng(2)
    z = rng.normal(0, 1.0, size=(32, 1000))
    t, m = oracle.gumbel_sample(z, 1e-4, seed=1, offset=9, row_id=np.arange(32, dtype=np.int32))
    assert np.array_equal(t, z.argmax(-1)) and (m > 0).all() and np.isfinite(m).all()
    # with -inf logits elsewhere the only finite one wins whatever the noise
    z2 = np.full((4, 100), -np.inf)
    z2[np.arange(4), [3, 50, 99, 0]] = 0.0
    t, _ = oracle.gumbel_sample(z2, 1.0, 1, 0, np.arange(4, dtype=np.int32))
    assert list(t) == [3, 50, 99, 0]
