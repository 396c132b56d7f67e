"""Seeded synthetic tensors.  Every array is a pure function of (seed, stream, shape).

Random bits come from numpy's counter-based Philox bit generator keyed by
(seed, stream), so any tensor can be regenerated alone, on any machine.
Values are rounded once to the storage type; both consumers read the rounded values.
bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class ModelShape:
    name: str
    dtype: int          # 0 fp32, 1 bf16
    hidden: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    k_masks: int
    batch: int
    ctx_lo: int         # cached context length range (inclusive); lo == hi -> fixed
    ctx_hi: int
    seed: int
    hidden_sigma: float
    logits_kind: str    # "gauss2" or "zipf"
    rope_base: float = 10000.0
    rms_eps: float = 1e-5

    def with_(self, **kw) -> "ModelShape":
        return replace(self, **kw)

    @property
    def rows(self) -> int:
        return self.k_masks + 1

    def weight_bytes(self) -> int:
        """Bytes of the matrices one draft step streams (fc, layer, LM head)."""
        H, F, V = self.hidden, self.ffn, self.vocab
        Hkv = self.n_kv_heads * self.head_dim
        elems = 2 * H * H + 2 * H * H + 2 * Hkv * H + 3 * H * F + V * H
        return elems * (4 if self.dtype == 0 else 2)


CONFIGS = {
    # tiny fp32 drafter, CPU-seconds scale
    "tiny": ModelShape("tiny", 0, 256, 4, 4, 64, 688, 1000, 4, 1, 64, 64, 0, 0.02, "gauss2"),
    # Llama-2-7B-shaped
    "7b": ModelShape("7b", 1, 4096, 32, 32, 128, 11008, 32000, 4, 1, 512, 512, 2000, 1.0, "zipf"),
    # Llama-2-13B-shaped (the headline workload)
    "13b": ModelShape("13b", 1, 5120, 40, 40, 128, 13824, 32000, 4, 1, 1024, 1024, 3000, 1.0, "zipf"),
    # 13B-shaped batch/length sweep: batch and k_masks are overridden per point
    "13b_sweep": ModelShape("13b_sweep", 1, 5120, 40, 40, 128, 13824, 32000, 8, 64, 256, 2048, 4000, 1.0, "zipf"),
    # 33B-class
    "33b": ModelShape("33b", 1, 6656, 52, 52, 128, 17920, 32000, 8, 16, 1024, 4096, 5000, 1.0, "zipf"),
    # Llama-3-8B-shaped: grouped-query attention (8 KV heads) and a 128k vocabulary, where the
    # LM head is two thirds of the bytes (Sec. 2 names the 128,000+ vocabularies of Llama-3)
    "llama3_8b": ModelShape("llama3_8b", 1, 4096, 32, 8, 128, 14336, 128256, 4, 1, 1024, 1024, 6000, 1.0,
                            "zipf", rope_base=500000.0),
    # small bf16 shape for element-by-element parity in seconds (several tiles, ragged tails)
    "mini": ModelShape("mini", 1, 768, 6, 6, 128, 2072, 5000, 4, 3, 37, 203, 7000, 1.0, "zipf"),
    # small fp32 shape with odd sizes
    "mini32": ModelShape("mini32", 0, 320, 5, 5, 64, 872, 1500, 3, 2, 5, 77, 8000, 0.02, "gauss2"),
}


def _rng(seed: int, stream) -> np.random.Generator:
    if isinstance(stream, str):
        stream = zlib.crc32(stream.encode())
    key = np.array([np.uint64(seed), np.uint64(stream)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of finite float32 values to bf16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal(seed: int, stream, shape, sigma: float = 1.0, mean: float = 0.0, dtype: int = 0) -> np.ndarray:
    """N(mean, sigma^2) tensor in storage dtype (float32, or uint16 bf16 bits)."""
    x = _rng(seed, stream).standard_normal(size=shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    if mean != 0.0:
        x += np.float32(mean)
    return x if dtype == 0 else f32_to_bf16_bits(x)


def weights(s: ModelShape, with_bias: bool = False) -> dict:
    """All drafter tensors: matrices N(0, 0.02^2), norm gains 1 + N(0, 0.02^2)."""
    H, F, V, k = s.hidden, s.ffn, s.vocab, s.k_masks
    Hq, Hkv = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    shapes = dict(
        embed=(V, H), mask_embed=(k, H), mask_feat=(k, H), w_fc=(H, 2 * H), w_q=(Hq, H),
        w_k=(Hkv, H), w_v=(Hkv, H), w_o=(H, Hq), w_gate=(F, H), w_up=(F, H), w_down=(H, F),
        w_lm=(V, H),
    )
    out = {n: normal(s.seed, n, shp, 0.02, 0.0, s.dtype) for n, shp in shapes.items()}
    for n in ("g_in", "g_post", "g_final"):
        out[n] = normal(s.seed, n, (H,), 0.02, 1.0, s.dtype)
    out["b_fc"] = normal(s.seed, "b_fc", (H,), 0.02, 0.0, s.dtype) if with_bias else None
    return out


def hidden_states(s: ModelShape, stream, n: int) -> np.ndarray:
    """Stand-in for the target model's last-layer hidden states, [n][H]."""
    return normal(s.seed, ("hidden", stream).__repr__(), (n, s.hidden), s.hidden_sigma, 0.0, s.dtype)


def token_ids(s: ModelShape, stream, n: int) -> np.ndarray:
    return _rng(s.seed, ("tok", stream).__repr__()).integers(0, s.vocab, size=n, dtype=np.int32)


def ctx_lengths(s: ModelShape, batch: int) -> np.ndarray:
    """Ragged cached-context lengths, uniform in [ctx_lo, ctx_hi]."""
    if s.ctx_lo == s.ctx_hi:
        return np.full(batch, s.ctx_lo, np.int32)
    return _rng(s.seed, "ctx").integers(s.ctx_lo, s.ctx_hi + 1, size=batch, dtype=np.int32)


def kv_rows(s: ModelShape, stream, n: int):
    """Random cache contents N(0,1) for import when building the context by appends is too slow."""
    w = s.n_kv_heads * s.head_dim
    K = normal(s.seed, ("K", stream).__repr__(), (n, w), 1.0, 0.0, s.dtype)
    V = normal(s.seed, ("V", stream).__repr__(), (n, w), 1.0, 0.0, s.dtype)
    return K, V


def gauss_logits(seed: int, stream, shape, sigma: float = 2.0) -> np.ndarray:
    return normal(seed, ("gl", stream).__repr__(), shape, sigma)


def zipf_logits(seed: int, stream, batch: int, positions: int, vocab: int, a: float = 1.1) -> np.ndarray:
    """N(0,1) noise plus a rank bias -a*ln(rank), ranks permuted per (sequence, position)."""
    g = _rng(seed, ("zipf", stream).__repr__())
    z = g.standard_normal(size=(batch, positions, vocab), dtype=np.float32)
    bias = (-a * np.log(np.arange(1, vocab + 1, dtype=np.float64))).astype(np.float32)
    for b in range(batch):
        for p in range(positions):
            z[b, p] += bias[g.permutation(vocab)]
    return z


def noisy_draft_logits(seed: int, stream, target_logits: np.ndarray, sigma: float) -> np.ndarray:
    """Draft logits = target logits + N(0, sigma^2): tunes the acceptance length."""
    n = _rng(seed, ("noisy", stream).__repr__()).standard_normal(size=target_logits.shape, dtype=np.float32)
    return (target_logits + np.float32(sigma) * n).astype(np.float32)


def sample_from_logits(seed: int, stream, logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    """Host-side draw of one token per row from softmax(logits/T) (draft tokens x ~ q)."""
    g = _rng(seed, ("draw", stream).__repr__())
    z = logits.astype(np.float64) / temperature
    z -= z.max(axis=-1, keepdims=True)
    p = np.exp(z)
    cdf = np.cumsum(p, axis=-1)
    u = g.random(size=logits.shape[:-1])[..., None] * cdf[..., -1:]
    return np.minimum((cdf <= u).sum(axis=-1), logits.shape[-1] - 1).astype(np.int32)
