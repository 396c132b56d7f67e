"""Moves seeded synthetic tensors (numpy; bf16 as uint16 bit patterns) onto the GPU."""
from __future__ import annotations

import numpy as np
import torch

from .binding import Drafter


def to_device(a: np.ndarray | None, dtype: int | None = None):
    """numpy -> CUDA tensor.  uint16 arrays are reinterpreted as bfloat16 bit patterns."""
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def drafter_from_shape(shape, weights: dict, max_batch: int | None = None, max_ctx: int | None = None,
                       flags: int = 0) -> Drafter:
    """Builds a Drafter for a synth.ModelShape with its numpy weights."""
    w = {k: to_device(v) for k, v in weights.items()}
    return Drafter(dtype=shape.dtype, hidden=shape.hidden, n_heads=shape.n_heads,
                   n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, ffn=shape.ffn,
                   vocab=shape.vocab, k_masks=shape.k_masks, max_batch=max_batch or shape.batch,
                   max_ctx=max_ctx or (shape.ctx_hi + shape.k_masks + 1), weights=w,
                   rope_base=shape.rope_base, rms_eps=shape.rms_eps, flags=flags)
