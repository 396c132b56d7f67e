"""Seeded synthetic inputs shared by the oracle harness and the CUDA harness.

Data only: random tensors with the shapes and value distributions of the paper's
7B/13B-class workloads.  None of the method's arithmetic lives here.
"""
from .gen import (  # noqa: F401
    CONFIGS,
    ModelShape,
    bf16_bits_to_f32,
    ctx_lengths,
    f32_to_bf16_bits,
    gauss_logits,
    hidden_states,
    kv_rows,
    noisy_draft_logits,
    normal,
    sample_from_logits,
    token_ids,
    weights,
    zipf_logits,
)
