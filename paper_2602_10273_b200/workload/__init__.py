"""Seeded synthetic workloads (logits of a first-order stand-in LM, KV-cache fill).

Serves the CUDA path, the CPU oracle's tests and the benchmark alike; holds
none of the sampler's arithmetic.
"""
from .gen import (CONFIGS, Workload, bf16_bits_to_f32, f32_to_bf16_bits, hash5, kv_block, logits_block,
                  prompt_last_token, prompt_lengths, sm64, vocab_bias)

__all__ = ["CONFIGS", "Workload", "bf16_bits_to_f32", "f32_to_bf16_bits", "hash5", "kv_block",
           "logits_block", "prompt_last_token", "prompt_lengths", "sm64", "vocab_bias"]
