"""Seeded synthetic inputs shaped like the paper's workloads (numpy, CPU).

The paper evaluates on MATH500 with 1.7B-7B Hugging Face models (Section 6,
Table 1); neither is available offline, so a synthetic first-order language
model stands in: the logits of a row depend on (group, step, previous token)
only, through a counter hash, plus a Zipf-like bias over a hashed vocabulary
permutation.  The KV cache is filled with hashed N(0,1) values so that every
(layer, K/V, row, head, position, dim) element is distinct and a wrong gather
shows.  This module holds only input generation: no log-softmax, no sampling,
no weights.  A CUDA twin of `logits_block` / `kv_block` lives in
`csrc/workload.cu`; the two are cross-checked in the GPU tests.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_M64 = (1 << 64) - 1
STREAM_LOGIT, STREAM_PERM, STREAM_KV, STREAM_PROMPT = 4, 5, 6, 7

_U = np.uint64


def sm64(x):
    """splitmix64 finaliser on uint64 numpy arrays (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = np.asarray(x, dtype=np.uint64) + _U(0x9E3779B97F4A7C15)
        z = (z ^ (z >> _U(30))) * _U(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U(27))) * _U(0x94D049BB133111EB)
        return z ^ (z >> _U(31))


def hash5(a, b, c, d, e):
    """Five-part counter hash; any argument may be an array (broadcast)."""
    u = lambda v: np.asarray(v).astype(np.uint64) if not isinstance(v, int) else _U(v & _M64)
    h = sm64(u(a))
    h = sm64(h ^ u(b))
    h = sm64(h ^ u(c))
    h = sm64(h ^ u(d))
    return sm64(h ^ u(e))


def _box_muller(h):
    """N(0,1) from the two 32-bit halves of a hash, in double precision."""
    u1 = ((h >> _U(32)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    u2 = ((h & _U(0xFFFFFFFF)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def f32_to_bf16_bits(x):
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def vocab_bias(seed: int, V: int, slope: float) -> np.ndarray:
    """bias_v = -slope * ln(1 + rank_v); rank_v = place of v when ids are sorted by a seed hash."""
    keys = hash5(seed, STREAM_PERM, 0, 0, np.arange(V, dtype=np.uint64))
    order = np.argsort(keys, kind="stable")
    rank = np.empty(V, dtype=np.int64)
    rank[order] = np.arange(V)
    return (-slope * np.log1p(rank.astype(np.float64))).astype(np.float64)


def prompt_lengths(seed: int, G: int, lo: int, hi: int) -> np.ndarray:
    """Per-prompt synthetic prompt length, uniform on [lo, hi]."""
    if lo == hi:
        return np.full(G, lo, dtype=np.int32)
    h = hash5(seed, STREAM_PROMPT, np.arange(G, dtype=np.uint64), 0, 1)
    return (lo + (h % _U(hi - lo + 1)).astype(np.int64)).astype(np.int32)


def prompt_last_token(seed: int, G: int, plen: np.ndarray, V: int) -> np.ndarray:
    """Token that precedes the first generated one: hashed from (group, last prompt position)."""
    h = hash5(seed, STREAM_PROMPT, np.arange(G, dtype=np.uint64), (plen - 1).astype(np.uint64), 0)
    return (h % _U(V)).astype(np.int32)


def logits_block(seed: int, t: int, groups, prev_tokens, V: int, scale: float, bias: np.ndarray,
                 dtype: str) -> np.ndarray:
    """Rows of logits for step t: row r = scale * z(seed, group_r, t, prev_r, v) + bias_v.

    Returns float32 [R, V] for dtype 'f32', uint16 bf16 bit patterns for 'bf16'."""
    groups = np.asarray(groups, dtype=np.uint64).reshape(-1, 1)
    prev = np.asarray(prev_tokens).astype(np.uint64).reshape(-1, 1)
    v = np.arange(V, dtype=np.uint64).reshape(1, -1)
    h = hash5(seed, _U(STREAM_LOGIT) ^ (groups << _U(8)), t, prev, v)
    x = (scale * _box_muller(h) + bias.reshape(1, -1)).astype(np.float32)
    if dtype == "f32":
        return x
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)


def kv_block(seed: int, layer: int, which: int, rows, H: int, max_len: int, D: int, dtype: str) -> np.ndarray:
    """One layer's K (which=0) or V (which=1) tensor [len(rows), H, max_len, D] of hashed N(0,1)."""
    rows = np.asarray(rows, dtype=np.uint64).reshape(-1, 1, 1, 1)
    hh = np.arange(H, dtype=np.uint64).reshape(1, -1, 1, 1)
    pos = np.arange(max_len, dtype=np.uint64).reshape(1, 1, -1, 1)
    d = np.arange(D, dtype=np.uint64).reshape(1, 1, 1, -1)
    tag = _U(STREAM_KV) ^ (_U(layer) << _U(8)) ^ (_U(which) << _U(40))
    h = hash5(seed, tag, rows, hh * _U(max_len) + pos, d)
    x = _box_muller(h).astype(np.float32)
    return x if dtype == "f32" else f32_to_bf16_bits(x)


@dataclass(frozen=True)
class Workload:
    """One of the named configurations: shapes and sampler settings."""
    name: str
    G: int
    N: int
    V: int
    dtype: str          # 'f32' | 'bf16' (logits and KV)
    scale: float
    slope: float
    T: int              # decode steps after the prompt
    prompt_lo: int
    prompt_hi: int
    alpha: float
    tau: float
    kappa: float
    ramp: int
    n_layers: int
    n_kv_heads: int
    head_dim: int
    max_len: int
    eos: int = field(default=-1)

    @property
    def R(self):
        return self.G * self.N

    @property
    def eos_id(self):
        return self.V - 1 if self.eos < 0 else self.eos

    @property
    def elem(self):
        return 4 if self.dtype == "f32" else 2

    @property
    def logit_bytes_per_row(self):
        return self.V * self.elem

    @property
    def kv_bytes_per_pos_per_row(self):
        return 2 * self.n_layers * self.n_kv_heads * self.head_dim * self.elem


CONFIGS = {
    "tiny": Workload("tiny", 1, 4, 1024, "f32", 2.0, 1.5, 64, 64, 64, 4.0, 0.25, 0.5, 0, 2, 2, 64, 128),
    "llama2_7b": Workload("llama2_7b", 1, 8, 32000, "bf16", 3.0, 1.5, 512, 512, 512, 4.0, 0.25, 0.5, 0,
                          32, 32, 128, 1024),
    "qwen25_7b": Workload("qwen25_7b", 1, 16, 151936, "bf16", 3.0, 1.5, 2048, 256, 256, 4.0, 0.25, 0.5, 128,
                          28, 4, 128, 2304),
    "resample_stress": Workload("resample_stress", 1, 32, 151936, "bf16", 6.0, 1.5, 4096, 128, 128, 8.0,
                                0.125, 0.9, 256, 28, 4, 128, 4224),
    "batched_prompts": Workload("batched_prompts", 64, 8, 128256, "bf16", 3.0, 1.5, 1024, 64, 256, 4.0, 0.25,
                                0.5, 0, 32, 8, 128, 1280),
}
