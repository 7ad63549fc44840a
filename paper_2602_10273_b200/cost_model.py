"""Token-evaluation cost model of Section 5: Power-SMC against Metropolis-Hastings power sampling.

Host arithmetic only (no GPU, no state).  The unit is one token-eval: one forward pass of the language model for
one new token with the KV cache in place.  Symbols follow Section 5: T generated tokens, block length B (B divides
T, K = T / B blocks), M MH moves per block, N particles, s(b) the throughput multiplier of a batch of b sequences
relative to a batch of one (a batch-b step takes time proportional to b / s(b)).

Each expectation comes in two forms: the closed form the section prints (which replaces (n + 1) / 2 by n / 2), and
`exact=True`, the same expectation without that step.
"""
from __future__ import annotations

from typing import Iterable, Sequence


def _blocks(T: int, B: int) -> int:
    if T <= 0 or B <= 0 or T % B:
        raise ValueError("the block length must divide the number of generated tokens (T=%d, B=%d)" % (T, B))
    return T // B


def smc_token_evals(N: int, T: int) -> int:
    """Lemma 1: every one of T decode steps advances all N particles."""
    if N <= 0 or T < 0:
        raise ValueError("N must be positive and T non-negative")
    return N * T


def smc_time(N: int, T: int, s_N: float) -> float:
    """Lemma 1: wall-clock time in units of one batch-1 step, T steps of N / s(N) each."""
    if s_N < 1.0:
        raise ValueError("s(N) is at least 1 by definition")
    return T * N / s_N


def mh_token_evals(B: int, suffix_lengths: Sequence[Iterable[int]]) -> int:
    """Eq. 10: every block costs B token-evals to extend plus the regenerated suffix of each of its moves.

    suffix_lengths[k] holds the lengths L_{k,m} of the moves made in block k.
    """
    return sum(B + sum(moves) for moves in suffix_lengths)


def mh_global_edit_evals(T: int, B: int, M: int, exact: bool = False) -> float:
    """Lemma 2: moves of block k edit uniformly over the whole prefix of length kB.

    Closed form T (1 + M (K + 1) / 4); exactly, E[L_k] = (kB + 1) / 2.
    """
    K = _blocks(T, B)
    if exact:
        return T + M * sum((k * B + 1) / 2.0 for k in range(1, K + 1))
    return T * (1.0 + M * (K + 1) / 4.0)


def mh_last_block_evals(T: int, B: int, M: int, exact: bool = False) -> float:
    """Lemma 3: moves edit uniformly inside the newest block only.

    Closed form T (1 + M / 2); exactly, E[L_k] = (B + 1) / 2.
    """
    K = _blocks(T, B)
    if exact:
        return T + M * K * (B + 1) / 2.0
    return T * (1.0 + M / 2.0)


def global_edit_factor(M: int, K: int) -> float:
    """1 + M (K + 1) / 4: expected MH token-evals per generated token under global edits (Lemma 2)."""
    return 1.0 + M * (K + 1) / 4.0


def compute_ratio(N: int, M: int, K: int) -> float:
    """Corollary 2: E[C_MH] / C_SMC for global-edit MH."""
    return global_edit_factor(M, K) / N


def time_ratio(N: int, M: int, K: int, s_N: float) -> float:
    """Corollary 3: Time_MH / Time_SMC with MH at batch 1 and Power-SMC at batch N."""
    if s_N < 1.0:
        raise ValueError("s(N) is at least 1 by definition")
    return global_edit_factor(M, K) * s_N / N


def mh_overhead_floor(M: int) -> float:
    """Corollary 4: MH overhead over plain decoding under last-block edits, 1 + M / 2."""
    return 1.0 + M / 2.0


def break_even_multiplier(N: int, M: int, K: int) -> float:
    """The s(N) above which Power-SMC is faster than global-edit MH in wall-clock time (Corollary 3 set to 1)."""
    return N / global_edit_factor(M, K)
