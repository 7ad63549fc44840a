"""Section 5's cost model: the values the paper prints, and the expectations behind its closed forms by enumeration."""
import itertools
import os
from fractions import Fraction

import pytest

from paper_2602_10273_b200 import cost_model as C

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "cost_model_example.txt")


def _rows():
    with open(GOLDEN) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_worked_example_of_section_5():
    for N, M, K, factor, ratio2, floor in _rows():
        N, M, K = int(N), int(M), int(K)
        assert C.global_edit_factor(M, K) == float(factor)
        assert round(C.compute_ratio(N, M, K), 2) == float(ratio2)
        assert C.mh_overhead_floor(M) == float(floor)
        # Corollary 3 is Corollary 2 times s(N); at s(N) = 1 they coincide, and the break-even multiplier undoes it
        assert C.time_ratio(N, M, K, 1.0) == C.compute_ratio(N, M, K)
        assert C.time_ratio(N, M, K, C.break_even_multiplier(N, M, K)) == pytest.approx(1.0, rel=1e-15)


def test_smc_cost_is_one_batch_of_N_per_token():
    assert C.smc_token_evals(48, 1024) == 48 * 1024
    assert C.smc_time(48, 1024, 1.0) == 48 * 1024          # no batching gain: as slow as the token count
    assert C.smc_time(48, 1024, 48.0) == 1024               # perfect batching: as fast as plain decoding
    with pytest.raises(ValueError):
        C.smc_time(48, 1024, 0.5)


@pytest.mark.parametrize("B,K,M", [(1, 1, 1), (2, 3, 2), (3, 2, 1), (4, 2, 2)])
def test_expectations_by_enumerating_every_edit_point(B, K, M):
    """Average of Eq. 10 over every choice of edit points, in exact rational arithmetic."""
    T = B * K
    # global edit: in block k the edit index is uniform on {0..kB-1} and the suffix from it to kB is regenerated
    glob = [[k * B - e for e in range(k * B)] for k in range(1, K + 1)]
    # last-block edit: the offset to the block's end is uniform on {1..B}
    last = [list(range(1, B + 1)) for _ in range(K)]
    for choices, fn in ((glob, C.mh_global_edit_evals), (last, C.mh_last_block_evals)):
        per_move = [c for c in choices for _ in range(M)]          # K*M independent uniform draws
        total, count = Fraction(0), 0
        for draw in itertools.product(*per_move):
            blocks = [draw[k * M:(k + 1) * M] for k in range(K)]
            total += C.mh_token_evals(B, blocks)
            count += 1
        assert Fraction(fn(T, B, M, exact=True)).limit_denominator(10**6) == total / count


def test_closed_forms_are_the_exact_ones_with_n_plus_1_taken_as_n():
    T, B, M = 1024, 64, 10
    K = T // B
    # exact - approx = M * K / 2 in both regimes: the "+1" of every (n + 1) / 2, once per move
    assert C.mh_global_edit_evals(T, B, M, exact=True) - C.mh_global_edit_evals(T, B, M) == M * K / 2
    assert C.mh_last_block_evals(T, B, M, exact=True) - C.mh_last_block_evals(T, B, M) == M * K / 2
    assert C.mh_global_edit_evals(T, B, M) == T * C.global_edit_factor(M, K)
    assert C.mh_last_block_evals(T, B, M) == T * C.mh_overhead_floor(M)
    # Theta(T^2 / B): doubling T at fixed B roughly quadruples the move cost
    a = C.mh_global_edit_evals(T, B, M) - T
    b = C.mh_global_edit_evals(2 * T, B, M) - 2 * T
    assert 3.5 < b / a < 4.0


def test_block_length_must_divide_the_horizon():
    with pytest.raises(ValueError):
        C.mh_global_edit_evals(100, 64, 10)
