"""The named configurations at their stated length (Algorithm 1 runs to T_max), CUDA path against the oracle at every
token: the tolerance on log W and on S = log p(y_{1:t}) (1e-4 absolute) has to hold over the whole horizon, not just
over the first tokens, and the final draw walks an ancestry log of the full length (several batches of the
back-trace).  Caches keep the stated heads, head size and maximum length but one layer, to bound the host mirror.

With PSMC_TEST_REPORT=<file> every run appends one JSON line with its counts (steps, resampling events, slots
rewritten, choices the oracle adopted) and largest differences.
"""
import dataclasses
import json
import os

import numpy as np
import pytest
import torch

import parity as P
from paper_2602_10273_b200.workload import gen as W

pytestmark = pytest.mark.gpu


def _report(label, st):
    path = os.environ.get("PSMC_TEST_REPORT")
    print(label, st)
    if path:
        with open(path, "a") as f:
            f.write(json.dumps({"run": label, **dataclasses.asdict(st)}) + "\n")


@pytest.mark.parametrize("name", ["llama2_7b", "qwen25_7b", "resample_stress"])
def test_closed_loop_at_the_stated_length(name):
    c = W.CONFIGS[name]
    st = P.closed_loop(c, seed=1, T=c.T, kv_shape=(1, c.n_kv_heads, c.max_len, c.head_dim))
    assert st.steps == c.T and st.resample_events > 0 and st.slots_moved > 0
    _report("%s, T = %d" % (name, c.T), st)


def test_batched_prompts_eight_prompts_at_the_stated_length():
    c = W.CONFIGS["batched_prompts"]
    st = P.closed_loop(c, seed=1, T=c.T, G=8, kv_shape=(1, c.n_kv_heads, c.max_len, c.head_dim))
    assert st.steps == c.T and st.resample_events > 0
    _report("batched_prompts, 8 of 64 prompts, T = %d" % c.T, st)


def test_batched_prompts_full_width_sixty_four_tokens():
    c = W.CONFIGS["batched_prompts"]
    st = P.closed_loop(c, seed=2, T=64, kv_shape=(1, c.n_kv_heads, c.max_len, c.head_dim))
    assert st.live_rows == 64 * 512 and st.resample_events > 0
    _report("batched_prompts, 64 prompts, T = 64", st)


@pytest.mark.parametrize("rule", [dict(top_k=50), dict(top_p=0.9)])
def test_restricted_proposals_over_three_thousand_tokens(rule):
    """The fast exponential returns its values low by 5e-8 of the value on average, every sum of such terms is low by
    that fraction, and log p(y_{1:t}) adds the same error at every token: 1.5e-4 after 3000 tokens unless the kernels
    take it out.  The restricted proposals form their sums in a kernel of their own."""
    c = W.Workload("restricted_long", 1, 8, 4096, "bf16", 3.0, 1.5, 3000, 4, 4, 4.0, 0.25, 0.5, 0, 1, 1, 8, 3008)

    def no_eos(t, lg):          # keep the particles alive to the end
        lg[:, c.eos_id] = -40.0

    st = P.closed_loop(c, seed=3, T=c.T, logit_bias_fn=no_eos, **rule)
    assert st.steps == c.T and st.live_rows == c.T * c.N and st.resample_events > 0
    _report("restricted_long %r, T = %d" % (rule, c.T), st)


def _long_small(name, N=8, dtype="bf16", alpha=4.0, tau=0.25, T=3000):
    return W.Workload(name, 1, N, 4096, dtype, 3.0, 1.5, T, 4, 4, alpha, tau, 0.5, 0, 1, 1, 8, T + 8)


def _no_eos(c):
    def edit(t, lg):            # keep the particles alive to the end
        lg[:, c.eos_id] = -40.0
    return edit


@pytest.mark.parametrize("label,kw", [("fp32 logits", dict(dtype="f32")),
                                      ("beta = 3 (no squaring)", dict(alpha=3.0, tau=1.0 / 3.0)),
                                      ("beta = 2", dict(alpha=2.0, tau=0.5)),
                                      ("33 particles (the step as two kernels)", dict(N=33, T=2000))])
def test_other_forms_of_the_step_over_thousands_of_tokens(label, kw):
    """The same horizon for the forms of the logit pass the named configurations do not reach: fp32 logits, an
    exponent that is not a power of two, groups too large for the one-kernel step."""
    c = _long_small("long_small", **kw)
    st = P.closed_loop(c, seed=5, T=c.T, logit_bias_fn=_no_eos(c))
    assert st.steps == c.T and st.live_rows == c.T * c.N and st.resample_events > 0
    _report("long_small, %s, T = %d" % (label, c.T), st)


def test_vocabulary_sharded_step_over_three_thousand_tokens():
    from test_gpu_vocab_shard import sharded_loop
    c = _long_small("long_sharded")
    st, owners = sharded_loop(c, 6, c.T, [(0, 1500), (1500, 2596)], logit_edit=_no_eos(c))
    assert st.steps == c.T and (owners > 0).all()
    _report("long_sharded, 2 ranks, T = %d" % c.T, st)


def test_tile_fed_step_over_three_thousand_tokens():
    from test_gpu_tile_fed import tile_fed_loop
    c = _long_small("long_tiles")
    st = tile_fed_loop(c, 7, c.T, 1024, logit_edit=_no_eos(c))
    assert st.steps == c.T
    _report("long_tiles, width 1024, T = %d" % c.T, st)


@pytest.mark.parametrize("N,V,T,kappa", [(33, 64, 300, 0.9), (1024, 32, 9, 1.0), (8, 50, 1200, 0.7)])
def test_back_trace_over_several_batches(N, V, T, kappa):
    """The output step stages its ancestry log in batches of 4096 integers; T * N beyond that takes several batches.
    Frequent resampling and early EOS make the walk non-trivial (V is small, so EOS is drawn often)."""
    c = W.Workload("trace", 1, N, V, "f32", 2.0, 1.5, T, 3, 3, 2.0, 0.5, kappa, 0, 1, 1, 8, T + 8)
    st = P.closed_loop(c, seed=7, T=T)
    assert st.steps == T and T * N > 4096 and st.resample_events > 0
