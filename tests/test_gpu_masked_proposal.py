"""Steps whose proposal is restricted to the top-k tokens of each row, or to a nucleus of the tempered distribution,
against the oracle's masked row (closed loops through the C-ABI, as for the unrestricted step).

The size of the support is an integer decided by counting (top-k: must match exactly) or by comparing masses
(nucleus: the oracle adopts the CUDA size when it misses the rule by no more than parity.K_MARGIN of the mass).
"""
import numpy as np
import pytest
import torch

import parity as P
from oracle import oracle as O
from paper_2602_10273_b200 import binding as B
from paper_2602_10273_b200.workload import gen as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("top_k", [1, 2, 7, 64, 1023, 1024, 5000])
def test_top_k_small_vocabulary_fp32(top_k):
    cfg = W.CONFIGS["tiny"]
    st = P.closed_loop(cfg, 3, 48, top_k=top_k)
    assert st.steps == 48 and st.k_adopted == 0
    if top_k >= 64:
        assert st.resample_events > 0


@pytest.mark.parametrize("top_p", [0.05, 0.5, 0.9, 0.999, 1.0])
def test_nucleus_small_vocabulary_fp32(top_p):
    cfg = W.CONFIGS["tiny"]
    st = P.closed_loop(cfg, 4, 48, top_p=top_p)
    assert st.steps == 48


@pytest.mark.parametrize("name,G,T,rule", [("llama2_7b", None, 24, dict(top_k=50)), ("llama2_7b", 3, 16, dict(top_p=0.9)),
                                           ("qwen25_7b", None, 12, dict(top_k=40)), ("qwen25_7b", None, 12, dict(top_p=0.95)),
                                           ("resample_stress", None, 10, dict(top_k=1000)),
                                           ("batched_prompts", 6, 6, dict(top_p=0.8)), ("batched_prompts", 6, 6, dict(top_k=20))])
def test_masked_steps_model_vocabularies_bf16(name, G, T, rule):
    st = P.closed_loop(W.CONFIGS[name], 7, T, G=G, **rule)
    assert st.steps == T


@pytest.mark.parametrize("rule", [dict(top_k=50), dict(top_k=1000), dict(top_p=0.9)])
def test_masked_steps_batched_prompts_full_size(rule):
    """All 64 prompts x 8 particles x 128256 logits: the launch shape `bench.py --top-k / --top-p` times (one CTA per
    row, two per SM), every row compared with the oracle."""
    st = P.closed_loop(W.CONFIGS["batched_prompts"], 1, 3, **rule)
    assert st.live_rows == 3 * 512


@pytest.mark.parametrize("name,rule,flat", [("llama2_7b", dict(top_k=20000), False), ("llama2_7b", dict(top_p=0.97), True),
                                            ("qwen25_7b", dict(top_k=100000), False), ("qwen25_7b", dict(top_k=9000), True),
                                            ("qwen25_7b", dict(top_k=100), True), ("tiny", dict(top_p=0.9), True)])
def test_supports_too_large_for_the_candidate_list(name, rule, flat):
    """More candidates at the cut than the kernel's shared-memory list holds (4096): it sweeps the row for every
    remaining step instead (a large top_k; a flat row, which makes every nucleus large and puts crowds of equal
    logits at a small top_k's threshold)."""
    def flatten(t, lg):
        lg.copy_((lg.float() * 0.02).to(lg.dtype))

    st = P.closed_loop(W.CONFIGS[name], 6, 8, logit_bias_fn=flatten if flat else None, **rule)
    assert st.steps == 8


@pytest.mark.parametrize("rule", [dict(top_k=37), dict(top_k=300), dict(top_p=0.6)])
@pytest.mark.parametrize("name", ["tiny", "llama2_7b"])
def test_ties_at_the_cut_are_taken_in_id_order(name, rule):
    """Logits rounded to whole numbers: a handful of distinct values, so the k-th rank falls inside a large group of
    equal logits and only its first members (by token id) belong to the set."""
    def coarse(t, lg):
        lg.copy_(torch.round(lg.float()).to(lg.dtype))

    st = P.closed_loop(W.CONFIGS[name], 9, 12, logit_bias_fn=coarse, **rule)
    assert st.steps == 12


@pytest.mark.parametrize("top_k", [1, 5, 50, 100, 120, 127, 128, 129, 200])
@pytest.mark.parametrize("name", ["llama2_7b", "tiny"])
def test_ties_straddle_the_cut_of_a_short_candidate_list(name, top_k):
    """A few logits equal to the k-th largest, scattered over the row: the candidate list stays short (up to 128
    entries are ranked by one warp, longer lists by the whole CTA: sizes on both sides of that limit), and which of the
    equal logits belong to the set is decided by token id."""
    cfg = W.CONFIGS[name]
    gen = torch.Generator(device="cuda").manual_seed(top_k)

    def plant(t, lg):
        kth = torch.topk(lg.float(), top_k, dim=1).values[:, -1:]                  # [R, 1]
        cols = torch.randint(0, cfg.V - 1, (lg.shape[0], 6), device="cuda", generator=gen)
        lg.scatter_(1, cols, kth.expand(-1, 6).to(lg.dtype))

    st = P.closed_loop(cfg, 13, 10, logit_bias_fn=plant, top_k=top_k)
    assert st.steps == 10 and st.k_adopted == 0


def test_signed_zeros_and_masked_columns():
    cfg = W.CONFIGS["tiny"]

    def edit(t, lg):
        lg.zero_()
        lg[:, 1::2] = -0.0                     # -0 and +0 are one value: ties in id order, not by sign
        lg[:, 600:] = float("-inf")            # fewer finite logits than k at some steps
        if t % 2:
            lg[:, 17] = 1.5

    for rule in (dict(top_k=5), dict(top_k=700), dict(top_p=0.5)):
        st = P.closed_loop(cfg, 5, 6, logit_bias_fn=edit, **rule)
        assert st.steps == 6


@pytest.mark.parametrize("rule", [dict(top_k=5), dict(top_k=3000), dict(top_p=0.9), dict(top_p=1.0)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_rows_with_nan_or_inf_are_flagged(rule, dtype):
    """A NaN of either sign or a +inf anywhere in a row (inside the 16-byte vectors or at the ragged ends; the bf16
    sweeps take maxima two logits at a time) makes the row unusable: token -1, PSMC_E_NUMERIC, the other rows as usual.
    A row of -inf only has nothing to draw from either."""
    V, N = 4099, 8
    as_int = torch.int16 if dtype == torch.bfloat16 else torch.int32
    bads = [(1, 0, float("nan")), (2, 1001, "-nan"), (3, 2222, float("inf")), (4, V - 1, float("nan")),
            (5, V - 2, "-nan"), (6, 7, float("inf"))]
    for row, col, val in bads:
        ps = B.Psmc(N, V, 4.0, 0.25, 0.5, 0, 11, V - 1, T_max=2)
        ps.set_proposal_mask(**rule)
        lg = (torch.randn(N, V + 3, device="cuda") * 2.0).to(dtype)[:, 1:V + 1]   # rows start off a 16-byte boundary
        if val == "-nan":
            lg.view(as_int)[row, col] = -1                                         # all bits set: a NaN with the sign bit
            assert bool(torch.isnan(lg[row, col]))
        else:
            lg[row, col] = val
        ps.step(lg)
        assert ps.sync_status() == B.E_NUMERIC
        tok = ps.tokens.numpy()
        assert tok[row] == -1 or tok[row] == V - 1    # (the group update maps a flagged row's token to a valid id)
        ps.destroy()
    ps = B.Psmc(N, V, 4.0, 0.25, 0.5, 0, 11, V - 1, T_max=2)
    ps.set_proposal_mask(**rule)
    lg = (torch.randn(N, V, device="cuda") * 2.0).to(dtype)
    lg[3] = float("-inf")
    ps.step(lg)
    assert ps.sync_status() == B.E_NUMERIC
    ps.destroy()


def test_support_sizes_and_the_tokens_outside_it():
    """Every drawn token is among the row's top_k; the reported size is min(top_k, V)."""
    cfg = W.CONFIGS["llama2_7b"]
    wl, ps, orc = P.make_pair(cfg, 2, T_max=4, top_k=10)
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    for t in range(1, 5):
        wl.fill(lg, t, prev)
        ps.step(lg)
        toks = ps.tokens.numpy()
        assert (ps.mask_sizes.numpy() == 10).all()
        top = torch.topk(lg.float(), 10, dim=1).values[:, -1].cpu().numpy()       # the 10th largest logit of each row
        drawn = lg.float().cpu().numpy()[np.arange(ps.R), toks]
        assert (drawn >= top).all()
        prev.copy_(ps.device_view("psmc_last_tokens", ps.R))
    assert ps.sync_status() == B.OK
    ps.destroy()


def test_mask_argument_checks_and_snapshot():
    cfg = W.CONFIGS["tiny"]
    wl, ps, orc = P.make_pair(cfg, 1, T_max=8)
    for bad in ((3, 0.5), (-1, 0.0), (0, 1.5), (0, -0.1)):
        with pytest.raises(B.PsmcError) as e:
            ps.set_proposal_mask(*bad)
        assert e.value.code == B.E_INVAL
    ps.set_proposal_mask(top_p=0.7)
    tr = torch.empty((ps.R, 3), dtype=torch.float64, device="cuda")
    lg = wl.new_logits()
    wl.fill(lg, 1, wl.first_prev.clone())
    with pytest.raises(B.PsmcError) as e:
        ps.shard_sweep(lg, tr)                 # ranking a row needs all of its columns
    assert e.value.code == B.E_STATE
    ps.step(lg)
    k1 = ps.mask_sizes.numpy().copy()
    assert (k1 >= 1).all() and (k1 < cfg.V).all()
    # the rule travels with a snapshot
    blob = ps.state_save()
    other = B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, cfg.ramp, 99, cfg.eos_id, G=ps.G, T_max=8,
                   prompt_len=wl.prompt_len)
    other.state_load(blob)
    wl.fill(lg, 2, ps.device_view("psmc_last_tokens", ps.R).clone())
    ps.step(lg)
    other.step(lg)
    assert np.array_equal(ps.tokens.numpy(), other.tokens.numpy())
    assert np.array_equal(ps.mask_sizes.numpy(), other.mask_sizes.numpy())
    ps.set_proposal_mask(0, 0.0)               # off again: the plain step
    other.set_proposal_mask(0, 0.0)
    assert ps.sync_status() == B.OK and other.sync_status() == B.OK
    ps.destroy()
    other.destroy()


def test_masked_steps_random_settings():
    """Sixteen seeded draws of (groups, particles, vocabulary, dtype, alpha, tau, ramp) with a random rule each."""
    rng = np.random.default_rng(20260213)
    for case in range(16):
        N = int(rng.choice([1, 3, 8, 17, 33]))
        G = int(rng.integers(1, 4))
        V = int(rng.choice([16, 100, 1024, 3001, 20000, 70001]))
        alpha = float(rng.choice([1.0, 2.0, 4.0, 1.0 + 4.0 * rng.random()]))
        tau = 1.0 / alpha if rng.random() < 0.6 else float(0.2 + rng.random())
        c = W.Workload("masked%d" % case, G, N, V, "bf16" if rng.random() < 0.5 else "f32", float(rng.choice([1.0, 3.0, 6.0])),
                       1.5, 12, 3, 9, alpha, tau, float(rng.choice([0.3, 0.5, 0.9])), int(rng.choice([0, 0, 4])),
                       1, 2, 16, 32)
        if rng.random() < 0.5:
            rule = dict(top_k=int(rng.choice([1, 5, 40, 300, 2500, 10**6])))
        else:
            rule = dict(top_p=float(rng.choice([0.1, 0.5, 0.9, 0.99, 0.99995, 1.0])))
        st = P.closed_loop(c, seed=200 + case, T=8, **rule)
        assert st.steps == 8, (case, rule)
