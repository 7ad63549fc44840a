"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong
sign, transposed exponent, off-by-one index) fails it.
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy import special, stats

from oracle import oracle as O


# ---------------------------------------------------------------- randomness
def test_splitmix64_published_vectors(golden_dir):
    want = [int(l, 16) for l in open(os.path.join(golden_dir, "splitmix64_seed0.txt")) if not l.startswith("#")]
    golden = 0x9E3779B97F4A7C15
    got = [O.sm64((k * golden) % 2**64) for k in range(len(want))]
    assert got == want


def test_hash5_is_the_chained_finaliser_and_uniform_is_open_interval():
    a, b, c, d, e = 7, 1, 3, 99, 5
    h = O.sm64(O.sm64(O.sm64(O.sm64(O.sm64(a) ^ b) ^ c) ^ d) ^ e)
    assert O.hash5(a, b, c, d, e) == h
    assert O.uniform(0) == 2.0**-53 > 0.0
    assert O.uniform(2**64 - 1) == 1.0 - 2.0**-53 < 1.0
    assert O.uniform(1 << 63) == 0.5 + 2.0**-53
    assert O.uniform((1 << 12) - 1) == O.uniform(0)       # the low 12 bits are not used
    # order of the counter parts matters
    assert O.hash5(1, 2, 3, 4, 5) != O.hash5(1, 2, 3, 5, 4)
    u = np.array([O.uniform(O.hash5(11, 1, 0, t, i)) for t in range(200) for i in range(50)])
    assert stats.kstest(u, "uniform").pvalue > 1e-3


# ---------------------------------------------------------------- Eq. 7 / Theorem 1 on one row
def test_two_level_row_hand_worked(golden_dir):
    l = np.array([math.log(4.0), 0.0, 0.0, 0.0])
    for line in open(os.path.join(golden_dir, "two_level_row.txt")):
        if line.startswith("#") or not line.strip():
            continue
        U, tok, lw, lp, lq = line.split()
        r = O.row(l, 2.0, 2.0, float(U))
        assert r["y"] == int(tok)
        assert r["log_omega"] == pytest.approx(float(lw), abs=1e-13)
        assert r["logp_y"] == pytest.approx(float(lp), abs=1e-13)
        assert r["logq_y"] == pytest.approx(float(lq), abs=1e-13)


@pytest.mark.parametrize("alpha", [1.0, 2.0, 4.0, 8.0, 2.5])
def test_constant_and_one_hot_rows(alpha):
    V = 37
    r = O.row(np.full(V, 3.25), alpha, alpha, 0.41)
    assert r["log_omega"] == pytest.approx((1.0 - alpha) * math.log(V), abs=1e-12)
    assert r["y"] == int(math.ceil(0.41 * V)) - 1  # uniform q: first v with (v+1)/V >= U
    l = np.full(V, -np.inf)
    l[11] = 2.0
    r = O.row(l, alpha, alpha, 0.9)
    assert r["y"] == 11 and r["log_omega"] == pytest.approx(0.0, abs=1e-14)


@pytest.mark.parametrize("alpha", [2.0, 4.0, 8.0, 1.75])
def test_renyi_identity_sign_and_token_independence(alpha):
    rng = np.random.default_rng(3)
    l = rng.normal(0, 3, size=50)
    p = special.softmax(l)
    renyi = math.log(np.sum(p**alpha)) / (1.0 - alpha)
    vals = [O.row(l, alpha, alpha, 0.5, force=v)["log_omega"] for v in range(l.size)]
    assert max(vals) - min(vals) < 1e-12          # Theorem 1: the same for every token
    assert vals[0] == pytest.approx((1.0 - alpha) * renyi, abs=1e-12)
    assert vals[0] <= 0.0
    r = O.row(l, alpha, alpha, 0.5)
    assert r["L1"] == pytest.approx(special.logsumexp(l), abs=1e-12)
    assert r["Lbeta"] == pytest.approx(special.logsumexp(alpha * l), abs=1e-12)
    assert r["logp_y"] == pytest.approx(math.log(p[r["y"]]), abs=1e-12)


@pytest.mark.parametrize("alpha,beta", [(4.0, 1.0), (4.0, 2.5), (2.0, 3.0), (3.0, 0.5)])
def test_mean_of_incremental_weight_is_invariant_to_the_proposal(alpha, beta):
    """Step 1 of the proof of Theorem 1: sum_v q(v) omega(v) = sum_v p(v)^alpha for any q."""
    rng = np.random.default_rng(5)
    l = rng.normal(0, 2, size=23)
    p = special.softmax(l)
    q = special.softmax(beta * l)
    acc = 0.0
    for v in range(l.size):
        r = O.row(l, beta, alpha, 0.5, force=v)
        assert r["logq_y"] == pytest.approx(math.log(q[v]), abs=1e-12)
        acc += q[v] * math.exp(r["log_omega"])
    assert acc == pytest.approx(float(np.sum(p**alpha)), rel=1e-12)
    # and the weights do depend on the token when beta != alpha
    a = O.row(l, beta, alpha, 0.5, force=0)["log_omega"]
    b = O.row(l, beta, alpha, 0.5, force=1)["log_omega"]
    assert abs(a - b) > 1e-6


def test_inverse_cdf_first_index_rule_and_limits():
    l = np.array([-np.inf, 0.0, -np.inf, math.log(3.0), -np.inf])  # masses 0, 1/4, 0, 3/4, 0 at beta=1
    assert O.row(l, 1.0, 1.0, 1e-300)["y"] == 1       # U -> 0: first token with mass
    assert O.row(l, 1.0, 1.0, 0.25)["y"] == 1         # boundary hit exactly: inclusive prefix >= U
    assert O.row(l, 1.0, 1.0, 0.2500001)["y"] == 3
    assert O.row(l, 1.0, 1.0, 1.0 - 2.0**-54)["y"] == 3  # U -> 1: last token with mass
    r = O.row(l, 1.0, 1.0, 0.2500001)
    assert r["margin"] == pytest.approx(1e-7, rel=1e-3)
    # beta reshapes the masses: at beta=2 they are 1/10 and 9/10
    assert O.row(l, 2.0, 2.0, 0.11)["y"] == 3 and O.row(l, 2.0, 2.0, 0.09)["y"] == 1


def test_sampling_frequencies_follow_softmax_beta():
    rng = np.random.default_rng(9)
    l = rng.normal(0, 1.5, size=6)
    beta = 3.0
    q = special.softmax(beta * l)
    n = 20000
    counts = np.zeros(6)
    for k in range(n):
        U = O.uniform(O.hash5(123, O.STREAM_TOKEN, 0, k, 0))
        counts[O.row(l, beta, beta, U)["y"]] += 1
    assert stats.chisquare(counts, q * n).pvalue > 1e-3


def test_bad_rows_are_refused():
    for bad in ([0.0, float("nan"), 1.0], [float("inf"), 0.0], [-float("inf")] * 3):
        with pytest.raises(FloatingPointError):
            O.row(np.array(bad), 2.0, 2.0, 0.5)


# ---------------------------------------------------------------- Eq. 5
def test_ess_textbook_values():
    assert O.ess(np.full(9, -3.7))["ess"] == pytest.approx(9.0, abs=1e-12)
    lw = np.full(7, -np.inf)
    lw[2] = 5.0
    assert O.ess(lw)["ess"] == pytest.approx(1.0, abs=1e-12)
    w = np.array([0.5, 0.25, 0.125, 0.125])
    assert O.ess(np.log(w) + 100.0)["ess"] == pytest.approx(1.0 / np.sum(w**2), rel=1e-12)  # shift-invariant


# ---------------------------------------------------------------- systematic resampling and the slot map
@pytest.mark.parametrize("N", [1, 2, 5, 32, 257])
def test_systematic_resampling_properties(N):
    rng = np.random.default_rng(N)
    for trial in range(40):
        w = rng.exponential(size=N) ** 3
        u0 = O.uniform(O.hash5(1, O.STREAM_RESAMPLE, 0, trial, 0))
        A, _ = O.systematic(w, u0)
        assert A.size == N and np.all(np.diff(A) >= 0) and A.min() >= 0 and A.max() < N
        off = np.bincount(A, minlength=N)
        nw = N * w / w.sum()
        assert np.all(off >= np.floor(nw - 1e-9)) and np.all(off <= np.ceil(nw + 1e-9))
        assert off.sum() == N
        # the textbook formulation through a library routine: first j with C_j >= p_i
        ref = np.searchsorted(np.cumsum(w) / w.sum(), (u0 + np.arange(N)) / N, side="left")
        assert np.array_equal(A, np.minimum(ref, N - 1))
        A_id, _ = O.systematic(np.ones(N) * 0.3, u0)
        assert np.array_equal(A_id, np.arange(N))    # uniform weights: identity for any offset


def test_systematic_resampling_hand_example():
    # weights 0.1 0.2 0.3 0.4 -> prefix 0.1 0.3 0.6 1.0 ; positions (0.5+i)/4 = .125 .375 .625 .875
    A, mg = O.systematic(np.array([0.1, 0.2, 0.3, 0.4]), 0.5)
    assert A.tolist() == [1, 2, 3, 3]
    assert mg == pytest.approx(0.025, abs=1e-12)  # |0.625 - 0.6| and |0.125 - 0.1| are the closest calls


# ---------------------------------------------------------------- the other schemes of Appendix E
def test_other_resamplers_hand_example():
    # weights .1 .5 .05 .35 -> prefix .1 .6 .65 1 ; uniforms .3 .9 .2 .6
    w, u = np.array([0.1, 0.5, 0.05, 0.35]), np.array([0.3, 0.9, 0.2, 0.6])
    A, mg = O.resample(O.STRATIFIED, w, u)           # positions .075 .475 .55 .9
    assert A.tolist() == [0, 1, 1, 3] and mg == pytest.approx(0.025, abs=1e-12)
    A, mg = O.resample(O.MULTINOMIAL, w, u)          # positions .3 .9 .2 .6 ; .6 sits exactly on the prefix .6
    assert A.tolist() == [1, 3, 1, 1] and mg == pytest.approx(0.0, abs=1e-15)
    # N W = .4 2 .2 1.4 -> two copies of 1, one of 3, one slot left; residual weights .4 0 .2 .4, first uniform .3
    A, _ = O.resample(O.RESIDUAL, w, u)
    assert A.tolist() == [1, 1, 3, 0]


@pytest.mark.parametrize("N", [1, 2, 5, 32, 257])
def test_other_resamplers_against_library_search(N):
    rng = np.random.default_rng(100 + N)
    for trial in range(20):
        w = rng.exponential(size=N) ** 3
        u = np.array([O.uniform(O.hash5(2, O.STREAM_RESAMPLE, 0, trial, 1 + i)) for i in range(N)])
        W = w / w.sum()
        cdf = np.cumsum(w) / w.sum()
        A, _ = O.resample(O.STRATIFIED, w, u)
        assert np.array_equal(A, np.minimum(np.searchsorted(cdf, (np.arange(N) + u) / N, side="left"), N - 1))
        assert np.all(np.diff(A) >= 0)
        off = np.bincount(A, minlength=N)
        assert np.all(np.abs(off - N * W) < 2.0)      # stratified counts stay within two of their mean
        A, _ = O.resample(O.MULTINOMIAL, w, u)
        assert np.array_equal(A, np.minimum(np.searchsorted(cdf, u, side="left"), N - 1))
        A, _ = O.resample(O.RESIDUAL, w, u)
        fl = np.floor(N * W + 1e-12).astype(int)
        D = int(fl.sum())
        assert np.array_equal(A[:D], np.repeat(np.arange(N), fl))      # the deterministic copies, in order
        res = N * W - fl
        if D < N:
            rc = np.cumsum(res) / res.sum()
            assert np.array_equal(A[D:], np.minimum(np.searchsorted(rc, u[: N - D], side="left"), N - 1))
        assert np.all(np.bincount(A, minlength=N) >= fl)


@pytest.mark.parametrize("kind", [O.SYSTEMATIC, O.STRATIFIED, O.MULTINOMIAL, O.RESIDUAL])
def test_every_resampler_is_unbiased(kind):
    """E[offspring of j] = N W_j (the property Appendix E asks of a resampling scheme), by Monte Carlo."""
    w = np.array([0.03, 0.4, 0.07, 0.25, 0.2, 0.05])
    N, n = w.size, 20000
    counts = np.zeros((n, N))
    for s in range(n):
        if kind == O.SYSTEMATIC:
            A, _ = O.systematic(w, O.uniform(O.hash5(7, O.STREAM_RESAMPLE, 0, s, 0)))
        else:
            A, _ = O.resample(kind, w, [O.uniform(O.hash5(7, O.STREAM_RESAMPLE, 0, s, 1 + i)) for i in range(N)])
        counts[s] = np.bincount(A, minlength=N)
    sem = counts.std(axis=0, ddof=1) / math.sqrt(n)
    assert np.all(np.abs(counts.mean(axis=0) - N * w / w.sum()) < 4.0 * sem + 1e-9)


@pytest.mark.parametrize("kind", [O.STRATIFIED, O.MULTINOMIAL, O.RESIDUAL])
def test_normaliser_estimate_is_unbiased_under_every_resampler(kind):
    V, T, alpha = 3, 4, 4.0
    lm = TinyLM(V, 55)
    _, gam = lm.enumerate(T, alpha, V - 1)
    Z = gam.sum()
    n = 12000
    o = O.Oracle(N=4, V=V, alpha=alpha, tau=1.0 / alpha, kappa=0.9, ramp=0, seed=0, eos=V - 1, T_max=T)
    o.set_resampler(kind)
    zs = np.empty(n)
    resamples = 0
    for s in range(n):
        o.reset(5000 + s)
        for _ in range(T):
            o.step(lm.logits(o.last_tokens))
            resamples += int(o.resampled[0])
        zs[s] = math.exp(o.log_z_final[0])
    assert resamples > n // 20
    sem = zs.std(ddof=1) / math.sqrt(n)
    assert abs(zs.mean() - Z) < 4.0 * sem + 1e-12, (zs.mean(), Z, sem)


def test_slot_map_properties_and_hand_examples():
    assert O.slot_map([1, 2, 3, 3]).tolist() == [3, 1, 2, 3]
    assert O.slot_map([0, 0, 0, 0]).tolist() == [0, 0, 0, 0]
    assert O.slot_map([0, 1, 2, 3]).tolist() == [0, 1, 2, 3]
    assert O.slot_map([2, 2, 2, 5, 5, 7, 7, 7]).tolist() == [2, 2, 2, 5, 7, 5, 7, 7]
    rng = np.random.default_rng(0)
    for N in (1, 3, 8, 32, 100):
        for _ in range(50):
            A, _ = O.systematic(rng.exponential(size=N) ** 4, rng.uniform())
            m = O.slot_map(A)
            assert sorted(m.tolist()) == sorted(A.tolist())        # same multiset of particles
            alive = np.bincount(A, minlength=N) > 0
            assert np.all(m[alive] == np.arange(N)[alive])          # survivors keep their slot
            written = np.nonzero(m != np.arange(N))[0]
            assert not set(written) & set(m.tolist())               # nothing is both read and written


# ---------------------------------------------------------------- the schedule
def test_alpha_schedule():
    assert O.alpha_at(4.0, 0, 0) == 4.0 and O.alpha_at(4.0, 0, 17) == 4.0
    assert O.alpha_at(4.0, 128, 0) == 1.0
    assert O.alpha_at(4.0, 128, 64) == 2.5
    assert O.alpha_at(4.0, 128, 128) == 4.0 and O.alpha_at(4.0, 128, 500) == 4.0
    assert O.beta_at(4.0, 0.25, 128, 64) == 2.5      # tau = 1/alpha: proposal exponent = alpha_t
    assert O.beta_at(4.0, 0.5, 0, 3) == 2.0
    assert O.beta_at(1.0, 1.0, 0, 3) == 1.0


# ---------------------------------------------------------------- a small first-order language model
class TinyLM:
    """p(v | prev) from a random logit table; index V of the table is the start state."""

    def __init__(self, V, seed, spread=1.5):
        rng = np.random.default_rng(seed)
        self.V = V
        self.table = rng.normal(0, spread, size=(V + 1, V))

    def logits(self, last_tokens):
        prev = np.where(np.asarray(last_tokens) < 0, self.V, last_tokens)
        return self.table[prev]

    def logp(self):
        return special.log_softmax(self.table, axis=1)

    def enumerate(self, T, alpha, eos):
        """All length-T strings of the absorbing-EOS model with p(y)^alpha; returns (strings, gamma)."""
        lp = self.logp()
        strings, gam = [], []
        for y in itertools.product(range(self.V), repeat=T):
            prev, s, ok, ended = self.V, 0.0, True, False
            for tok in y:
                if ended:
                    if tok != eos:
                        ok = False
                        break
                    continue
                s += lp[prev, tok]
                prev = tok
                ended = tok == eos
            if ok:
                strings.append(y)
                gam.append(math.exp(alpha * s))
        return strings, np.array(gam)


def run_smc(lm, o, T, force_tok=None):
    for _ in range(T):
        o.step(lm.logits(o.last_tokens), force_tok=force_tok)


def test_alpha_one_tau_one_never_resamples():
    lm = TinyLM(5, 1)
    o = O.Oracle(N=6, V=5, alpha=1.0, tau=1.0, kappa=0.99, ramp=0, seed=3, eos=4, T_max=12)
    for _ in range(12):
        o.step(lm.logits(o.last_tokens))
        assert np.all(np.abs(o.log_inc) < 1e-14) and np.all(np.abs(o.log_weights) < 1e-13)
        assert o.ess[0] == pytest.approx(6.0, abs=1e-10) and o.resampled[0] == 0


@pytest.mark.parametrize("ramp", [0, 3, 7, 20])
def test_ramp_telescopes_to_the_final_exponent(ramp):
    """With resampling switched off the path weight is alpha_T * log p(y) - sum log q_t(y_t)."""
    V, T, alpha, tau = 6, 12, 4.0, 0.25
    lm = TinyLM(V, 2)
    o = O.Oracle(N=5, V=V, alpha=alpha, tau=tau, kappa=1e-9, ramp=ramp, seed=8, eos=V - 1, T_max=T)
    sum_logq = np.zeros(5)
    sum_logp = np.zeros(5)
    last = o.last_tokens
    done = np.zeros(5, bool)
    for t in range(1, T + 1):
        lg = lm.logits(last)
        beta = O.alpha_at(alpha, ramp, t) / (alpha * tau)
        o.step(lg)
        tok = o.tokens
        for i in range(5):
            if not done[i]:
                sum_logq[i] += special.log_softmax(beta * lg[i])[tok[i]]
                sum_logp[i] += special.log_softmax(lg[i])[tok[i]]
        done |= tok == V - 1
        last = o.last_tokens
        assert o.resampled[0] == 0
    a_T = O.alpha_at(alpha, ramp, T)
    assert np.allclose(o.log_weights, a_T * sum_logp - sum_logq, atol=1e-10)
    assert np.allclose(o.cum_logp, sum_logp, atol=1e-12)


def test_eos_is_absorbing():
    V, T = 5, 9
    lm = TinyLM(V, 4)
    o = O.Oracle(N=3, V=V, alpha=3.0, tau=1 / 3.0, kappa=1e-9, ramp=4, seed=1, eos=V - 1, T_max=T)
    o.step(lm.logits(o.last_tokens))
    o.step(lm.logits(o.last_tokens), force_tok=np.array([-1, V - 1, -1]))   # particle 1 is put on EOS
    assert o.tokens[1] == V - 1 and o.done.tolist()[1] == 1
    inc_at_eos = o.log_inc[1]
    assert inc_at_eos != 0.0                  # the EOS token's own factor is applied
    len1, S1 = o.lens[1], o.cum_logp[1]
    for _ in range(3):
        before = o.log_weights[1]
        t_next = o.t + 1
        delta = O.alpha_at(3.0, 4, t_next) - O.alpha_at(3.0, 4, t_next - 1)
        o.step(lm.logits(o.last_tokens))
        assert o.tokens[1] == V - 1 and o.log_inc[1] == 0.0
        assert o.lens[1] == len1 and o.cum_logp[1] == S1
        assert o.log_weights[1] == pytest.approx(before + delta * S1, abs=1e-12)  # only the stage boundary moves it
    assert o.lens[0] == 5 and o.lens[1] == 2


def test_resampling_copies_state_and_resets_weights():
    V, N = 7, 8
    lm = TinyLM(V, 6, spread=3.0)
    mk = lambda: O.Oracle(N=N, V=V, alpha=4.0, tau=0.25, kappa=1.0, ramp=0, seed=5, eos=V - 1, T_max=30,
                          prompt_len=np.array([10]))
    o, o2 = mk(), mk()
    for x in (o, o2):                      # token 1: shared prefix, Theorem 1 => equal weights, no resampling
        x.step(lm.logits(x.last_tokens))
        assert x.resampled[0] == 0 and x.ess[0] == pytest.approx(N, abs=1e-9)
    # token 2, first with resampling held back to look at the state it would act on ...
    o.step(lm.logits(o.last_tokens), force_resample=np.array([0]))
    lens_b, S_b, lw_b, tok_b = o.lens, o.cum_logp, o.log_weights, o.tokens
    assert o.resampled[0] == 0 and o.resampled_own[0] == int(O.ess(lw_b)["ess"] < 1.0 * N) == 1
    # ... then for real on the twin (kappa = 1: any unevenness triggers)
    o2.step(lm.logits(o2.last_tokens))
    assert o2.resampled[0] == 1
    m, A = o2.slot_map, o2.ancestors
    assert np.array_equal(m, O.slot_map(A))
    assert np.array_equal(o2.lens, lens_b[m]) and np.array_equal(o2.cum_logp, S_b[m])
    assert np.array_equal(o2.last_tokens, tok_b[m]) and np.array_equal(o2.tokens, tok_b)
    assert np.all(o2.log_weights == 0.0)
    e = O.ess(lw_b)
    assert o2.log_z[0] == pytest.approx(e["M"] + math.log(e["s1"] / N), abs=1e-13)
    w = np.exp(lw_b - e["M"])
    u0 = O.uniform(O.hash5(5, O.STREAM_RESAMPLE, 0, 2, 0))
    assert np.array_equal(A, O.systematic(w, u0)[0])
    assert np.all(o2.lens[np.bincount(A, minlength=N) > 0] == 12)


def test_first_step_rows_share_logits_but_not_uniforms():
    V, N = 50, 16
    lm = TinyLM(V, 7)
    o = O.Oracle(N=N, V=V, alpha=2.0, tau=0.5, kappa=1e-9, ramp=0, seed=2, eos=V - 1, T_max=2)
    lg = lm.logits(o.last_tokens)
    assert np.all(lg == lg[0])
    o.step(lg)
    assert len(set(o.tokens.tolist())) > 1
    for i in range(N):
        U = O.uniform(O.hash5(2, O.STREAM_TOKEN, 0, 1, i))
        assert o.tokens[i] == O.row(lg[i], 2.0, 2.0, U)["y"]


# ---------------------------------------------------------------- brute force on tiny V and T
@pytest.mark.parametrize("V,T,alpha,ramp,kappa", [(3, 3, 4.0, 0, 0.9), (4, 4, 2.0, 0, 0.9), (3, 5, 4.0, 3, 0.8),
                                                  (4, 3, 3.0, 2, 1.0)])
def test_normaliser_estimate_is_unbiased(V, T, alpha, ramp, kappa):
    """E[Z-hat] = Z_T = sum over all strings of p(y_{1:T})^alpha (Eq. 1 and Eq. 6), by enumeration."""
    lm = TinyLM(V, 100 + V + T)
    _, gam = lm.enumerate(T, alpha, V - 1)
    Z = gam.sum()
    n, N = 12000, 4
    o = O.Oracle(N=N, V=V, alpha=alpha, tau=1.0 / alpha, kappa=kappa, ramp=ramp, seed=0, eos=V - 1, T_max=T)
    zs = np.empty(n)
    resamples = 0
    for s in range(n):
        o.reset(1000 + s)
        for _ in range(T):
            o.step(lm.logits(o.last_tokens))
            resamples += int(o.resampled[0])
        zs[s] = math.exp(o.log_z_final[0])
    assert resamples > n // 20                       # the resampling branch is really exercised
    sem = zs.std(ddof=1) / math.sqrt(n)
    assert abs(zs.mean() - Z) < 4.0 * sem + 1e-12, (zs.mean(), Z, sem)


def test_normaliser_estimate_is_unbiased_for_a_non_optimal_proposal():
    V, T, alpha = 3, 4, 3.0
    lm = TinyLM(V, 77)
    _, gam = lm.enumerate(T, alpha, V - 1)
    n = 12000
    o = O.Oracle(N=4, V=V, alpha=alpha, tau=0.7, kappa=0.6, ramp=0, seed=0, eos=V - 1, T_max=T)
    zs = np.empty(n)
    for s in range(n):
        o.reset(5000 + s)
        run_smc(lm, o, T)
        zs[s] = math.exp(o.log_z_final[0])
    sem = zs.std(ddof=1) / math.sqrt(n)
    assert abs(zs.mean() - gam.sum()) < 4.0 * sem


def test_selected_strings_approach_the_power_distribution():
    """The output law tends to pi_alpha (Eq. 1) as N grows; the finite-N bias shrinks like 1/N."""
    V, T, alpha = 3, 4, 3.0
    lm = TinyLM(V, 31, spread=1.0)
    strings, gam = lm.enumerate(T, alpha, V - 1)
    pi = gam / gam.sum()
    index = {s: k for k, s in enumerate(strings)}
    tv = {}
    for N, runs in ((4, 6000), (64, 3000), (1024, 1500)):
        o = O.Oracle(N=N, V=V, alpha=alpha, tau=1.0 / alpha, kappa=0.5, ramp=0, seed=0, eos=V - 1, T_max=T)
        counts = np.zeros(len(strings))
        for s in range(runs):
            o.reset(9000 + s)
            run_smc(lm, o, T)
            toks, ln, ix = o.select()
            y = tuple(int(x) for x in toks[0, :T])
            counts[index[y]] += 1          # the string must be a legal one (KeyError otherwise)
            first_eos = y.index(V - 1) + 1 if (V - 1) in y else T
            assert ln[0] == first_eos
        tv[N] = 0.5 * np.abs(counts / runs - pi).sum()
        noise = 0.5 * np.sum(np.sqrt(pi * (1 - pi) / runs)) * math.sqrt(2 / math.pi)  # E[TV] of an exact sampler
        if N >= 64:
            assert tv[N] < 3.0 * noise + 2.0 / N, (N, tv[N], noise)
    assert tv[4] > tv[64]
    # low-temperature decoding alone (N = 1, no correction possible) is visibly off the target
    q_lp = np.zeros(len(strings))
    lpq = special.log_softmax(alpha * lm.table, axis=1)
    for k, y in enumerate(strings):
        prev, s, ended = V, 0.0, False
        for tok in y:
            if not ended:
                s += lpq[prev, tok]
                prev = tok
                ended = tok == V - 1
        q_lp[k] = math.exp(s)
    assert 0.5 * np.abs(q_lp - pi).sum() > 3 * tv[1024]


def test_select_backtrace_follows_the_ancestry():
    V, N, T = 6, 8, 25
    lm = TinyLM(V, 12, spread=2.5)
    o = O.Oracle(N=N, V=V, alpha=4.0, tau=0.25, kappa=0.8, ramp=5, seed=4, eos=V - 1, T_max=T)
    paths = [[] for _ in range(N)]                    # explicit prefix copies, as Algorithm 1 states them
    for _ in range(T):
        o.step(lm.logits(o.last_tokens))
        tok, m = o.tokens, o.slot_map
        paths = [paths[i] + [int(tok[i])] for i in range(N)]
        paths = [list(paths[m[k]]) for k in range(N)]
    toks, ln, ix = o.select()
    assert toks[0, :T].tolist() == paths[ix[0]]
    lw = o.log_weights
    w = np.exp(lw - lw.max())
    U = O.uniform(O.hash5(4, O.STREAM_SELECT, 0, 0, 0))
    assert ix[0] == int(np.searchsorted(np.cumsum(w), U * w.sum(), side="left"))


# ---------------------------------------------------------------- Appendix C
def test_reindex_is_index_select_on_the_particle_dimension():
    rng = np.random.default_rng(1)
    R, H, L, D = 6, 3, 10, 4
    src = rng.normal(size=(R, H, L, D)).astype(np.float32)
    idx = np.array([4, 4, 0, 5, 1, 1], dtype=np.int32)
    dst = np.zeros_like(src)
    O.reindex_tensor(dst, src, idx)
    assert np.array_equal(dst, src[idx])
    # in place with a hazard-free map and live lengths: only [0, len) moves, the tail stays
    m = O.slot_map([1, 1, 1, 3, 3, 5])           # -> slots 0, 2, 4 are rewritten
    lens = np.array([7, 7, 7, 4, 4, 9], dtype=np.int32)
    buf = src.copy()
    O.reindex_tensor(buf, buf, m, lens)
    want = src.copy()
    for k in range(R):
        if m[k] != k:
            want[k, :, : lens[k]] = src[m[k], :, : lens[k]]
    assert np.array_equal(buf, want)
    assert np.array_equal(buf[0, :, 7:], src[0, :, 7:]) and not np.array_equal(buf[0], src[0])
    # positions below copy_from stay as well: the form for rows that share a prompt
    start = np.array([3, 3, 3, 2, 2, 0], dtype=np.int32)
    buf = src.copy()
    O.reindex_tensor(buf, buf, m, lens, start)
    want = src.copy()
    for k in range(R):
        if m[k] != k:
            want[k, :, start[k]: lens[k]] = src[m[k], :, start[k]: lens[k]]
    assert np.array_equal(buf, want)
    assert np.array_equal(buf[0, :, :3], src[0, :, :3]) and np.array_equal(buf[0, :, 3:7], src[1, :, 3:7])


# ---------------------------------------------------------------- proposal restricted to top-k / a nucleus
def test_masked_proposal_hand_worked(golden_dir):
    l = np.array([math.log(4.0), 0.0, math.log(2.0), 0.0])
    for line in open(os.path.join(golden_dir, "masked_proposal_row.txt")):
        if line.startswith("#") or not line.strip():
            continue
        top_k, top_p, U, k, tok, lw, lq = line.split()
        r = O.row_masked(l, 2.0, 2.0, float(U), top_k=int(top_k), top_p=float(top_p))
        assert (r["k"], r["y"]) == (int(k), int(tok))
        assert r["log_omega"] == pytest.approx(float(lw), abs=1e-13)
        assert r["logq_y"] == pytest.approx(float(lq), abs=1e-13)


def test_masked_proposal_with_the_whole_vocabulary_is_the_plain_row():
    rng = np.random.default_rng(3)
    l = rng.normal(0, 3, 50)
    l[7] = -np.inf
    for U in (0.01, 0.37, 0.93):
        a, b = O.row(l, 1.7, 2.5, U), O.row_masked(l, 1.7, 2.5, U, top_k=50)
        c = O.row_masked(l, 1.7, 2.5, U, top_k=10**6)
        for key in ("y", "logp_y", "logq_y", "log_omega", "margin"):
            assert a[key] == b[key] == c[key]


def test_top_1_is_greedy_with_weight_p_to_the_alpha():
    l = np.array([0.3, 2.0, -1.0, 2.0, 0.5])                     # two equal maxima: the lower id wins
    lp = l - special.logsumexp(l)
    for U in (0.001, 0.5, 0.999):
        r = O.row_masked(l, 3.0, 4.0, U, top_k=1)
        assert r["y"] == 1 and r["logq_y"] == 0.0
        assert r["log_omega"] == pytest.approx(4.0 * lp[1], abs=1e-14)


@pytest.mark.parametrize("rule", [dict(top_k=6), dict(top_p=0.8)])
def test_masked_weight_is_constant_on_the_set_when_beta_equals_alpha(rule):
    """Theorem 1 carried over to S: with beta = alpha_t, omega = sum_{v in S} p_v^alpha for every token of S."""
    rng = np.random.default_rng(5)
    l = rng.normal(0, 2, 20)
    p = special.softmax(l)
    seen = {}
    for U in np.linspace(0.0005, 0.9995, 400):
        r = O.row_masked(l, 3.0, 3.0, float(U), **rule)
        seen[r["y"]] = r["log_omega"]
        k = r["k"]
    S = np.argsort(-l, kind="stable")[:k]
    assert set(seen) <= set(S.tolist()) and len(seen) >= min(k, 4)
    want = math.log((p[S] ** 3.0).sum())
    for lw in seen.values():
        assert lw == pytest.approx(want, abs=1e-12)


@pytest.mark.parametrize("alpha,beta,rule", [(2.0, 1.3, dict(top_k=5)), (4.0, 4.0, dict(top_p=0.9)), (3.0, 0.8, dict(top_p=0.5))])
def test_masked_weights_average_to_the_restricted_normaliser(alpha, beta, rule):
    """sum_{v in S} q_S(v) omega(v) = sum_{v in S} p_v^alpha: enumerate S through the forcing hook, and check that
    the frequencies of the draws over a fine grid of U are q_S."""
    rng = np.random.default_rng(11)
    l = rng.normal(0, 2.5, 16)
    p = special.softmax(l)
    k = O.row_masked(l, beta, alpha, 0.5, **rule)["k"]
    S = np.argsort(-l, kind="stable")[:k]
    qS = np.zeros(16)
    qS[S] = special.softmax(beta * l[S])
    acc = 0.0
    for v in S:
        r = O.row_masked(l, beta, alpha, 0.5, force=int(v), **rule)
        assert r["logq_y"] == pytest.approx(math.log(qS[v]), abs=1e-12)
        assert r["logp_y"] == pytest.approx(math.log(p[v]), abs=1e-12)          # p over the WHOLE vocabulary
        acc += qS[v] * math.exp(r["log_omega"])
    assert acc == pytest.approx((p[S] ** alpha).sum(), rel=1e-12)
    n = 20000
    counts = np.zeros(16)
    for U in (np.arange(n) + 0.5) / n:
        counts[O.row_masked(l, beta, alpha, float(U), **rule)["y"]] += 1
    assert np.abs(counts / n - qS).max() <= 1.0 / n + 1e-12                       # inverse CDF on a grid: exact to 1/n
    assert counts[np.setdiff1d(np.arange(16), S)].sum() == 0


def test_nucleus_size_rule_ties_and_uniform_rows():
    # uniform row: every token has mass 1/V, so k = ceil(top_p V), lower ids first
    l = np.zeros(10)
    for top_p, k in ((0.05, 1), (0.31, 4), (0.95, 10), (1.0, 10)):
        r = O.row_masked(l, 2.0, 2.0, 0.999999, top_p=top_p)
        assert r["k"] == k and r["y"] == k - 1                                  # the last token of S is id k-1
    # ranked masses 0.5, 0.3, 0.15, 0.05 under beta = 1, stored out of order
    l = np.log(np.array([0.15, 0.5, 0.05, 0.3]))
    for top_p, k, last in ((0.4, 1, 1), (0.7, 2, 3), (0.85, 3, 3), (0.96, 4, 3)):
        r = O.row_masked(l, 1.0, 2.0, 0.999999, top_p=top_p)
        assert r["k"] == k and r["y"] == last
    # the margin is the distance of top_p to the nearer of the two cumulative masses that fence the decision
    r = O.row_masked(l, 1.0, 2.0, 0.5, top_p=0.7)
    assert r["k_margin"] == pytest.approx(0.1, abs=1e-12)
    # an imposed size: zero margin if it satisfies the rule, else by how much it misses
    assert O.row_masked(l, 1.0, 2.0, 0.5, top_p=0.7, force_k=2)["k_margin"] == pytest.approx(0.1, abs=1e-12)
    assert O.row_masked(l, 1.0, 2.0, 0.5, top_p=0.7, force_k=1)["k_margin"] == pytest.approx(0.2, abs=1e-12)   # 0.5 < 0.7
    assert O.row_masked(l, 1.0, 2.0, 0.5, top_p=0.7, force_k=3)["k_margin"] == pytest.approx(0.1, abs=1e-12)   # 0.8 > 0.7 already
    with pytest.raises(ValueError):
        O.row_masked(l, 1.0, 2.0, 0.5, top_k=2, top_p=0.5)
    with pytest.raises(ValueError):
        O.row_masked(l, 1.0, 2.0, 0.5)


def test_masked_steps_keep_the_normaliser_estimate_unbiased_for_the_restricted_target():
    """With top-k proposals the particle system targets p^alpha restricted to strings whose every token lies in its
    step's top-k set: E[Z-hat] is the sum of p(y)^alpha over exactly those strings (brute force on a tiny LM)."""
    V, T, alpha, k = 4, 3, 3.0, 2
    lm = TinyLM(V, 41)
    eos = V - 1
    # enumerate reachable strings by walking the tiny LM with the same top-k rule
    Z = 0.0
    stack = [((), 0.0, -1)]
    while stack:
        pref, logp, last = stack.pop()
        if len(pref) == T or last == eos:
            Z += math.exp(alpha * logp)
            continue
        l = lm.logits(np.array([last]))[0].astype(np.float64)
        lp = l - special.logsumexp(l)
        for v in np.argsort(-l, kind="stable")[:k]:
            stack.append((pref + (int(v),), logp + lp[v], int(v)))
    n = 12000
    o = O.Oracle(N=4, V=V, alpha=alpha, tau=1.0 / alpha, kappa=0.9, ramp=0, seed=0, eos=eos, T_max=T)
    o.set_proposal_mask(top_k=k)
    zs = np.empty(n)
    for s in range(n):
        o.reset(9000 + s)
        run_smc(lm, o, T)
        zs[s] = math.exp(o.log_z_final[0])
        assert (o.k_used[:] == k).all()
    sem = zs.std(ddof=1) / math.sqrt(n)
    assert abs(zs.mean() - Z) < 4.0 * sem + 1e-12, (zs.mean(), Z, sem)
