"""Parity of the CUDA path (through the C-ABI) with the CPU oracle.  Needs a B200."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2602_10273_b200 import binding as B
from paper_2602_10273_b200.workload import cuda as WC
from paper_2602_10273_b200.workload import gen as W

import parity as P

pytestmark = pytest.mark.gpu


def _bf16_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _to_double(t):
    if t.dtype == torch.bfloat16:
        return W.bf16_bits_to_f32(_bf16_bits(t)).astype(np.float64)
    return t.cpu().numpy().astype(np.float64)


def run_logits_pass(logits, beta, alpha_t, u, done=None):
    R, V = logits.shape
    dev = logits.device
    scratch = torch.full((B.logits_pass_scratch_bytes(R, V) + 256,), 0xA5, dtype=torch.uint8, device=dev)
    off = (-scratch.data_ptr()) % 256
    scratch = scratch[off:off + B.logits_pass_scratch_bytes(R, V)]
    tok = torch.full((R,), -7, dtype=torch.int32, device=dev)
    logp = torch.zeros(R, dtype=torch.float64, device=dev)
    loginc = torch.zeros(R, dtype=torch.float64, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ud = torch.from_numpy(np.asarray(u, dtype=np.float64)).to(dev)
    dd = None if done is None else torch.from_numpy(np.asarray(done, dtype=np.uint8)).to(dev)
    for _ in range(2):  # twice: nothing of the first call may leak into the second through the scratch
        B.logits_pass(logits, beta, alpha_t, ud, dd, scratch, tok, logp, loginc, status)
    torch.cuda.synchronize()
    return tok.cpu().numpy(), logp.cpu().numpy(), loginc.cpu().numpy(), int(status.item())


check_rows_against_oracle = P.check_rows_against_oracle


# ------------------------------------------------------------------ the logit pass alone
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("beta", [1.0, 2.0, 4.0, 8.0, 2.71875])
@pytest.mark.parametrize("V", [1000, 1024, 5003, 40000])
def test_logits_pass_matches_oracle(dtype, beta, V):
    torch.manual_seed(V + int(beta * 8))
    R = 9
    logits = (torch.randn(R, V, device="cuda") * 3.0).to(dtype)
    logits[3, : V // 2] = -math.inf                       # zero-mass stretch
    logits[4] = 1.5                                       # flat row
    logits[5] = -math.inf
    logits[5, V - 3] = 0.25                               # one-hot row
    u = np.array([O.uniform(O.hash5(9, 1, 0, V, r)) for r in range(R)])
    u[6], u[7] = 2.0**-53, 1.0 - 2.0**-53                  # the two ends of (0,1)
    tok, logp, loginc, status = run_logits_pass(logits, beta, beta, u)
    assert status == B.OK
    check_rows_against_oracle(logits, beta, beta, u, tok, logp, loginc)
    assert tok[5] == V - 3 and abs(loginc[5]) < 1e-6      # one-hot row: log omega = 0 (closed form), one approximate ex2 away
    assert abs(loginc[4] - (1.0 - beta) * math.log(V)) < 1e-5


def test_logits_pass_random_shapes():
    """Forty seeded draws of (rows, vocabulary, row stride, dtype, beta, alpha_t, finished rows, -inf stretches)."""
    rng = np.random.default_rng(20260211)
    for case in range(40):
        R = int(rng.integers(1, 70))
        V = int(rng.choice([2, 3, 7, 8, 9, 31, 257, 1023, 1024, 1025, 4097, 8999]) if case % 2 else rng.integers(2, 9000))
        dtype = torch.bfloat16 if rng.random() < 0.6 else torch.float32
        ld = V + int(rng.choice([0, 0, 1, 3, 8, 13]))
        beta = float(rng.choice([1.0, 2.0, 4.0, 8.0, 1.0 + 6.0 * rng.random()]))
        alpha_t = beta if rng.random() < 0.6 else beta + 2.0 * rng.random()
        buf = torch.full((R, ld), 7.0, device="cuda").to(dtype)          # the padding must never be read as logits
        vals = torch.from_numpy(rng.normal(0.0, 3.0, size=(R, V)).astype(np.float32)).cuda()
        if rng.random() < 0.4:
            lo = int(rng.integers(0, V))
            vals[int(rng.integers(0, R)), lo: lo + int(rng.integers(1, V))] = -math.inf
            vals[:, int(rng.integers(0, V))] = torch.maximum(vals[:, int(rng.integers(0, V))], torch.tensor(0.0, device="cuda"))
        vals = vals.to(dtype)
        if torch.isinf(vals).all(dim=1).any():
            continue                                                      # a row without mass is the error case, tested elsewhere
        buf[:, :V] = vals
        logits = buf[:, :V]
        done = (rng.random(R) < 0.2).astype(np.uint8)
        u = np.array([O.uniform(O.hash5(77, 1, case, V, r)) for r in range(R)])
        tok, logp, loginc, status = run_logits_pass(logits, beta, alpha_t, u, done=done)
        assert status == B.OK, (case, R, V, ld, dtype, beta)
        live = np.nonzero(done == 0)[0]
        assert (tok[done == 1] == -7).all()
        check_rows_against_oracle(logits, beta, alpha_t, u, tok, logp, loginc, rows=live)


def test_logits_pass_very_long_rows():
    """More spans per row than a lane keeps in registers (300001 logits = 293 spans of 1024), ragged end included."""
    torch.manual_seed(7)
    R, V = 3, 300001
    for dtype, beta in ((torch.bfloat16, 4.0), (torch.float32, 2.71875)):
        logits = (torch.randn(R, V, device="cuda") * 3.0).to(dtype)
        u = np.array([O.uniform(O.hash5(13, 1, 0, V, r)) for r in range(R)])
        u[1] = 1.0 - 2.0**-53                               # lands in the last spans
        tok, logp, loginc, status = run_logits_pass(logits, beta, 4.0, u)
        assert status == B.OK
        check_rows_against_oracle(logits, beta, 4.0, u, tok, logp, loginc)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_logits_pass_unaligned_rows_and_non_optimal_proposal(dtype):
    torch.manual_seed(3)
    R, V = 5, 3001
    u = np.array([O.uniform(O.hash5(3, 1, 0, 1, r)) for r in range(R)])
    # ld 3007: rows are not 16-byte aligned (scalar loads); ld 3008: aligned rows with a ragged tail of one logit
    for ld in (3007, 3008):
        base = (torch.randn(R, ld, device="cuda") * 2.0).to(dtype)
        logits = base[:, :V]
        for beta, alpha_t in ((4.0, 4.0), (1.5, 4.0), (3.0, 2.0)):
            tok, logp, loginc, status = run_logits_pass(logits, beta, alpha_t, u)
            assert status == B.OK
            check_rows_against_oracle(logits, beta, alpha_t, u, tok, logp, loginc)


def test_logits_pass_skips_done_rows_and_flags_bad_rows():
    R, V = 6, 4096
    logits = torch.randn(R, V, device="cuda").to(torch.bfloat16)
    u = np.full(R, 0.37)
    done = np.array([0, 1, 0, 0, 1, 0], dtype=np.uint8)
    tok, logp, loginc, status = run_logits_pass(logits, 4.0, 4.0, u, done)
    assert status == B.OK and tok[1] == -7 and tok[4] == -7 and (tok[[0, 2, 3, 5]] >= 0).all()
    for bad in (float("nan"), float("inf")):
        l2 = logits.clone()
        l2[2, 100] = bad
        tok, _, _, status = run_logits_pass(l2, 4.0, 4.0, u)
        assert status == B.E_NUMERIC and tok[2] == -1 and tok[0] >= 0
    l2 = logits.clone()
    l2[3] = -math.inf
    tok, _, _, status = run_logits_pass(l2, 4.0, 4.0, u)
    assert status == B.E_NUMERIC and tok[3] == -1


def test_logits_pass_token_independence_on_device():
    """Theorem 1 on the CUDA path: at beta = alpha the increment does not depend on the uniform."""
    V = 20000
    logits = (torch.randn(1, V, device="cuda") * 3).to(torch.bfloat16).repeat(16, 1).contiguous()
    u = (np.arange(16) + 0.5) / 16
    tok, logp, loginc, status = run_logits_pass(logits, 4.0, 4.0, u)
    assert status == B.OK and len(set(tok.tolist())) > 3
    assert np.ptp(loginc) == 0.0
    assert np.all(np.diff(tok) >= 0)                      # the inverse CDF is monotone in U


# ------------------------------------------------------------------ weights / ESS / resampling on identical state
@pytest.mark.parametrize("resampler", [B.SYSTEMATIC, B.STRATIFIED, B.MULTINOMIAL, B.RESIDUAL])
@pytest.mark.parametrize("N", [1, 2, 4, 8, 32, 33, 100, 1024])
def test_resampling_kernel_bit_exact_on_identical_log_weights(N, resampler):
    rng = np.random.default_rng(N)
    V, G = 64, 3
    for trial in range(4):
        ps = B.Psmc(N, V, 2.0, 0.5, 1.0, 0, 11 + trial, V - 1, G=G, T_max=4, prompt_len=[5, 6, 7])
        orc = O.Oracle(N, V, 2.0, 0.5, 1.0, 0, 11 + trial, V - 1, G=G, T_max=4, prompt_len=[5, 6, 7])
        ps.set_resampler(resampler)
        orc.set_resampler(resampler)
        lw = rng.normal(0, 2.0 + trial, size=G * N)
        lw[N:2 * N] = -1.25                                # group 1: uniform weights, must not resample
        S = rng.normal(-3, 1, size=G * N)
        lens = np.repeat([5, 6, 7], N).astype(np.int32) + rng.integers(0, 3, size=G * N).astype(np.int32)
        ps.set_state(log_w=lw, cum_logp=S, lens=lens)
        orc.set_state(logW=lw, S=S, lens=lens)
        logits = torch.zeros(G * N, V, device="cuda")      # flat logits: log omega = (1-2) ln 64 for every row
        ps.step(logits)
        orc.step(logits.cpu().numpy(), force_tok=ps.tokens.numpy())
        assert ps.sync_status() == B.OK
        assert np.array_equal(ps.resampled.numpy(), orc.resampled) and orc.resampled[1] == 0
        if not np.array_equal(ps.ancestors.numpy(), orc.ancestors):
            # only where the oracle itself reports a position within rounding of a weight prefix (the CUDA prefix
            # is summed in another order) may the two differ
            bad = np.nonzero((ps.ancestors.numpy() != orc.ancestors).reshape(G, N).any(axis=1))[0]
            assert all(orc.anc_margin[g] <= 1e-12 for g in bad), (bad, orc.anc_margin)
            ps.destroy()
            continue                                       # a genuine tie: nothing further to compare in this trial
        assert np.array_equal(ps.slot_map.numpy(), orc.slot_map)
        assert np.array_equal(ps.lens.numpy(), orc.lens)
        assert np.allclose(ps.ess.numpy(), orc.ess, rtol=1e-12)
        assert np.allclose(ps.log_weights.numpy(), orc.log_weights, atol=1e-9)
        assert np.allclose(ps.cum_logp.numpy(), orc.cum_logp, atol=1e-9)
        assert np.allclose(ps.log_z.numpy(), orc.log_z, atol=1e-9)
        ps.destroy()


# ------------------------------------------------------------------ closed loops on the named configurations
def test_closed_loop_tiny_full():
    c = W.CONFIGS["tiny"]
    st = P.closed_loop(c, seed=1, T=c.T, kv_shape=(c.n_layers, c.n_kv_heads, c.max_len, c.head_dim))
    assert st.steps == 64 and st.resample_events > 0 and st.slots_moved > 0
    print("tiny:", st)


@pytest.mark.parametrize("seed", [2, 3])
def test_closed_loop_tiny_other_seeds(seed):
    c = W.CONFIGS["tiny"]
    P.closed_loop(c, seed=seed, T=c.T, kv_shape=(c.n_layers, c.n_kv_heads, c.max_len, c.head_dim))


@pytest.mark.parametrize("resampler", [B.STRATIFIED, B.MULTINOMIAL, B.RESIDUAL])
def test_closed_loop_other_resamplers(resampler):
    c = W.CONFIGS["tiny"]
    st = P.closed_loop(c, seed=4, T=c.T, kv_shape=(c.n_layers, c.n_kv_heads, c.max_len, c.head_dim), resampler=resampler)
    assert st.resample_events > 0 and st.slots_moved > 0
    c = W.CONFIGS["resample_stress"]
    st = P.closed_loop(c, seed=3, T=24, ramp=8, resampler=resampler)
    assert st.resample_events >= 5
    c = W.CONFIGS["batched_prompts"]
    st = P.closed_loop(c, seed=2, T=12, G=4, resampler=resampler)
    assert st.resample_events > 0


def test_closed_loop_random_settings():
    """Twenty seeded draws of (groups, particles, vocabulary, alpha, tau, kappa, ramp, resampler), twelve tokens each."""
    rng = np.random.default_rng(20260212)
    for case in range(20):
        N = int(rng.choice([1, 2, 3, 5, 8, 17, 32, 33, 64]))
        G = int(rng.integers(1, 5))
        V = int(rng.choice([16, 100, 1024, 3001, 20000]))
        alpha = float(rng.choice([1.0, 2.0, 4.0, 8.0, 1.0 + 4.0 * rng.random()]))
        tau = 1.0 / alpha if rng.random() < 0.6 else float(0.2 + rng.random())
        c = W.Workload("case%d" % case, G, N, V, "bf16" if rng.random() < 0.5 else "f32", float(rng.choice([1.0, 3.0, 6.0])),
                       1.5, 12, 3, 9, alpha, tau, float(rng.choice([0.3, 0.5, 0.9, 1.0])), int(rng.choice([0, 0, 4, 30])),
                       1, 2, 16, 32)
        st = P.closed_loop(c, seed=100 + case, T=12, kv_shape=(1, 2, 32, 16), resampler=int(rng.integers(0, 4)))
        assert st.steps == 12


@pytest.mark.parametrize("G,N,V,dtype", [(300, 8, 104, "bf16"), (330, 8, 2048, "bf16"), (1000, 8, 16, "f32"), (40, 32, 1000, "f32")])
def test_closed_loop_many_rows_per_cta(G, N, V, dtype):
    """Shapes whose logit block gives every CTA of the one-kernel step many short rows: 16-18 segments per CTA (beyond
    the fifteen named barriers: the helper polls mbarriers instead), rows of a few granules split over two CTAs, and
    54 rows per CTA (beyond the segment table: the step runs as two kernels)."""
    c = W.Workload("many", G, N, V, dtype, 3.0, 1.5, 6, 2, 5, 4.0, 0.25, 0.7, 0, 1, 1, 8, 16)
    st = P.closed_loop(c, seed=5, T=6, kv_shape=(1, 1, 16, 8))
    assert st.steps == 6 and st.resample_events > 0


@pytest.mark.parametrize("G,N,V,dtype,resampler", [(1, 64, 32000, "bf16", 0), (2, 100, 8192, "bf16", 1), (3, 33, 5000, "f32", 3),
                                                   (1, 128, 151936, "bf16", 0), (1, 1024, 512, "f32", 2)])
def test_closed_loop_groups_of_more_than_32_particles(G, N, V, dtype, resampler):
    """Groups that one warp cannot update (the paper's own runs use 64 particles): the one-kernel step leaves the rows'
    tokens and weights in memory and a second kernel updates the groups.  Sizes that are not multiples of 32, several
    groups, every resampler."""
    c = W.Workload("large_groups", G, N, V, dtype, 3.0, 1.5, 8, 3, 6, 4.0, 0.25, 0.6, 0, 1, 1, 8, 24)
    st = P.closed_loop(c, seed=11, T=8, kv_shape=(1, 1, 24, 8), resampler=resampler)
    assert st.steps == 8 and st.resample_events > 0


def test_closed_loop_llama_shape():
    c = W.CONFIGS["llama2_7b"]
    st = P.closed_loop(c, seed=1, T=96, kv_shape=(2, 4, 512 + 96 + 8, c.head_dim))
    assert st.resample_events > 0
    print("llama2_7b:", st)


def test_closed_loop_qwen_shape_with_ramp():
    c = W.CONFIGS["qwen25_7b"]
    st = P.closed_loop(c, seed=1, T=48, kv_shape=(2, c.n_kv_heads, 256 + 48 + 8, c.head_dim))
    print("qwen25_7b (ramp steps):", st)
    st = P.closed_loop(c, seed=2, T=40, ramp=16)          # leaves the ramp after 16 tokens: beta = 4 exactly
    assert st.resample_events > 0
    print("qwen25_7b (ramp 16):", st)


def test_closed_loop_resampling_stress():
    c = W.CONFIGS["resample_stress"]
    st = P.closed_loop(c, seed=1, T=40, ramp=8, kv_shape=(1, c.n_kv_heads, 128 + 40 + 8, c.head_dim))
    assert st.resample_events >= 10
    print("resample_stress (ramp 8):", st)
    st = P.closed_loop(c, seed=2, T=24)                   # inside the 256-token ramp: fractional exponents
    print("resample_stress (in ramp):", st)


def test_closed_loop_batched_prompts():
    c = W.CONFIGS["batched_prompts"]
    st = P.closed_loop(c, seed=1, T=24, G=8, kv_shape=(1, 2, 256 + 24 + 8, c.head_dim))
    assert st.resample_events > 0
    print("batched_prompts (8 prompts):", st)


def test_closed_loop_batched_prompts_full_size():
    """All 64 prompts x 8 particles x 128256 logits, i.e. the launch configuration the benchmark times (two kernels,
    148 CTAs), every row compared with the oracle; the cache carries every head and position of one layer."""
    c = W.CONFIGS["batched_prompts"]
    st = P.closed_loop(c, seed=1, T=5, kv_shape=(1, c.n_kv_heads, c.max_len, c.head_dim))
    assert st.live_rows == 5 * 512 and st.resample_events > 0 and st.slots_moved > 0
    print("batched_prompts (64 prompts, full size):", st)


@pytest.mark.parametrize("name,G,T", [("batched_prompts", 6, 16), ("tiny", None, 48)])
def test_reindex_leaves_a_shared_prompt_in_place(name, G, T):
    """Rows of a group prefilled with one prompt: only generated positions move, and the cache ends up as if whole
    live prefixes had been copied."""
    c = W.CONFIGS[name]
    st = P.closed_loop(c, seed=2, T=T, G=G, kv_shape=(2, 2, c.prompt_hi + T + 8, c.head_dim), skip_shared_prompt=True)
    assert st.slots_moved > 0


def test_snapshot_resumes_bit_for_bit():
    """Save after 10 tokens, load into a fresh context, go on: the oracle, which never stopped, still agrees at every
    step, and the final draw walks an ancestry log that spans the snapshot."""
    c = W.CONFIGS["tiny"]
    T = 40
    wl, ps, orc = P.make_pair(c, seed=6, T_max=T, resampler=B.RESIDUAL)
    st = P.LoopStats()
    kappa_f = float(np.float32(c.kappa))
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    for t in range(1, T + 1):
        wl.fill(lg, t, prev)
        ps.step(lg)
        P.compare_step(ps, orc, P.logits_to_numpy(lg), st, kappa_f)
        prev.copy_(ps.device_view("psmc_last_tokens", ps.R))
        if t == 10:
            blob = ps.state_save()
            assert len(blob) == B.lib().psmc_state_bytes(ps._h)
            ps.destroy()
            ps = B.Psmc(c.N, c.V, 2.0, 1.0, 0.3, 0, 999, 0, G=1, T_max=T, prompt_len=wl.prompt_len)  # other settings
            ps.state_load(blob)
            other = B.Psmc(c.N, c.V + 1, c.alpha, c.tau, c.kappa, 0, 6, c.eos_id, G=1, T_max=T)
            with pytest.raises(B.PsmcError):
                other.state_load(blob)                       # a different vocabulary: refused, nothing loaded
            other.destroy()
            other = B.Psmc(c.N, c.V, c.alpha, c.tau, c.kappa, 0, 6, c.eos_id, G=1, T_max=T, prompt_len=wl.prompt_len + 1)
            with pytest.raises(B.PsmcError):
                other.state_load(blob)                       # other prompt lengths: the cache calls would skip wrongly
            other.destroy()
    assert st.resample_events > 0
    toks, ln, ix = ps.select()
    o_toks, o_ln, o_ix = orc.select()
    assert np.array_equal(ix.cpu().numpy(), o_ix) and np.array_equal(toks.cpu().numpy(), o_toks)
    assert np.array_equal(ln.cpu().numpy(), o_ln)
    ps.destroy()


def test_eos_rows_freeze_and_are_not_read():
    c = W.CONFIGS["tiny"]

    def push_eos(t, lg):
        if t == 5:
            lg[1, c.eos_id] = 60.0                         # slot 1 is driven onto EOS at token 5

    st = P.closed_loop(c, seed=5, T=20, kappa=0.05, logit_bias_fn=push_eos)
    assert st.steps == 20


def test_finished_slots_are_rewritten_by_live_ancestors_at_every_step():
    """Finished flags that flip back to live while the step kernel is still reading flags elsewhere.  Every other
    token two live slots per group are declared finished with a low weight (on both sides); kappa = 1 resamples at
    once, so at the next token those slots are overwritten by live ancestors: a flag goes from 1 to 0 in a group that
    closes early, while CTAs that hold other parts of the block have not looked at their rows' flags yet.  Rows span
    several CTAs (5000 logits = 20 granules, 6.5 granules per CTA).  Every token is compared, the status stays clean."""
    c = W.Workload("flip", 6, 8, 5000, "bf16", 3.0, 1.5, 300, 5, 9, 4.0, 0.25, 1.0, 0, 1, 2, 16, 320)
    T = 300
    wl, ps, orc = P.make_pair(c, seed=11, T_max=T)
    st = P.LoopStats()
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    flips = 0
    for t in range(1, T + 1):
        before = ps.done.numpy().copy()
        wl.fill(lg, t, prev)
        ps.step(lg)
        P.compare_step(ps, orc, P.logits_to_numpy(lg), st, 1.0)
        after = ps.done.numpy()
        flips += int(((before == 1) & (after == 0)).sum())
        prev.copy_(ps.device_view("psmc_last_tokens", ps.R))
        if t % 2 == 0:
            lw, dn = ps.log_weights.numpy().copy(), after.copy()
            for g in range(c.G):
                live = [r for r in range(g * c.N, (g + 1) * c.N) if not dn[r]]
                for r in live[:2] if len(live) > 3 else []:
                    dn[r] = 1
                    lw[r] -= 40.0
            ps.set_state(log_w=lw, done=dn)
            orc.set_state(logW=lw, done=dn)
    assert ps.sync_status() == B.OK
    assert st.steps == T and st.resample_events > 100 and flips > 100
    ps.destroy()


def test_done_rows_logits_are_never_read():
    V, N = 2048, 4
    ps = B.Psmc(N, V, 4.0, 0.25, 0.01, 0, 3, V - 1, T_max=4)
    ps.set_state(done=np.array([0, 1, 0, 1], dtype=np.uint8))
    lg = torch.randn(N, V, device="cuda")
    lg[1] = float("nan")
    lg[3] = float("inf")
    ps.step(lg)
    assert ps.sync_status() == B.OK
    assert ps.tokens.numpy()[[1, 3]].tolist() == [V - 1, V - 1] and ps.log_inc.numpy()[[1, 3]].tolist() == [0.0, 0.0]
    ps.destroy()


# ------------------------------------------------------------------ KV reindex
@pytest.mark.parametrize("dtype,D", [(torch.bfloat16, 128), (torch.float32, 64), (torch.bfloat16, 20), (torch.float32, 3)])
def test_reindex_out_of_place_is_index_select(dtype, D):
    R, H, ML, L = 6, 3, 37, 2
    ps = B.Psmc(R, 16, 2.0, 0.5, 0.5, 0, 1, 15, T_max=2)
    ks = [torch.randn(R, H, ML, D, device="cuda").to(dtype) for _ in range(L)]
    vs = [torch.randn(R, H, ML, D, device="cuda").to(dtype) for _ in range(L)]
    kd = [torch.zeros_like(t) for t in ks]
    vd = [torch.zeros_like(t) for t in vs]
    idx = torch.tensor([4, 4, 0, 5, 1, 1], dtype=torch.int32, device="cuda")
    ps.reindex_kv(ps.make_kv_desc(ks, vs), ps.make_kv_desc(kd, vd), idx)
    assert ps.sync_status() == B.OK
    for s, d in zip(ks + vs, kd + vd):
        assert torch.equal(d, s[idx.long()])
    ps.destroy()


def test_reindex_more_layers_than_one_launch_takes():
    """70 layers: the pointer table of a launch holds 64, so the call takes two launches that share the unit queue."""
    R, H, ML, D, L = 6, 1, 8, 8, 70
    ps = B.Psmc(R, 16, 2.0, 0.5, 0.5, 0, 1, 15, T_max=2)
    ks = [torch.randn(R, H, ML, D, device="cuda").to(torch.bfloat16) for _ in range(L)]
    vs = [torch.randn(R, H, ML, D, device="cuda").to(torch.bfloat16) for _ in range(L)]
    want = [t.clone() for t in ks + vs]
    idx = torch.tensor([2, 1, 2, 2, 4, 4], dtype=torch.int32, device="cuda")
    for _ in range(2):                                      # twice: the queue must come back to zero in between
        ps.reindex_kv(ps.make_kv_desc(ks, vs), None, idx)
    assert ps.sync_status() == B.OK
    for t, w in zip(ks + vs, want):
        assert torch.equal(t, w[idx.long()])
    ps.destroy()


def test_reindex_in_place_override_and_hazard_detection():
    R, H, ML, D = 6, 2, 16, 64
    ps = B.Psmc(R, 16, 2.0, 0.5, 0.5, 0, 1, 15, T_max=2)
    ks = [torch.randn(R, H, ML, D, device="cuda").to(torch.bfloat16)]
    vs = [torch.randn(R, H, ML, D, device="cuda").to(torch.bfloat16)]
    want_k, want_v = ks[0].clone(), vs[0].clone()
    desc = ps.make_kv_desc(ks, vs)
    good = torch.tensor([1, 1, 1, 3, 3, 5], dtype=torch.int32, device="cuda")
    ps.reindex_kv(desc, None, good)
    assert ps.sync_status() == B.OK
    assert torch.equal(ks[0], want_k[good.long()]) and torch.equal(vs[0], want_v[good.long()])
    before = ks[0].clone()
    bad = torch.tensor([1, 2, 3, 3, 4, 5], dtype=torch.int32, device="cuda")   # row 1 is read and rewritten
    ps.reindex_kv(desc, None, bad)
    assert ps.sync_status() == B.E_HAZARD
    assert torch.equal(ks[0], before)                       # nothing was written
    ps.destroy()


def test_reindex_strided_cache_and_misaligned_base():
    """Caches that are views into larger buffers: row/head strides larger than the tight ones, odd offsets."""
    R, H, ML, D = 4, 2, 9, 8
    ps = B.Psmc(R, 16, 2.0, 0.5, 0.5, 0, 1, 15, T_max=2)
    for off in (0, 1, 3):                                   # element offsets: 2-byte and 6-byte misalignment
        big = torch.randn(R * (H + 1) * (ML + 2) * D + 8, device="cuda").to(torch.bfloat16)
        view = big[off: off + R * (H + 1) * (ML + 2) * D].view(R, H + 1, ML + 2, D)[:, :H, :ML, :]
        k, v = view, view.clone().contiguous()
        ref_k, ref_v, ref_big = k.clone(), v.clone(), big.clone()
        idx = torch.tensor([2, 1, 2, 2], dtype=torch.int32, device="cuda")
        # once the strided view, once a tight tensor of the same shape (each as both K and V of one layer)
        import ctypes as C
        for t, ref in ((k, ref_k), (v, ref_v)):
            arr = (C.c_void_p * 1)(t.data_ptr())
            d = B.KvDesc(1, C.cast(arr, C.POINTER(C.c_void_p)), C.cast(arr, C.POINTER(C.c_void_p)), H, D, ML, B.BF16,
                         t.stride(0), t.stride(1))
            ps.reindex_kv(d, None, idx)
            assert ps.sync_status() == B.OK
            assert torch.equal(t, ref[idx.long()])
        # the padding between heads/positions of the big buffer is untouched
        mask = torch.ones_like(big, dtype=torch.bool)
        mview = mask[off: off + R * (H + 1) * (ML + 2) * D].view(R, H + 1, ML + 2, D)
        mview[:, :H, :ML, :] = False
        assert torch.equal(big[mask], ref_big[mask])
    ps.destroy()


# ------------------------------------------------------------------ generators: CUDA twin vs numpy
def test_cuda_generators_match_numpy():
    seed, V, N = 4, 6000, 4
    bias = W.vocab_bias(seed, V, 1.5)
    prev = np.array([5, 5, 77, 4000, 1, 2, 3, 4], dtype=np.int32)
    for dtype, tdt in (("f32", torch.float32), ("bf16", torch.bfloat16)):
        dst = torch.empty(8, V, dtype=tdt, device="cuda")
        WC.fill_logits(dst, seed, 3, N, torch.from_numpy(prev).cuda(), 3.0, torch.from_numpy(bias).cuda())
        ref = W.logits_block(seed, 3, np.arange(8) // N, prev, V, 3.0, bias, dtype)
        got = P.logits_to_numpy(dst)
        flips = int((got != ref).sum())
        assert flips <= 3, "%d of %d elements differ" % (flips, got.size)   # last-ulp libm differences only
        if dtype == "f32":
            assert np.abs(got - ref).max() <= 4e-6
        kv = torch.empty(3, 2, 16, 32, dtype=tdt, device="cuda")
        WC.fill_kv(kv, seed, 1, 1, row0=2)
        ref = W.kv_block(seed, 1, 1, [2, 3, 4], 2, 16, 32, dtype)
        got = (kv.view(torch.int16) if tdt == torch.bfloat16 else kv).cpu().numpy()
        got = got.view(np.uint16) if dtype == "bf16" else got
        assert int((got != ref).sum()) <= 2


# ------------------------------------------------------------------ brute force through the C-ABI
@pytest.mark.parametrize("N,runs", [(4, 3000), (32, 1500)])
def test_power_distribution_and_normaliser_through_the_cabi(N, runs):
    from test_oracle_pins import TinyLM
    V, T, alpha = 3, 4, 3.0
    lm = TinyLM(V, 31, spread=1.0)
    strings, gam = lm.enumerate(T, alpha, V - 1)
    pi, Z = gam / gam.sum(), gam.sum()
    index = {s: k for k, s in enumerate(strings)}
    G = 500                                                # 500 independent runs per context, batched as groups
    table = torch.from_numpy(lm.table.astype(np.float32)).cuda()
    counts = np.zeros(len(strings))
    zs = []
    for rep in range(runs // G):
        ps = B.Psmc(N, V, alpha, 1.0 / alpha, 0.5, 0, 7000 + rep, V - 1, G=G, T_max=T)
        last = ps.device_view("psmc_last_tokens", ps.R)
        for t in range(T):
            prev = torch.where(last < 0, torch.full_like(last, V), last).long()
            ps.step(table[prev].contiguous())
        toks, ln, ix = ps.select()
        lw = ps.log_weights.numpy().reshape(G, N)
        M = lw.max(axis=1)
        zs.append(np.exp(ps.log_z.numpy() + M + np.log(np.exp(lw - M[:, None]).sum(axis=1) / N)))
        for row in toks.cpu().numpy()[:, :T]:
            counts[index[tuple(int(x) for x in row)]] += 1
        assert ps.sync_status() == B.OK
        ps.destroy()
    n = counts.sum()
    zs = np.concatenate(zs)
    assert abs(zs.mean() - Z) < 4.0 * zs.std(ddof=1) / math.sqrt(zs.size)
    tv = 0.5 * np.abs(counts / n - pi).sum()
    noise = 0.5 * np.sum(np.sqrt(pi * (1 - pi) / n)) * math.sqrt(2 / math.pi)
    if N >= 32:
        assert tv < 3.0 * noise + 2.0 / N, (tv, noise)
    else:
        assert tv < 0.5


# ------------------------------------------------------------------ host-visible errors
def test_argument_errors_return_codes():
    import ctypes as C
    L = B.lib()
    h = C.c_void_p()
    assert L.psmc_init(C.byref(h), 0, 100, 4.0, 0.25, 0.5, 0, 1, 99) == B.E_INVAL
    assert L.psmc_init(C.byref(h), 4, 1, 4.0, 0.25, 0.5, 0, 1, 0) == B.E_INVAL
    assert L.psmc_init(C.byref(h), 4, 100, 0.5, 0.25, 0.5, 0, 1, 99) == B.E_INVAL
    assert L.psmc_init(C.byref(h), 4, 100, 4.0, 0.0, 0.5, 0, 1, 99) == B.E_INVAL
    assert L.psmc_init(C.byref(h), 4, 100, 4.0, 0.25, 1.5, 0, 1, 99) == B.E_INVAL
    assert L.psmc_init(C.byref(h), 4, 100, 4.0, 0.25, 0.5, 0, 1, 100) == B.E_INVAL
    assert L.psmc_init(C.byref(h), 2000, 100, 4.0, 0.25, 0.5, 0, 1, 99) == B.E_INVAL
    assert L.psmc_step(None, None, 0, 0, None) == B.E_INVAL
    ps = B.Psmc(4, 100, 4.0, 0.25, 0.5, 0, 1, 99, T_max=1)
    lg = torch.zeros(4, 100, device="cuda")
    assert L.psmc_step(ps._h, lg.data_ptr(), 7, 100, None) == B.E_INVAL
    assert L.psmc_step(ps._h, lg.data_ptr(), 0, 99, None) == B.E_INVAL
    ps.step(lg)
    with pytest.raises(B.PsmcError) as e:
        ps.step(lg)
    assert e.value.code == B.E_STATE
    ps.destroy()


def test_step_host_matches_device_step():
    c = W.CONFIGS["tiny"]
    wl, ps, orc = P.make_pair(c, 9, T_max=6)
    ps2 = B.Psmc(c.N, c.V, c.alpha, c.tau, c.kappa, c.ramp, 9, c.eos_id, T_max=6, prompt_len=wl.prompt_len)
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    out = torch.empty(ps.R, dtype=torch.int32).pin_memory()
    for t in range(1, 7):
        wl.fill(lg, t, prev)
        ps.step(lg)
        host = lg.cpu().pin_memory()
        ps2.step_host(host, out)
        assert torch.equal(out, ps.last_tokens)
        assert torch.equal(ps2.log_weights, ps.log_weights)
        prev.copy_(ps.device_view("psmc_last_tokens", ps.R))
    ps.destroy()
    ps2.destroy()


@pytest.mark.parametrize("name", ["llama2_7b", "qwen25_7b"])
def test_two_contexts_on_two_streams_do_not_disturb_each_other(name):
    """Two runs with different seeds interleaved on two streams (each context owns its scratch, counters and move
    lists): every state view equals that of the same run made alone, bit for bit.  The step kernels of the two
    contexts may overlap or take turns on the SMs: no CTA of a step kernel waits for another CTA, so neither order
    can stall or time out (the second configuration streams 4.9 MB per step with 18-warp CTAs on every SM)."""
    c = W.CONFIGS[name]
    T, kv_shape = 12, (1, 2, c.prompt_hi + 20, c.head_dim)

    def prepare(seed):
        wl = WC.DeviceWorkload(c, seed)
        ps = B.Psmc(c.N, c.V, c.alpha, c.tau, c.kappa, c.ramp, seed, c.eos_id, G=c.G, T_max=T, prompt_len=wl.prompt_len)
        ks = [torch.empty((wl.R,) + kv_shape[1:], dtype=wl.tdtype, device="cuda") for _ in range(kv_shape[0])]
        vs = [torch.empty_like(k) for k in ks]
        for l, (k, v) in enumerate(zip(ks, vs)):
            WC.fill_kv(k, seed, l, 0)
            WC.fill_kv(v, seed, l, 1)
        return dict(wl=wl, ps=ps, ks=ks, vs=vs, desc=ps.make_kv_desc(ks, vs), lg=wl.new_logits(),
                    prev=wl.first_prev.clone(), last=ps.device_view("psmc_last_tokens", wl.R))

    def advance(run, t, stream):
        with torch.cuda.stream(stream):
            run["wl"].fill(run["lg"], t, run["prev"])
            run["ps"].step(run["lg"])
            run["ps"].reindex_kv(run["desc"])
            run["prev"].copy_(run["last"])

    def snapshot(run):
        torch.cuda.synchronize()
        ps = run["ps"]
        views = [getattr(ps, n).numpy().copy() for n in ("tokens", "last_tokens", "log_weights", "cum_logp", "slot_map",
                                                         "ancestors", "ess", "log_z", "lens", "done")]
        return views + [t.view(torch.int16).cpu().numpy().copy() for t in run["ks"] + run["vs"]]

    alone = []
    for seed in (21, 22):
        run = prepare(seed)
        for t in range(1, T + 1):
            advance(run, t, torch.cuda.current_stream())
        alone.append(snapshot(run))
        run["ps"].destroy()
    runs = [prepare(21), prepare(22)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for t in range(1, T + 1):
        for run, s in zip(runs, streams):
            advance(run, t, s)
    for run, want in zip(runs, alone):
        got = snapshot(run)
        assert all(np.array_equal(a, b, equal_nan=True) for a, b in zip(got, want))
        assert run["ps"].sync_status() == B.OK
        run["ps"].destroy()
