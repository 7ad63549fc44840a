"""Closed-loop parity harness: the CUDA path and the CPU oracle run side by side on the same bits.

Each step the device generator writes the logits block, the CUDA step consumes it in place, the
block is downloaded and the oracle consumes the same bytes.  Where the two may legitimately part
(a uniform within 1e-6 of a CDF boundary, an ESS within 1e-4*N of the threshold, a resampling
position within 2e-4 of a weight prefix) the oracle adopts the CUDA choice through its hooks and the
event is counted; any other difference fails.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle import oracle as O
from paper_2602_10273_b200 import binding as B
from paper_2602_10273_b200.workload import cuda as WC
from paper_2602_10273_b200.workload import gen as W

TOL_LOGW = 1e-4      # absolute, every step
TOL_LOGINC = 1e-5    # absolute, per step
TOK_MARGIN = 1e-6    # CDF units
ESS_MARGIN = 1e-4    # times N
ANC_MARGIN = 2e-4    # normalised weight-prefix units
K_MARGIN = 4e-6      # share of the proposal's mass: how far a nucleus size may miss the rule (fp32 masses, 2^-40 fixed point)


@dataclasses.dataclass
class LoopStats:
    steps: int = 0
    live_rows: int = 0
    tok_adopted: int = 0
    k_adopted: int = 0
    ess_adopted: int = 0
    anc_adopted: int = 0
    resample_events: int = 0
    slots_moved: int = 0
    max_logw_err: float = 0.0
    max_s_err: float = 0.0        # cumulative log p(y_{1:t}), never reset by resampling
    max_loginc_err: float = 0.0
    min_tok_margin: float = 1.0


def logits_to_numpy(t: torch.Tensor) -> np.ndarray:
    """Device logits -> host array the oracle reads (fp32 as is, bf16 as uint16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def logits_to_double(t: torch.Tensor) -> np.ndarray:
    """Device logits as the doubles they stand for (bf16 and fp32 are both exact in a double)."""
    if t.dtype == torch.bfloat16:
        return W.bf16_bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16)).astype(np.float64)
    return t.cpu().numpy().astype(np.float64)


def check_rows_against_oracle(logits, beta, alpha_t, u, tok, logp, loginc, rows=None):
    lg = logits_to_double(logits)
    flagged = 0
    for r in (range(lg.shape[0]) if rows is None else rows):
        o = O.row(lg[r], beta, alpha_t, float(u[r]))
        if o["y"] != tok[r]:
            assert o["margin"] <= TOK_MARGIN, "row %d: %d vs %d margin %.3e" % (r, tok[r], o["y"], o["margin"])
            flagged += 1
            o = O.row(lg[r], beta, alpha_t, float(u[r]), force=int(tok[r]))
        assert abs(o["log_omega"] - loginc[r]) <= TOL_LOGINC, (r, o["log_omega"], loginc[r])
        assert abs(o["logp_y"] - logp[r]) <= TOL_LOGINC
    return flagged


def make_pair(cfg: W.Workload, seed: int, G: int = None, T_max: int = None, ramp: int = None, kappa: float = None,
              resampler: int = 0, top_k: int = 0, top_p: float = 0.0):
    G = cfg.G if G is None else G
    T_max = cfg.T if T_max is None else T_max
    ramp = cfg.ramp if ramp is None else ramp
    kappa = cfg.kappa if kappa is None else kappa
    wl = WC.DeviceWorkload(cfg, seed, G=G)
    ps = B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, kappa, ramp, seed, cfg.eos_id, G=G, T_max=T_max,
                prompt_len=wl.prompt_len)
    orc = O.Oracle(cfg.N, cfg.V, float(np.float32(cfg.alpha)), float(np.float32(cfg.tau)), float(np.float32(kappa)),
                   ramp, seed, cfg.eos_id, G=G, T_max=T_max, prompt_len=wl.prompt_len)
    ps.set_resampler(resampler)
    orc.set_resampler(resampler)
    if top_k or top_p:
        ps.set_proposal_mask(top_k, top_p)
        orc.set_proposal_mask(top_k, top_p)
    return wl, ps, orc


def compare_step(ps: B.Psmc, orc: O.Oracle, lg_host: np.ndarray, st: LoopStats, kappa: float, masked: bool = False):
    """Feed the oracle the same block (adopting flagged CUDA choices) and compare everything."""
    N, G = ps.N, ps.G
    g_tok, g_res, g_anc = ps.tokens.numpy(), ps.resampled.numpy(), ps.ancestors.numpy()
    done_before = orc.done.astype(bool)
    g_k = ps.mask_sizes.numpy() if masked else None
    orc.step(lg_host, force_tok=g_tok, force_resample=g_res, force_anc=g_anc, force_k=g_k)
    assert ps.sync_status() == B.OK
    if masked:  # size of the proposal's support: equal, or (nucleus) the imposed size misses the rule by a rounding error
        k_own, k_mg = orc.k_own, orc.k_margin
        for r in np.nonzero((k_own != g_k) & ~done_before)[0]:
            assert k_mg[r] <= K_MARGIN, "row %d: support %d vs oracle %d, margin %.3e" % (r, g_k[r], k_own[r], k_mg[r])
            st.k_adopted += 1

    # tokens: equal, or the oracle's own draw sat within TOK_MARGIN of a CDF boundary
    own, mg = orc.tokens_own, orc.tok_margin
    diff = np.nonzero(own != g_tok)[0]
    for r in diff:
        assert mg[r] <= TOK_MARGIN, "row %d: token %d vs oracle %d, margin %.3e" % (r, g_tok[r], own[r], mg[r])
    st.tok_adopted += len(diff)
    live = ~done_before
    if live.any():
        st.min_tok_margin = min(st.min_tok_margin, float(mg[live].min()))
    st.live_rows += int(live.sum())

    # log omega and log p of the adopted token
    e = np.abs(ps.log_inc.numpy() - orc.log_inc).max()
    st.max_loginc_err = max(st.max_loginc_err, float(e))
    assert e <= TOL_LOGINC, "log omega differs by %.3e" % e
    assert np.abs(ps.logp_tok.numpy() - orc.logp_tok).max() <= TOL_LOGINC

    # trigger
    r_own, ess_o = orc.resampled_own, orc.ess
    for g in np.nonzero(r_own != g_res)[0]:
        assert abs(ess_o[g] - kappa * N) <= ESS_MARGIN * N, "group %d: trigger differs, ESS %.6f" % (g, ess_o[g])
        st.ess_adopted += 1
    assert np.abs(ps.ess.numpy() - ess_o).max() <= 1e-6 * N

    # ancestors (groups that resampled)
    a_own, a_mg = orc.anc_own.reshape(G, N), orc.anc_margin
    ga = g_anc.reshape(G, N)
    for g in np.nonzero(g_res)[0]:
        if r_own[g] and not np.array_equal(a_own[g], ga[g]):
            assert a_mg[g] <= ANC_MARGIN, "group %d: ancestors differ, margin %.3e" % (g, a_mg[g])
            st.anc_adopted += 1
    st.resample_events += int(g_res.sum())

    # state after the step: exact for integers, tolerance for log-weights
    m = ps.slot_map.numpy()
    assert np.array_equal(m, orc.slot_map)
    st.slots_moved += int((m.reshape(G, N) != np.arange(N)[None]).sum())
    assert np.array_equal(ps.done.numpy(), orc.done)
    assert np.array_equal(ps.lens.numpy(), orc.lens)
    assert np.array_equal(ps.last_tokens.numpy(), orc.last_tokens)
    assert ps.move_count == int((m.reshape(G, N) != np.arange(N)[None]).sum())
    e = np.abs(ps.log_weights.numpy() - orc.log_weights).max()
    st.max_logw_err = max(st.max_logw_err, float(e))
    assert e <= TOL_LOGW, "log W differs by %.3e at step %d" % (e, orc.t)
    e = np.abs(ps.cum_logp.numpy() - orc.cum_logp).max()
    st.max_s_err = max(st.max_s_err, float(e))
    assert e <= TOL_LOGW, "S differs by %.3e at step %d" % (e, orc.t)
    assert np.abs(ps.log_z.numpy() - orc.log_z).max() <= TOL_LOGW * max(1, orc.t)
    st.steps += 1


def closed_loop(cfg: W.Workload, seed: int, T: int, G: int = None, ramp: int = None, kappa: float = None,
                kv_shape=None, logit_bias_fn=None, resampler: int = 0, skip_shared_prompt: bool = False,
                top_k: int = 0, top_p: float = 0.0) -> LoopStats:
    """Run T tokens on both sides.  kv_shape=(layers, heads, max_len, dim) also carries a KV cache
    through every reindex on both sides and compares the whole buffers at the end."""
    wl, ps, orc = make_pair(cfg, seed, G=G, T_max=T, ramp=ramp, kappa=kappa, resampler=resampler, top_k=top_k,
                            top_p=top_p)
    kappa_f = float(np.float32(cfg.kappa if kappa is None else kappa))
    st = LoopStats()
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    kv = None
    if kv_shape is not None:
        L, H, ML, D = kv_shape
        tdt = wl.tdtype
        ks = [torch.empty((wl.R, H, ML, D), dtype=tdt, device="cuda") for _ in range(L)]
        vs = [torch.empty((wl.R, H, ML, D), dtype=tdt, device="cuda") for _ in range(L)]
        for l in range(L):
            WC.fill_kv(ks[l], seed, l, 0)
            WC.fill_kv(vs[l], seed, l, 1)
        copy_from = None
        if skip_shared_prompt:  # a group's rows were prefilled with one prompt: the same keys and values below its length
            for g in range(ps.G):
                pl = int(wl.prompt_len[g])
                for t_ in ks + vs:
                    t_[g * ps.N:(g + 1) * ps.N, :, :pl, :] = t_[g * ps.N, :, :pl, :].clone()
            copy_from = np.repeat(wl.prompt_len, ps.N).astype(np.int32)
        desc = ps.make_kv_desc(ks, vs, skip_shared_prompt=skip_shared_prompt)
        as_np = lambda t: (t.view(torch.int16) if t.dtype == torch.bfloat16 else t).cpu().numpy()
        kv = dict(desc=desc, ks=ks, vs=vs, host=[as_np(t).copy() for t in ks + vs], as_np=as_np, copy_from=copy_from)
        if skip_shared_prompt:  # second mirror moved in full: with shared prompts both forms give the same cache
            kv["host_full"] = [h.copy() for h in kv["host"]]
    last_view = ps.device_view("psmc_last_tokens", ps.R)
    for t in range(1, T + 1):
        wl.fill(lg, t, prev)
        if logit_bias_fn is not None:
            logit_bias_fn(t, lg)
        ps.step(lg)
        if kv is not None:
            ps.reindex_kv(kv["desc"])
        compare_step(ps, orc, logits_to_numpy(lg), st, kappa_f, masked=bool(top_k or top_p))
        if kv is not None:
            m = orc.slot_map.reshape(ps.G, ps.N) + (np.arange(ps.G) * ps.N)[:, None]
            idx, ln = m.reshape(-1).astype(np.int32), orc.lens
            for h in kv["host"]:
                O.reindex_tensor(h, h, idx, ln, kv["copy_from"])
            for h in kv.get("host_full", []):
                O.reindex_tensor(h, h, idx, ln)
        prev.copy_(last_view)
    if kv is not None:
        for dev, host in zip(kv["ks"] + kv["vs"], kv["host"]):
            assert np.array_equal(kv["as_np"](dev), host), "KV cache differs after the reindexes"
        for full, host in zip(kv.get("host_full", []), kv["host"]):
            assert np.array_equal(full, host), "leaving the shared prompt in place changed the cache"
    # final draw and back-trace
    toks, ln, ix = ps.select()
    o_toks, o_ln, o_ix = orc.select()
    assert np.array_equal(ix.cpu().numpy(), o_ix)
    assert np.array_equal(ln.cpu().numpy(), o_ln)
    assert np.array_equal(toks.cpu().numpy(), o_toks)
    assert ps.sync_status() == B.OK
    ps.destroy()
    return st
