"""The step with the vocabulary split over P ranks, against the oracle's step over the whole rows.

One GPU stands in for P ranks: P contexts take the three calls in lock step and the two all-gathers are a
torch.stack.  (The calls of different "ranks" never wait on one another on the device: the exchange is on the host
side of the launches, so running them one after the other is the same computation.)  Rank 0's context is compared
with the oracle as in every other closed loop; the other ranks' replicated state must equal rank 0's bit for bit.
"""
import numpy as np
import pytest
import torch

import parity as P
from paper_2602_10273_b200 import binding as B
from paper_2602_10273_b200 import vocab_shard as VS
from paper_2602_10273_b200.workload import gen as W

pytestmark = pytest.mark.gpu

VIEWS = ("tokens", "last_tokens", "log_weights", "log_inc", "logp_tok", "cum_logp", "ancestors", "slot_map",
         "resampled", "ess", "log_z", "lens", "done")


def _clone_ctx(ps0, cfg, wl, seed, T, ramp, kappa, resampler):
    ps = B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, kappa, ramp, seed, cfg.eos_id, G=ps0.G, T_max=T,
                prompt_len=wl.prompt_len)
    ps.set_resampler(resampler)
    return ps


def sharded_loop(cfg, seed, T, shards, G=None, ramp=None, kappa=None, resampler=0, logit_edit=None):
    wl, ps0, orc = P.make_pair(cfg, seed, G=G, T_max=T, ramp=ramp, kappa=kappa, resampler=resampler)
    kap = cfg.kappa if kappa is None else kappa
    rmp = cfg.ramp if ramp is None else ramp
    ranks = [ps0] + [_clone_ctx(ps0, cfg, wl, seed, T, rmp, kap, resampler) for _ in shards[1:]]
    n = len(shards)
    R = ps0.R
    triples = [torch.empty((R, 3), dtype=torch.float64, device="cuda") for _ in ranks]
    picks = [torch.empty((R, 2), dtype=torch.int32, device="cuda") for _ in ranks]
    st = P.LoopStats()
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    last_view = ps0.device_view("psmc_last_tokens", R)
    owners = np.zeros(n, dtype=np.int64)
    for t in range(1, T + 1):
        wl.fill(lg, t, prev)
        if logit_edit is not None:
            logit_edit(t, lg)
        for p, (v0, vl) in enumerate(shards):
            ranks[p].shard_sweep(lg[:, v0:v0 + vl], triples[p])
        all_tr = torch.stack(triples)
        for p, (v0, vl) in enumerate(shards):
            ranks[p].shard_locate(v0, all_tr, p, picks[p])
        all_pk = torch.stack(picks)
        for p in range(n):
            ranks[p].shard_finish(all_tr, all_pk)
        # exactly one rank names each live row's token, and the token lies in that rank's columns
        pk = all_pk[:, :, 0].cpu().numpy()
        live = ps0.tokens.numpy() >= 0
        was_live = orc.done == 0
        named = (pk >= 0).sum(axis=0)
        assert np.array_equal(named[was_live], np.ones(int(was_live.sum()), dtype=named.dtype))
        assert (named[~was_live] == 0).all() and live.all()
        for p, (v0, vl) in enumerate(shards):
            mine = pk[p][pk[p] >= 0]
            assert ((mine >= v0) & (mine < v0 + vl)).all()
            owners[p] += len(mine)
        P.compare_step(ps0, orc, P.logits_to_numpy(lg), st, float(np.float32(kap)))
        for p in range(1, n):
            for name in VIEWS:
                a, b = getattr(ps0, name).numpy(), getattr(ranks[p], name).numpy()
                assert np.array_equal(a, b, equal_nan=True), "rank %d: %s differs from rank 0 at step %d" % (p, name, t)
            assert ranks[p].move_count == ps0.move_count and ranks[p].sync_status() == B.OK
        prev.copy_(last_view)
    toks, ln, ix = ps0.select()
    o_toks, o_ln, o_ix = orc.select()
    assert np.array_equal(ix.cpu().numpy(), o_ix) and np.array_equal(ln.cpu().numpy(), o_ln)
    assert np.array_equal(toks.cpu().numpy(), o_toks)
    for ps in ranks:
        ps.destroy()
    return st, owners


@pytest.mark.parametrize("world", [1, 2, 3, 4])
def test_sharded_step_small_vocabulary(world):
    cfg = W.CONFIGS["tiny"]
    st, owners = sharded_loop(cfg, 5, 48, VS.vocab_shards(cfg.V, world))
    assert st.resample_events > 0 and (owners > 0).all()


def test_sharded_step_more_ranks_than_lanes():
    """40 ranks: the row totals are then formed by walking the gathered triples in global memory instead of handing
    one rank's triple to each lane of a warp."""
    cfg = W.CONFIGS["tiny"]
    st, owners = sharded_loop(cfg, 8, 12, VS.vocab_shards(cfg.V, 40))
    assert st.steps == 12 and owners.sum() == st.live_rows


def test_sharded_step_uneven_unaligned_shards():
    """Shards that start off the 16-byte grid (scalar load path) and differ widely in size."""
    cfg = W.CONFIGS["tiny"]                       # V = 1024, fp32
    shards = [(0, 3), (3, 510), (513, 2), (515, 509)]
    st, owners = sharded_loop(cfg, 7, 40, shards)
    assert st.resample_events > 0 and owners[1] > 0 and owners[3] > 0


@pytest.mark.parametrize("name,world,T,G", [("llama2_7b", 2, 24, None), ("llama2_7b", 8, 16, 3), ("qwen25_7b", 4, 12, None),
                                            ("batched_prompts", 8, 6, 4), ("resample_stress", 8, 6, None)])
def test_sharded_step_model_vocabularies(name, world, T, G):
    cfg = W.CONFIGS[name]
    st, owners = sharded_loop(cfg, 11, T, VS.vocab_shards(cfg.V, world), G=G)
    assert st.steps == T and owners.sum() == st.live_rows


def test_sharded_step_batched_prompts_full_size():
    """All 64 prompts x 8 particles, the vocabulary of 128256 over 8 ranks: every row of rank 0 against the oracle's
    whole-row step, every other rank bit-equal to rank 0."""
    cfg = W.CONFIGS["batched_prompts"]
    st, owners = sharded_loop(cfg, 1, 3, VS.vocab_shards(cfg.V, 8))
    assert st.live_rows == 3 * 512 and (owners > 0).all()


def test_sharded_step_three_ranks_need_more_span_triples_than_the_whole_row():
    """480 rows of 128256 logits are cut into 32 spans of 4096; a third of such a row is cut into 42 spans of 1024,
    so the context has to grow the scratch it sized for whole rows."""
    cfg = W.CONFIGS["batched_prompts"]
    G = 60
    assert B.logits_pass_scratch_bytes(G * cfg.N, VS.vocab_shards(cfg.V, 3)[0][1]) > B.logits_pass_scratch_bytes(G * cfg.N, cfg.V)
    st, owners = sharded_loop(cfg, 3, 4, VS.vocab_shards(cfg.V, 3), G=G)
    assert st.steps == 4 and (owners > 0).all()


@pytest.mark.parametrize("resampler", [B.STRATIFIED, B.RESIDUAL])
def test_sharded_step_other_resamplers_and_ramp(resampler):
    cfg = W.CONFIGS["tiny"]
    st, _ = sharded_loop(cfg, 9, 40, VS.vocab_shards(cfg.V, 2), ramp=16, kappa=0.8, resampler=resampler)
    assert st.resample_events > 0


def test_a_rank_whose_columns_are_all_masked():
    cfg = W.CONFIGS["tiny"]
    shards = VS.vocab_shards(cfg.V, 4)
    v0, vl = shards[2]

    def mask(t, lg):
        lg[:, v0:v0 + vl] = float("-inf")
        if t % 3 == 0:                            # and sometimes the first rank too: rank 1 then owns the smallest U
            lg[:, :shards[0][1]] = float("-inf")

    st, owners = sharded_loop(cfg, 13, 30, shards, logit_edit=mask)
    assert owners[2] == 0 and owners[1] > 0 and owners[3] > 0


def test_one_hot_rows_across_ranks():
    """All mass on one token of the last rank: every row's owner is that rank whatever U is."""
    cfg = W.CONFIGS["tiny"]
    shards = VS.vocab_shards(cfg.V, 4)
    hot = cfg.V - 5

    def edit(t, lg):
        lg.fill_(float("-inf"))
        lg[:, hot] = 3.0

    st, owners = sharded_loop(cfg, 2, 6, shards, logit_edit=edit)
    assert owners[3] == st.live_rows and owners[:3].sum() == 0


def test_call_order_is_enforced():
    cfg = W.CONFIGS["tiny"]
    wl, ps, orc = P.make_pair(cfg, 1, T_max=4)
    lg = wl.new_logits()
    wl.fill(lg, 1, wl.first_prev.clone())
    tr = torch.empty((ps.R, 3), dtype=torch.float64, device="cuda")
    pk = torch.empty((ps.R, 2), dtype=torch.int32, device="cuda")
    with pytest.raises(B.PsmcError) as e:
        ps.shard_locate(0, tr.unsqueeze(0).contiguous(), 0, pk)
    assert e.value.code == B.E_STATE
    ps.shard_sweep(lg, tr)
    with pytest.raises(B.PsmcError) as e:
        ps.step(lg)                               # a sharded step is under way
    assert e.value.code == B.E_STATE
    with pytest.raises(B.PsmcError) as e:
        ps.shard_finish(tr.unsqueeze(0).contiguous(), pk.unsqueeze(0).contiguous())
    assert e.value.code == B.E_STATE
    all_tr = tr.unsqueeze(0).contiguous()
    ps.shard_locate(0, all_tr, 0, pk)
    ps.shard_finish(all_tr, pk.unsqueeze(0).contiguous())
    assert ps.step_index == 1 and ps.sync_status() == B.OK
    # one rank holding every column is the unsharded step
    orc.step(P.logits_to_numpy(lg))
    assert np.array_equal(ps.tokens.numpy(), orc.tokens_own)
    ps.destroy()
