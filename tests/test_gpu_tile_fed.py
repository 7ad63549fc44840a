"""The step fed one vocabulary tile at a time (psmc_tiles_feed / _need / _finish), against the oracle's step over the
whole rows: the tiles are slices of the full logit block handed over in order, the tiles asked for again are gathered
from the same block, and everything the step leaves behind is compared as in every other closed loop."""
import numpy as np
import pytest
import torch

import parity as P
from paper_2602_10273_b200 import binding as B
from paper_2602_10273_b200.workload import gen as W

pytestmark = pytest.mark.gpu


def tile_fed_loop(cfg, seed, T, width, G=None, ramp=None, kappa=None, resampler=0, logit_edit=None):
    wl, ps, orc = P.make_pair(cfg, seed, G=G, T_max=T, ramp=ramp, kappa=kappa, resampler=resampler)
    kap = float(np.float32(cfg.kappa if kappa is None else kappa))
    R, V = ps.R, cfg.V
    st = P.LoopStats()
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    last = ps.device_view("psmc_last_tokens", R)
    need = torch.empty(R, dtype=torch.int32, device="cuda")
    cols = torch.arange(width, device="cuda")[None, :]
    for t in range(1, T + 1):
        wl.fill(lg, t, prev)
        if logit_edit is not None:
            logit_edit(t, lg)
        for v0 in range(0, V, width):
            ps.tiles_feed(lg[:, v0:min(V, v0 + width)].clone(), v0)      # a tile is a buffer of its own
        ps.tiles_need(need)
        first = need.long().clamp(min=0)[:, None]
        idx = first + cols                                               # [R, width] columns of each row's tile
        row_tiles = torch.gather(lg, 1, idx.clamp(max=V - 1))
        row_tiles = torch.where(idx < V, row_tiles, torch.full_like(row_tiles, float("-inf")))
        ps.tiles_finish(row_tiles)
        live = orc.done == 0
        n = need.cpu().numpy()
        assert (n[live] >= 0).all() and (n[live] % width == 0).all() and (n[~live] == -1).all()
        P.compare_step(ps, orc, P.logits_to_numpy(lg), st, kap)
        tok = ps.tokens.numpy()
        assert ((tok[live] >= n[live]) & (tok[live] < n[live] + width)).all()   # the token lies in the tile asked for
        prev.copy_(last)
    toks, ln, ix = ps.select()
    o_toks, o_ln, o_ix = orc.select()
    assert np.array_equal(ix.cpu().numpy(), o_ix) and np.array_equal(toks.cpu().numpy(), o_toks)
    assert ps.sync_status() == B.OK
    ps.destroy()
    return st


@pytest.mark.parametrize("name,G,T,width", [("tiny", None, 40, 256), ("tiny", None, 24, 1000), ("llama2_7b", None, 24, 4096),
                                            ("batched_prompts", 6, 12, 16384), ("qwen25_7b", None, 20, 8192)])
def test_tile_fed_step_matches_the_whole_row_step(name, G, T, width):
    c = W.CONFIGS[name]
    st = tile_fed_loop(c, seed=3, T=T, width=width, G=G)
    assert st.steps == T


def test_tile_fed_step_with_ramp_other_resampler_and_odd_tiles():
    c = W.Workload("odd", 3, 5, 3001, "f32", 3.0, 1.5, 20, 4, 9, 4.0, 0.25, 0.9, 6, 1, 2, 16, 40)
    st = tile_fed_loop(c, seed=9, T=20, width=777, resampler=B.RESIDUAL)          # 3001 = 3 * 777 + 670
    assert st.resample_events > 0

    def one_hot(t, lg):
        if t == 3:
            lg[2] = float("-inf")
            lg[2, 1234] = 0.0                                                       # all mass in the second tile

    tile_fed_loop(c, seed=10, T=8, width=777, logit_edit=one_hot)


def test_tile_fed_calls_out_of_order_are_refused():
    c = W.CONFIGS["tiny"]
    wl, ps, orc = P.make_pair(c, 1, T_max=4)
    lg = wl.new_logits()
    wl.fill(lg, 1, wl.first_prev)
    need = torch.empty(ps.R, dtype=torch.int32, device="cuda")
    h = ps._h
    L = B.lib()
    s = torch.cuda.current_stream().cuda_stream
    t0 = lg[:, :256].clone()
    assert L.psmc_tiles_need(h, need.data_ptr(), s) == B.E_STATE               # nothing fed
    assert L.psmc_tiles_feed(h, t0.data_ptr(), B.F32, 256, 256, 256, s) == B.E_STATE   # the first tile starts at 0
    assert L.psmc_tiles_feed(h, t0.data_ptr(), B.F32, 256, 0, 256, s) == B.OK
    assert L.psmc_tiles_feed(h, t0.data_ptr(), B.F32, 256, 512, 256, s) == B.E_STATE   # a gap
    assert L.psmc_tiles_need(h, need.data_ptr(), s) == B.E_STATE               # the vocabulary is not covered yet
    assert L.psmc_step(h, lg.data_ptr(), B.F32, c.V, s) == B.E_STATE           # a tile-fed step is under way
    assert L.psmc_tiles_finish(h, t0.data_ptr(), B.F32, 256, s) == B.E_STATE
    assert L.psmc_tiles_feed(h, t0.data_ptr(), B.F32, 256, 256, 128, s) == B.E_INVAL   # a narrow tile that is not the last
    ps.reset(1)                                                                  # abandons the step
    ps.step(lg)
    assert ps.sync_status() == B.OK
    ps.destroy()
