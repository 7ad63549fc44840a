"""Paged KV cache with copy-on-write resampling, against the oracle's dense cache.

The oracle keeps one dense cache row per slot and moves whole live prefixes (Appendix C as written).  The CUDA
path keeps blocks and a block table; read through the table it must hold the same keys and values at every live
position, after every step, and its bookkeeping (reference counts, free list, private last blocks) must add up.
"""
import numpy as np
import pytest
import torch

import parity as P
from oracle import oracle as O
from paper_2602_10273_b200 import binding as B
from paper_2602_10273_b200.workload import cuda as WC
from paper_2602_10273_b200.workload import gen as W

pytestmark = pytest.mark.gpu


def _gather_dense(pool, table, lens, block_len):
    """pool [n_blocks, H, block_len, D], table [R, MB] -> list of per-row arrays [H, len, D] read through the table."""
    out = []
    for r in range(table.shape[0]):
        n = int(lens[r])
        pos = torch.arange(n, device=pool.device)
        blk = table[r, pos // block_len].long()
        assert (blk >= 0).all(), "row %d: a live position has no block" % r
        out.append(pool[blk, :, pos % block_len, :].permute(1, 0, 2))  # [H, n, D]
    return out


def _check_bookkeeping(ps, n_blocks, block_len, prepared=False):
    """prepared: the rows already hold the block of their next position (after a reindex that is not the last)."""
    table = ps.kv_paged_table.cpu().numpy()
    refc = ps.kv_paged_refcount.cpu().numpy()
    lens = ps.lens.numpy()
    done = ps.done.numpy()
    used = table[table >= 0]
    assert np.array_equal(np.bincount(used, minlength=n_blocks), refc), "reference counts do not match the table"
    assert ps.kv_paged_free_count + int((refc > 0).sum()) == n_blocks, "blocks leaked or freed twice"
    for r in range(table.shape[0]):
        nb = -(-int(lens[r]) // block_len)
        if prepared and lens[r] % block_len == 0 and not done[r]:
            nb += 1                                                  # an empty block waits for the next position
        assert (table[r, :nb] >= 0).all() and (table[r, nb:] == -1).all(), "row %d holds the wrong number of blocks" % r
        if lens[r] % block_len or (prepared and not done[r]):
            assert refc[table[r, nb - 1]] == 1, "row %d shares its partly filled block" % r


@pytest.mark.parametrize("name,G,T,block_len,share,every", [("tiny", None, 56, 16, True, True), ("tiny", None, 40, 8, False, False),
                                                            ("tiny", None, 56, 16, True, False),
                                                            ("batched_prompts", 6, 24, 16, True, False)])
def test_paged_cache_holds_what_the_dense_reorder_holds(name, G, T, block_len, share, every):
    """every: psmc_kv_paged_append before every token (harmless), else only before the first: the reindex prepares
    the blocks of the token that follows it."""
    _paged_loop(W.CONFIGS[name], G, T, block_len, share, every, check_every=8)


@pytest.mark.parametrize("block_len,share", [(8, True), (16, False)])
def test_paged_cache_over_six_hundred_tokens(block_len, share):
    """Blocks are handed out, shared, copied on write and given back at every resampling step: a leak or a count that
    is off by one shows only after many of them.  Two groups of 16 particles, kappa = 0.9, prompts of 5 to 19
    positions, 600 tokens (75 blocks of 8 per row)."""
    c = W.Workload("paged_long", 2, 16, 2048, "f32", 3.0, 1.5, 600, 5, 19, 4.0, 0.25, 0.9, 0, 1, 2, 8, 640)
    st = _paged_loop(c, None, c.T, block_len, share, False, check_every=50)
    assert st.resample_events > 200


def _paged_loop(c, G, T, block_len, share, every, check_every):
    wl, ps, orc = P.make_pair(c, seed=3, G=G, T_max=T)
    R, N, H, D, L = wl.R, c.N, 2, c.head_dim, 2
    ML = c.prompt_hi + T + 8
    # what slot r writes at position p, layer by layer (hashed N(0,1)); prompts are the same within a group
    init = []
    for l in range(L):
        for which in (0, 1):
            t = torch.empty((R, H, ML, D), dtype=wl.tdtype, device="cuda")
            WC.fill_kv(t, 3, l, which)
            for g in range(ps.G):
                pl = int(wl.prompt_len[g])
                t[g * N:(g + 1) * N, :, :pl, :] = t[g * N, :, :pl, :].clone()
            init.append(t)
    as_np = lambda t: (t.view(torch.int16) if t.dtype == torch.bfloat16 else t).cpu().numpy()
    mirror = [as_np(t).copy() for t in init]                      # the oracle's dense caches

    MB = -(-ML // block_len)
    n_blocks = R * MB
    ps.kv_paged_create(n_blocks, block_len, MB, share_prompt=share)
    pools = [torch.zeros((n_blocks, H, block_len, D), dtype=wl.tdtype, device="cuda") for _ in init]
    desc = ps.make_kv_pools(pools[0::2], pools[1::2])
    table = ps.kv_paged_table                                      # device view, follows the library's updates

    def write_positions(rows, pos):                                # the language model's cache writes
        rows_t = torch.as_tensor(rows, device="cuda", dtype=torch.long)
        pos_t = torch.as_tensor(pos, device="cuda", dtype=torch.long)
        blk = table[rows_t, pos_t // block_len].long()
        assert (blk >= 0).all()
        for pool, src in zip(pools, init):
            pool[blk, :, pos_t % block_len, :] = src[rows_t, :, pos_t, :]

    for g in range(ps.G):                                          # prefill
        pl = int(wl.prompt_len[g])
        for i in range(N):
            write_positions([g * N + i] * pl, list(range(pl)))
    _check_bookkeeping(ps, n_blocks, block_len)
    if share and block_len <= c.prompt_lo:                         # full prompt blocks are shared by the group
        assert int(ps.kv_paged_refcount.max()) == N

    st = P.LoopStats()
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    last_view = ps.device_view("psmc_last_tokens", R)
    kappa_f = float(np.float32(c.kappa))
    for t in range(1, T + 1):
        if every or t == 1:
            ps.kv_paged_append()
        lens, done = ps.lens.numpy(), ps.done.numpy()
        live = np.nonzero(done == 0)[0]
        write_positions(live.tolist(), lens[live].tolist())        # position len[r] of every live row
        wl.fill(lg, t, prev)
        ps.step(lg)
        ps.reindex_kv_paged(desc)
        P.compare_step(ps, orc, P.logits_to_numpy(lg), st, kappa_f)
        m = orc.slot_map.reshape(ps.G, N) + (np.arange(ps.G) * N)[:, None]
        for h in mirror:
            O.reindex_tensor(h, h, m.reshape(-1).astype(np.int32), orc.lens)
        prev.copy_(last_view)
        if t % check_every == 0 or t == T:
            assert ps.sync_status() == B.OK
            _check_bookkeeping(ps, n_blocks, block_len, prepared=t < T)
            lens = ps.lens.numpy()
            for pool, host in zip(pools, mirror):
                rows = _gather_dense(pool, table, lens, block_len)
                for r in range(R):
                    assert np.array_equal(as_np(rows[r]), host[r, :, :lens[r], :]), "row %d differs at step %d" % (r, t)
    assert st.resample_events > 0 and st.slots_moved > 0
    ps.destroy()
    return st


def test_paged_cache_reports_an_empty_free_list():
    c = W.CONFIGS["tiny"]
    wl, ps, orc = P.make_pair(c, seed=1, T_max=8)
    MB = -(-(c.prompt_hi + 16) // 16)
    ps.kv_paged_create(4 * (c.prompt_hi // 16), 16, MB, share_prompt=False)   # exactly the prompts' blocks, none to spare
    assert ps.sync_status() == B.OK and ps.kv_paged_free_count == 0
    ps.kv_paged_append()                                             # every row needs a block now
    assert ps.sync_status() == B.E_NOMEM
    ps.destroy()
