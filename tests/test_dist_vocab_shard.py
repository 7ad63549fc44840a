"""Host side of the step on a vocabulary-sharded LM head: how the columns are cut, and the two all-gathers.

The kernels cannot run here, so two `gloo` ranks drive `VocabShardedStep` with a stand-in for the library calls that
follows the C header's contract in numpy (triples -> owner -> pick -> Eq. 7).  What comes out is compared with the
oracle's row function on the WHOLE row: that the exchange carries the right numbers in the right order, and that
24 + 8 bytes per row and rank are enough to reproduce the unsharded draw and weight.
"""
import json
import math
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2602_10273_b200 import vocab_shard as VS  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


@pytest.mark.parametrize("V,world,align", [(1024, 1, 8), (1024, 3, 8), (32000, 8, 8), (151936, 3, 8), (128256, 8, 8),
                                           (1027, 4, 8), (20, 4, 8), (9, 4, 8), (151936, 64, 4)])
def test_vocab_shards_tile_the_vocabulary(V, world, align):
    cuts = VS.vocab_shards(V, world, align)
    assert len(cuts) == world and cuts[0][0] == 0 and cuts[-1][0] + cuts[-1][1] == V
    assert all(a[0] + a[1] == b[0] for a, b in zip(cuts, cuts[1:])) and all(n >= 2 for _, n in cuts)
    if V // align >= world:
        assert all(v0 % align == 0 for v0, _ in cuts)
        assert max(n for _, n in cuts[:-1] or cuts) - min(n for _, n in cuts) <= align


def test_vocab_shards_refuses_too_many_ranks():
    with pytest.raises(ValueError):
        VS.vocab_shards(7, 4)


class _NumpyRank:
    """Stand-in for binding.Psmc's three shard calls, in plain fp64 numpy, one step only."""

    def __init__(self, R, N, beta, alpha_t, uniforms):
        self.R, self.N, self.beta, self.alpha_t, self.U = R, N, beta, alpha_t, uniforms
        self.calls = []

    def shard_sweep(self, logits_local, triples_out, stream=None):
        self.calls.append("sweep")
        self.x = logits_local.numpy().astype(np.float64) * math.log2(math.e)
        C = np.ceil(self.x.max(axis=1))
        triples_out[:, 0] = torch.from_numpy(C)
        triples_out[:, 1] = torch.from_numpy(np.exp2(self.x - C[:, None]).sum(axis=1))
        triples_out[:, 2] = torch.from_numpy(np.exp2(self.beta * (self.x - C[:, None])).sum(axis=1))
        self.logits = logits_local.numpy()

    def _totals(self, all_triples):
        a = all_triples.numpy()
        C = a[:, :, 0].max(axis=0)
        f1 = np.exp2(a[:, :, 0] - C[None])
        fb = np.exp2(self.beta * (a[:, :, 0] - C[None]))
        b = a[:, :, 2] * fb                                            # [P, R] masses in the row's scale
        return C, (a[:, :, 1] * f1).sum(axis=0), b.sum(axis=0), b

    def shard_locate(self, v0, all_triples, rank, picks_out, stream=None):
        self.calls.append("locate")
        C, S1, Sb, b = self._totals(all_triples)
        incl = np.cumsum(b, axis=0)
        picks_out[:, 0] = -1
        picks_out[:, 1] = 0
        for r in range(self.R):
            target = self.U[r] * Sb[r]
            owner = int(np.argmax(incl[:, r] >= target)) if (incl[:, r] >= target).any() else b.shape[0] - 1
            if owner != rank:
                continue
            base = incl[owner, r] - b[owner, r]
            run = base + np.cumsum(np.exp2(self.beta * (self.x[r] - C[r])))
            y = int(np.argmax(run >= target)) if (run >= target).any() else self.x.shape[1] - 1
            picks_out[r, 0] = v0 + y
            picks_out[r, 1] = int(np.float32(self.logits[r, y]).view(np.int32))

    def shard_finish(self, all_triples, all_picks, stream=None):
        self.calls.append("finish")
        C, S1, Sb, _ = self._totals(all_triples)
        pk = all_picks.numpy()
        self.tok = pk[:, :, 0].max(axis=0)
        who = pk[:, :, 0].argmax(axis=0)
        logit = pk[who, np.arange(self.R), 1].astype(np.int32).view(np.float32).astype(np.float64)
        dl = logit - C * math.log(2.0)
        self.logp = dl - np.log(S1)
        self.loginc = (self.alpha_t - self.beta) * dl - self.alpha_t * np.log(S1) + np.log(Sb)


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from oracle import oracle as O
    from paper_2602_10273_b200.workload import gen

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg, seed, G, t = gen.CONFIGS["tiny"], 4, 3, 1
        R = G * cfg.N
        bias = gen.vocab_bias(seed, cfg.V, cfg.slope)
        plen = gen.prompt_lengths(seed, G, cfg.prompt_lo, cfg.prompt_hi)
        prev = np.repeat(gen.prompt_last_token(seed, G, plen, cfg.V), cfg.N)
        block = gen.logits_block(seed, t, np.repeat(np.arange(G), cfg.N), prev, cfg.V, cfg.scale, bias, cfg.dtype)
        block = np.asarray(block, dtype=np.float32)                      # every rank builds the same [R, V] block ...
        v0, vl = VS.vocab_shards(cfg.V, world)[rank]
        mine = torch.from_numpy(block[:, v0:v0 + vl].copy())             # ... and keeps only its columns
        alpha_t = O.alpha_at(cfg.alpha, 0, t)
        beta = O.beta_at(cfg.alpha, cfg.tau, 0, t)
        U = np.array([O.uniform(O.hash5(seed, 1, r // cfg.N, t, r % cfg.N)) for r in range(R)])
        ps = _NumpyRank(R, cfg.N, beta, alpha_t, U)
        VS.VocabShardedStep(ps, v0, VS.TorchDistExchange(), device="cpu").step(mine)
        want = [O.row(block[r], beta, alpha_t, U[r]) for r in range(R)]
        json.dump({"calls": ps.calls, "tok": ps.tok.tolist(), "loginc": ps.loginc.tolist(), "logp": ps.logp.tolist(),
                   "want_tok": [w["y"] for w in want], "want_loginc": [w["log_omega"] for w in want],
                   "want_logp": [w["logp_y"] for w in want], "margin": [w["margin"] for w in want]},
                  open(os.path.join(out_dir, "r%d.json" % rank), "w"))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_gloo_ranks_reproduce_the_unsharded_row(tmp_path, world):
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / ("r%d.json" % r))) for r in range(world)]
    for r in res:
        assert r["calls"] == ["sweep", "locate", "finish"]
        assert r["tok"] == res[0]["tok"] and r["loginc"] == res[0]["loginc"]          # replicated, bit for bit
        for y, w, m in zip(r["tok"], r["want_tok"], r["margin"]):
            assert y == w or m < 1e-9
        assert np.abs(np.array(r["loginc"]) - np.array(r["want_loginc"])).max() < 1e-9
        assert np.abs(np.array(r["logp"]) - np.array(r["want_logp"])).max() < 1e-9
    assert len(set(res[0]["tok"])) > 1
