"""The multi-GPU form of the path is "independent replicas": one process per GPU, prompts sharded, no data-path
collective.  What the ranks do share is the bookkeeping of a measurement.  These tests run that host logic as
two `gloo` ranks on CPU, and check the rank gating of the benchmark's reference arm.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    from oracle import oracle as O
    from paper_2602_10273_b200 import replicas
    from paper_2602_10273_b200.workload import gen

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        G = 2
        plan = replicas.rank_plan(G, base_seed=1)
        cfg = gen.CONFIGS["tiny"]
        # this rank's own prompts: a few tokens of the CPU oracle stand in for the device path
        bias = gen.vocab_bias(plan.seed, cfg.V, cfg.slope)
        plen = gen.prompt_lengths(plan.seed, G, cfg.prompt_lo, cfg.prompt_hi)
        prev = np.repeat(gen.prompt_last_token(plan.seed, G, plen, cfg.V), cfg.N)
        groups = np.repeat(np.arange(G), cfg.N)
        o = O.Oracle(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, 0, plan.seed, cfg.eos_id, G=G, T_max=4, prompt_len=plen)
        units = 0
        for t in range(1, 5):
            units += G * cfg.N - int(o.done.sum())
            o.step(gen.logits_block(plan.seed, t, groups, prev, cfg.V, cfg.scale, bias, cfg.dtype))
            prev = o.last_tokens.copy()
        ms_local = 10.0 * (rank + 1)          # rank 1 is the slow one
        replicas.barrier()
        rate, ms, total = replicas.job_throughput(units, ms_local)
        toks = torch.from_numpy(o.last_tokens.astype(np.int64))
        gathered = [torch.zeros_like(toks) for _ in range(world)]
        dist.all_gather(gathered, toks)
        json.dump({"rank": rank, "seed": plan.seed, "offset": plan.group_offset, "units": units, "rate": rate,
                   "ms": ms, "total": total, "tokens": [g.tolist() for g in gathered]},
                  open(os.path.join(out_dir, "r%d.json" % rank), "w"))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_like_the_benchmark(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / ("r%d.json" % r))) for r in range(world)]
    assert [r["seed"] for r in res] == [1, 2] and [r["offset"] for r in res] == [0, 2]
    total = sum(r["units"] for r in res)
    for r in res:
        assert r["total"] == total and r["ms"] == 20.0            # sum of the units, time of the slowest rank
        assert abs(r["rate"] - total / 0.020) < 1e-6
    assert res[0]["tokens"] == res[1]["tokens"]                    # both ranks saw the same gathered picture
    assert res[0]["tokens"][0] != res[0]["tokens"][1]              # replicas decode different prompts


def test_shard_groups_tiles_the_prompts():
    sys.path.insert(0, ROOT)
    from paper_2602_10273_b200 import replicas
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            cuts = [replicas.shard_groups(n, world, r) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            sizes = [hi - lo for lo, hi in cuts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.shard_groups(4, 2, 2)
    with pytest.raises(ValueError):
        replicas.rank_plan(4, env={"WORLD_SIZE": "2", "RANK": "5"})


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--steps", "2",
           "--warmup", "1"]
    p = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""
    env.update(RANK="0", LOCAL_RANK="0")
    p = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
