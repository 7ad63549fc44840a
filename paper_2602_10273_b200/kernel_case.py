"""Run one kernel of the path on a named shape, a few times, with CUDA-event timing.

Meant for profiling sessions (a small, self-ending program to put under ncu) and for quick
what-does-this-shape-cost questions:

  python -m paper_2602_10273_b200.kernel_case logits --rows 512 --vocab 128256 --beta 4 --iters 5
  python -m paper_2602_10273_b200.kernel_case reindex --rows 64 --layers 8 --heads 8 --len 1024 --iters 3
  python -m paper_2602_10273_b200.kernel_case step --workload qwen25_7b --iters 20
  python -m paper_2602_10273_b200.kernel_case shard_step --workload batched_prompts --ranks 8 --iters 20
  python -m paper_2602_10273_b200.kernel_case select --workload batched_prompts --groups 8 --steps 1024 --iters 3

Each case rotates through enough distinct input buffers to exceed the L2 cache, so that the
device-time and DRAM counters describe HBM-bound behaviour.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from .workload import cuda as WC
from .workload import gen

L2_BYTES = 126 << 20


def _time(fn, iters, warmup=2):
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for i, (a, b) in enumerate(ev):
        a.record()
        fn(warmup + i)
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) * 1e3 for a, b in ev]  # microseconds


def case_logits(a):
    R, V = a.rows, a.vocab
    dt = torch.bfloat16 if a.dtype == "bf16" else torch.float32
    esize = 2 if a.dtype == "bf16" else 4
    n_buf = max(2, -(-2 * L2_BYTES // (R * V * esize)))
    n_buf = min(n_buf, 64)
    bufs = []
    for i in range(n_buf):
        x = torch.randn(R, V, device="cuda") * a.scale
        x -= 1.5 * torch.log1p(torch.arange(V, device="cuda", dtype=torch.float32))[torch.randperm(V, device="cuda")]
        bufs.append(x.to(dt))
    nbytes = B.logits_pass_scratch_bytes(R, V)
    scratch = torch.zeros(nbytes + 256, dtype=torch.uint8, device="cuda")
    off = (-scratch.data_ptr()) % 256
    scratch = scratch[off: off + nbytes]
    tok = torch.empty(R, dtype=torch.int32, device="cuda")
    logp = torch.empty(R, dtype=torch.float64, device="cuda")
    loginc = torch.empty(R, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    u = torch.rand(R, dtype=torch.float64, device="cuda").clamp_(1e-9, 1 - 1e-9)

    def run(i):
        B.logits_pass(bufs[i % n_buf], a.beta, a.beta, u, None, scratch, tok, logp, loginc, status)

    us = _time(run, a.iters)
    assert int(status.item()) == 0
    byts = R * V * esize
    return {"case": "logits", "rows": R, "vocab": V, "dtype": a.dtype, "beta": a.beta, "buffers": n_buf,
            "us": us, "us_median": float(np.median(us)), "bytes": byts,
            "gb_per_s": byts / (np.median(us) * 1e-6) / 1e9}


def case_reindex(a):
    """In-place reindex of a cache [rows, heads, len, dim] x layers where every second row is overwritten by its
    left neighbour (half the slots dead, each survivor duplicated once) over the full length."""
    R, H, L, D, NL = a.rows, a.heads, a.len, a.dim, a.layers
    dt = torch.bfloat16 if a.dtype == "bf16" else torch.float32
    ps = B.Psmc(R, 16, 2.0, 0.5, 0.5, 0, 1, 15, T_max=2)
    ks = [torch.randn(R, H, L, D, device="cuda").to(dt) for _ in range(NL)]
    vs = [torch.randn(R, H, L, D, device="cuda").to(dt) for _ in range(NL)]
    desc = ps.make_kv_desc(ks, vs)
    idx = torch.arange(R, dtype=torch.int32, device="cuda")
    idx[1::2] = idx[0::2][: idx[1::2].numel()]
    want = [t[idx.long()].clone() for t in ks[:1]]

    def run(i):
        ps.reindex_kv(desc, None, idx)

    us = _time(run, a.iters)
    assert ps.sync_status() == B.OK and torch.equal(ks[0], want[0])
    moved = R // 2
    byts = 2 * moved * 2 * NL * H * L * D * ks[0].element_size()  # read + write, K and V
    ps.destroy()
    return {"case": "reindex", "rows": R, "layers": NL, "heads": H, "len": L, "dim": D, "dtype": a.dtype,
            "us": us, "us_median": float(np.median(us)), "bytes": byts,
            "gb_per_s": byts / (np.median(us) * 1e-6) / 1e9}


def case_step(a):
    """psmc_step (logit pass + weights/ESS/resampling) on a named workload, logits rotated beyond L2."""
    cfg = gen.CONFIGS[a.workload]
    G = cfg.G if a.groups is None else a.groups
    wl = WC.DeviceWorkload(cfg, 1, G=G)
    n_buf = min(64, max(2, -(-2 * L2_BYTES // (wl.R * cfg.logit_bytes_per_row))))
    T = 3 * a.iters + 12
    ps = B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, 0 if a.no_ramp else cfg.ramp, 1, cfg.eos_id, G=G,
                T_max=T, prompt_len=wl.prompt_len)
    if a.top_k or a.top_p:
        ps.set_proposal_mask(a.top_k, a.top_p)
    bufs = [wl.new_logits() for _ in range(n_buf)]
    prev = wl.first_prev.clone()
    last = ps.device_view("psmc_last_tokens", wl.R)
    # The blocks follow a real run for its first tokens (every row's logits depend on its own last token), so that the
    # particles of a group see different rows, their weights differ and resampling fires as it does in a decoding
    # loop; with the same previous token in every row of a group no step would ever resample.
    wl.fill(bufs[0], 1, prev)
    ps.step(bufs[0])
    prev.copy_(last)
    for i, b in enumerate(bufs):
        wl.fill(b, 2 + i, prev)
        if i < 8:
            ps.step(b)
            prev.copy_(last)
    ps.reset(1)

    def run(i):
        ps.step(bufs[i % n_buf])

    us = _time(run, a.iters)
    assert ps.sync_status() == B.OK
    # the same launches back to back between ONE pair of events: what a step costs in a run of steps, where the next
    # launch is already queued when a kernel ends
    ps.reset(1)
    for i in range(2):
        run(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(a.iters):
        run(2 + i)
    e1.record()
    torch.cuda.synchronize()
    back_to_back = e0.elapsed_time(e1) * 1e3 / a.iters
    assert ps.sync_status() == B.OK
    # the kernels of the step, each bracketed by events on the stream
    ps.reset(1)
    ps.timing_enable(True)
    for i in range(a.iters):
        run(i)
    kms, kn = ps.timing_read()
    ps.timing_enable(False)
    ps.destroy()
    return {"case": "step", "workload": cfg.name, "rows": wl.R, "vocab": cfg.V, "buffers": n_buf, "us": us,
            "top_k": a.top_k, "top_p": a.top_p, "back_to_back_us": back_to_back,
            "logits_stream_us": 1e3 * kms[0] / max(kn[0], 1), "finish_weights_us": 1e3 * kms[1] / max(kn[1], 1),
            "us_median": float(np.median(us)), "bytes": wl.R * cfg.logit_bytes_per_row,
            "gb_per_s": wl.R * cfg.logit_bytes_per_row / (np.median(us) * 1e-6) / 1e9}


def case_select(a):
    """psmc_select (final draw + back-trace of the ancestry log) after --steps tokens of a named workload."""
    cfg = gen.CONFIGS[a.workload]
    G = cfg.G if a.groups is None else a.groups
    wl = WC.DeviceWorkload(cfg, 1, G=G)
    T = a.steps
    ps = B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, 0 if a.no_ramp else cfg.ramp, 1, cfg.eos_id, G=G,
                T_max=T, prompt_len=wl.prompt_len)
    lg = wl.new_logits()
    prev = wl.first_prev.clone()
    last = ps.device_view("psmc_last_tokens", wl.R)
    for t in range(1, T + 1):
        wl.fill(lg, t, prev)
        ps.step(lg)
        prev.copy_(last)
    out = ps.select()

    def run(i):
        ps.select(*out)

    us = _time(run, a.iters)
    assert ps.sync_status() == B.OK
    ps.destroy()
    return {"case": "select", "workload": cfg.name, "groups": G, "particles": cfg.N, "steps": T, "us": us,
            "us_median": float(np.median(us)), "log_bytes": 2 * 4 * wl.R * T}


def case_shard_step(a):
    """One rank's share of the step on a vocabulary split over --ranks ranks (this GPU plays every rank in turn; the
    all-gathers are a stack on the device and are not timed).  Reports rank 0's three calls."""
    from . import vocab_shard as VS
    cfg = gen.CONFIGS[a.workload]
    G = cfg.G if a.groups is None else a.groups
    wl = WC.DeviceWorkload(cfg, 1, G=G)
    shards = VS.vocab_shards(cfg.V, a.ranks)
    n_buf = min(64, max(2, -(-2 * L2_BYTES * a.ranks // (wl.R * cfg.logit_bytes_per_row))))
    T = a.iters + 4
    ranks = [B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, 0 if a.no_ramp else cfg.ramp, 1, cfg.eos_id, G=G,
                    T_max=T, prompt_len=wl.prompt_len) for _ in shards]
    bufs = [wl.new_logits() for _ in range(n_buf)]
    prev = wl.first_prev.clone()
    for i, b in enumerate(bufs):
        wl.fill(b, 1 + i, prev)
    tr = [torch.empty((wl.R, 3), dtype=torch.float64, device="cuda") for _ in shards]
    pk = [torch.empty((wl.R, 2), dtype=torch.int32, device="cuda") for _ in shards]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = []
    for i in range(T - 1):
        lg = bufs[i % n_buf]
        m = [ev() for _ in range(6)]
        for p in range(len(shards) - 1, -1, -1):          # rank 0 last, so that its bracket is followed by the stack
            v0, vl = shards[p]
            if p == 0:
                m[0].record()
            ranks[p].shard_sweep(lg[:, v0:v0 + vl], tr[p])
            if p == 0:
                m[1].record()
        all_tr = torch.stack(tr)
        for p in range(len(shards) - 1, -1, -1):
            if p == 0:
                m[2].record()
            ranks[p].shard_locate(shards[p][0], all_tr, p, pk[p])
            if p == 0:
                m[3].record()
        all_pk = torch.stack(pk)
        for p in range(len(shards) - 1, -1, -1):
            if p == 0:
                m[4].record()
            ranks[p].shard_finish(all_tr, all_pk)
            if p == 0:
                m[5].record()
        marks.append(m)
    torch.cuda.synchronize()
    assert all(r.sync_status() == B.OK for r in ranks)
    marks = marks[-a.iters:]
    med = lambda k: float(np.median([m[k].elapsed_time(m[k + 1]) * 1e3 for m in marks]))
    for r in ranks:
        r.destroy()
    local_bytes = wl.R * shards[0][1] * (2 if cfg.dtype == "bf16" else 4)
    return {"case": "shard_step", "workload": cfg.name, "rows": wl.R, "vocab": cfg.V, "ranks": a.ranks,
            "local_columns": shards[0][1], "buffers": n_buf, "sweep_us": med(0), "locate_us": med(2), "finish_us": med(4),
            "local_logit_bytes": local_bytes, "sweep_gb_per_s": local_bytes / (med(0) * 1e-6) / 1e9,
            "gathered_bytes_per_rank": wl.R * (24 + 8)}


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("case", choices=["logits", "reindex", "step", "shard_step", "select"])
    ap.add_argument("--steps", type=int, default=1024, help="select: tokens decoded before the final draw")
    ap.add_argument("--ranks", type=int, default=8)
    ap.add_argument("--top-k", type=int, default=0, help="step: proposal restricted to the top-k tokens")
    ap.add_argument("--top-p", type=float, default=0.0, help="step: proposal restricted to the nucleus of this share")
    ap.add_argument("--rows", type=int, default=512)
    ap.add_argument("--vocab", type=int, default=128256)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--beta", type=float, default=4.0)
    ap.add_argument("--scale", type=float, default=3.0)
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--heads", type=int, default=8)
    ap.add_argument("--len", type=int, default=1024)
    ap.add_argument("--dim", type=int, default=128)
    ap.add_argument("--workload", default="batched_prompts", choices=sorted(gen.CONFIGS))
    ap.add_argument("--groups", type=int, default=None)
    ap.add_argument("--no-ramp", action="store_true")
    ap.add_argument("--iters", type=int, default=5)
    a = ap.parse_args()
    out = {"logits": case_logits, "reindex": case_reindex, "step": case_step, "shard_step": case_shard_step,
           "select": case_select}[a.case](a)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
