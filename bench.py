#!/usr/bin/env python
"""Benchmark of the Power-SMC hot path on B200: one "step" = one decoded token for every particle =
logit pass + weights/ESS/resampling + KV-cache reindex, on synthetic inputs shaped like the paper's.

  python bench.py --gpus 1 --steps 1016 --warmup 8           # this repository's CUDA path (the defaults)
  python bench.py --impl reference --steps 3 --warmup 1      # the CPU oracle as the reference arm

Prints ONE JSON line.  `value` is particle-tokens/s with every input resident in HBM; `e2e` is the
same metric through psmc_step_host (pinned host logits copied in, tokens copied out, every step).
Multi-GPU (torchrun): every rank runs its own set of prompts (no data-path collective; weak scaling);
time is the max over ranks of the device time of the K timed steps.

The K steps are made several times: once to record the bytes each step moves, once for the headline time, once with
CUDA events around every kernel (`kernels`, `roofline`), once with one bracket per psmc_step (`step_without_kv`), once
without the cache moves (`kernels.*.without_cache_moves`), and a few of them through psmc_step_host (`e2e`).
Supplementary runs: --paged-kv, --skip-shared-prompt, --top-k K, --top-p P (see their help lines).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2602_10273_b200.workload import gen  # noqa: E402

METRIC = "particle_tokens_per_s"
UNIT = "particle-tokens/s"
N_BLOCKS = 6           # distinct logit blocks rotated through (6 x 131 MB at the default workload: beyond L2)
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per algorithmic byte, from the ncu captures summarised
# under profiles/ (logits_stream_kernel__batched_prompts.md, reindex_bulk_kernel__64rows_8layers_len1024.md; the
# reindex capture ran on a smaller cache and its traffic scales with the bytes moved).  An entry goes back to None
# when its kernel changes, until the counters are taken again.
TRAFFIC_PER_ALGORITHMIC_BYTE = {"logits_stream_kernel": 1.03, "reindex_bulk_kernel": 0.978}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML while a region runs (read-only)."""

    def __init__(self, local_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz, self._stop = [], set(), None, threading.Event()
        self.period = period_s
        self.thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            entry = vis.split(",")[local_index].strip() if vis else str(local_index)
            if entry.isdigit():
                self.h = pynvml.nvmlDeviceGetHandleByIndex(int(entry))
            else:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(entry.encode() if hasattr(entry, "encode") else entry)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                    nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = get(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self.thread is not None:
            self.thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def logits_to_numpy(t: torch.Tensor) -> np.ndarray:
    """Device logits -> host array the oracle reads (fp32 as is, bf16 as uint16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def moved_bytes(slot_map, lens, G, N, bytes_per_pos, skip=None):
    """Algorithmic bytes of one KV reindex: each source with surplus offspring is read once, each rewritten slot
    written once; lens are the post-step live lengths (a rewritten slot carries its source's length).  skip [G]:
    positions at the start of every row of the group that stay in place (a prompt shared by the group)."""
    m = slot_map.reshape(G, N)
    ln = lens.reshape(G, N)
    if skip is not None:
        ln = np.maximum(ln - np.asarray(skip).reshape(G, 1), 0)
    moved = m != np.arange(N)[None, :]
    wr = int(ln[moved].sum())
    rd = 0
    for g in np.nonzero(moved.any(axis=1))[0]:
        srcs = np.unique(m[g][moved[g]])
        rd += int(ln[g][srcs].sum())
    return (rd + wr) * bytes_per_pos, int(moved.sum())


def run_ours(args):
    from paper_2602_10273_b200 import binding as B
    from paper_2602_10273_b200.workload import cuda as WC

    from paper_2602_10273_b200 import replicas

    cfg = gen.CONFIGS[args.workload]
    plan = replicas.rank_plan(cfg.G if args.groups is None else args.groups)
    world, rank, local = plan.world, plan.rank, plan.local_rank
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    hbm_peak, peak_kind = load_peaks()

    K, Wm = args.steps, args.warmup
    T_total = K + Wm
    if cfg.prompt_hi + T_total > cfg.max_len:
        raise SystemExit("steps + warmup exceed the cache length of the workload")
    # shrink the number of prompts only if the cache does not fit this GPU (never the shapes)
    G = cfg.G if args.groups is None else args.groups
    free_b, _ = torch.cuda.mem_get_info(dev)
    per_group = cfg.N * cfg.max_len * cfg.kv_bytes_per_pos_per_row
    fixed = N_BLOCKS * cfg.N * cfg.logit_bytes_per_row  # per group
    while G > 1 and G * (per_group + fixed) + (6 << 30) > free_b:
        G -= 1
    seed = plan.seed
    wl = WC.DeviceWorkload(cfg, seed, G=G, device=dev)
    R, N = wl.R, cfg.N
    ps = B.Psmc(N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, cfg.ramp, seed, cfg.eos_id, G=G, T_max=T_total,
                prompt_len=wl.prompt_len)
    if args.top_k or args.top_p:  # supplementary run: proposal restricted to the top of each row
        ps.set_proposal_mask(args.top_k, args.top_p)
    skip = wl.prompt_len if args.skip_shared_prompt else None
    PAGE = 16  # positions per block in the supplementary paged run
    if args.paged_kv:  # same capacity as the dense cache, cut into blocks reached through a table
        max_blocks = -(-cfg.max_len // PAGE)
        n_blocks = R * max_blocks
        shape = (n_blocks, cfg.n_kv_heads, PAGE, cfg.head_dim)
        kpools = [torch.empty(shape, dtype=wl.tdtype, device=dev) for _ in range(cfg.n_layers)]
        vpools = [torch.empty(shape, dtype=wl.tdtype, device=dev) for _ in range(cfg.n_layers)]
        ps.kv_paged_create(n_blocks, PAGE, max_blocks, share_prompt=True)
        ps.kv_paged_append()
        pdesc = ps.make_kv_pools(kpools, vpools)

        def reset_all():
            ps.reset(seed)
            ps.kv_paged_create(n_blocks, PAGE, max_blocks, share_prompt=True)
            ps.kv_paged_append()  # blocks for the first token; psmc_reindex_kv_paged sees to every later one

        def before_step():
            pass

        def move_cache():
            ps.reindex_kv_paged(pdesc)
    else:
        ks, vs = wl.new_kv()
        desc = ps.make_kv_desc(ks, vs, skip_shared_prompt=args.skip_shared_prompt)

        def reset_all():
            ps.reset(seed)

        def before_step():
            pass

        def move_cache():
            ps.reindex_kv(desc)
    last = ps.device_view("psmc_last_tokens", R)

    # logit blocks: generated along a short closed loop, then reused cyclically by every pass below
    blocks = [wl.new_logits() for _ in range(N_BLOCKS)]
    prev = wl.first_prev.clone()
    for t in range(1, N_BLOCKS + 1):
        wl.fill(blocks[t - 1], t, prev)
        ps.step(blocks[t - 1])
        prev.copy_(last)
    assert ps.sync_status() == B.OK
    reset_all()

    def one_pass(n_steps, first_t=1):
        for t in range(first_t, first_t + n_steps):
            before_step()
            ps.step(blocks[(t - 1) % N_BLOCKS])
            move_cache()

    # recording pass: per-step algorithmic KV bytes and live rows (deterministic, so the timed passes repeat it)
    kv_bytes, moved_slots, live_rows = [], [], []
    for t in range(1, T_total + 1):
        live_rows.append(R - int(ps.done.numpy().sum()))  # rows that are live when step t starts
        one_pass(1, t)
        if args.paged_kv:  # one partly filled block per rewritten slot, read and written once
            sm, ln = ps.slot_map.numpy().reshape(G, N), ps.lens.numpy().reshape(G, N)
            mvd = sm != np.arange(N)[None, :]
            b, mv = 2 * int((ln[mvd] % PAGE).sum()) * cfg.kv_bytes_per_pos_per_row, int(mvd.sum())
        else:
            b, mv = moved_bytes(ps.slot_map.numpy(), ps.lens.numpy(), G, N, cfg.kv_bytes_per_pos_per_row, skip)
        kv_bytes.append(b)
        moved_slots.append(mv)
    assert ps.sync_status() == B.OK
    live_timed = int(np.sum(live_rows[Wm:]))

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize(dev)

    def max_over_ranks(x):
        return replicas.max_over_ranks(x, dev)

    def sum_over_ranks(x):
        return replicas.sum_over_ranks(x, dev)

    # ---- pass A: the headline. K steps, device-resident inputs, one pair of events around all of them ----
    reset_all()
    one_pass(Wm, 1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(local) as clk:
        e0.record()
        one_pass(K, Wm + 1)
        e1.record()
        torch.cuda.synchronize(dev)
    barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    assert ps.sync_status() == B.OK
    value = sum_over_ranks(live_timed) / (ms_total * 1e-3)

    # ---- pass B: same K steps with every kernel bracketed by events, for the roofline of each kernel ----
    reset_all()
    one_pass(Wm, 1)
    torch.cuda.synchronize(dev)
    ps.timing_enable(True)
    one_pass(K, Wm + 1)
    kms, kn = ps.timing_read()
    ps.timing_enable(False)
    k1_bytes = float(np.sum(live_rows[Wm:])) * cfg.logit_bytes_per_row
    k3_bytes = float(np.sum(kv_bytes[Wm:]))
    k1_gbs = k1_bytes / (kms[0] * 1e-3) / 1e9 if kms[0] > 0 else 0.0
    k3_gbs = k3_bytes / (kms[2] * 1e-3) / 1e9 if kms[2] > 0 and k3_bytes > 0 else 0.0
    shares = [m / max(sum(kms), 1e-12) for m in kms]

    def traffic(kernel, algorithmic_bytes, launches):
        r = TRAFFIC_PER_ALGORITHMIC_BYTE.get(kernel)
        return None if r is None or launches < 1 else r * algorithmic_bytes / launches

    dominant = int(np.argmax(kms))
    kv_name = "paged_release_acquire_copy_kernels" if args.paged_kv else "reindex_bulk_kernel"
    # with a restricted proposal the logit pass and the group update are two other kernels, bracketed together
    k1_name = "masked_rows_kernel+rows_weights_kernel" if (args.top_k or args.top_p) else "logits_stream_kernel"
    names = [k1_name, "finish_weights_resample_kernel", kv_name]
    roofs = {
        k1_name: {"bound": "hbm", "achieved": k1_gbs, "peak": hbm_peak, "unit": "GB/s",
                               "frac": k1_gbs / hbm_peak, "traffic": traffic(k1_name, k1_bytes, kn[0]),
                               "peak_kind": peak_kind,
                               "avg_launch_us": 1e3 * kms[0] / max(kn[0], 1), "time_share": shares[0],
                               "bytes_per_launch": k1_bytes / max(kn[0], 1)},
        kv_name: {"bound": "hbm", "achieved": k3_gbs, "peak": hbm_peak, "unit": "GB/s",
                                "frac": k3_gbs / hbm_peak, "traffic": traffic(kv_name, k3_bytes, kn[2]),
                                "peak_kind": peak_kind,
                                "avg_launch_us": 1e3 * kms[2] / max(kn[2], 1), "time_share": shares[2],
                                "bytes_per_launch": k3_bytes / max(kn[2], 1)},
        "finish_weights_resample_kernel": {"bound": "latency", "avg_launch_us": 1e3 * kms[1] / max(kn[1], 1),
                                    "time_share": shares[1]},
    }
    roofline = dict(roofs[names[dominant]] if dominant != 1 else roofs[kv_name])
    roofline["kernel"] = names[dominant] if dominant != 1 else kv_name

    # ---- pass C: the same K steps with one bracket around each psmc_step (its kernels keep their chained launches) ----
    reset_all()
    one_pass(Wm, 1)
    torch.cuda.synchronize(dev)
    ps.timing_enable(2)
    one_pass(K, Wm + 1)
    cms, cn = ps.timing_read()
    ps.timing_enable(False)
    step_us = 1e3 * cms[0] / max(cn[0], 1)
    step_gbs = k1_bytes / (cms[0] * 1e-3) / 1e9 if cms[0] > 0 else 0.0

    # ---- pass D: the same K steps without the cache moves between them, per-kernel brackets: the logit pass when no
    # reindex has left its writes in L2 for it to drain (the particle state does not depend on the caches) ----
    reset_all()
    for t in range(1, Wm + 1):
        ps.step(blocks[(t - 1) % N_BLOCKS])
    torch.cuda.synchronize(dev)
    ps.timing_enable(True)
    for t in range(Wm + 1, Wm + K + 1):
        ps.step(blocks[(t - 1) % N_BLOCKS])
    dms, dn = ps.timing_read()
    ps.timing_enable(False)
    if dms[0] > 0:
        alone_gbs = k1_bytes / (dms[0] * 1e-3) / 1e9
        roofs[k1_name]["without_cache_moves"] = {"avg_launch_us": 1e3 * dms[0] / max(dn[0], 1), "achieved": alone_gbs,
                                                 "frac": alone_gbs / hbm_peak}

    # ---- e2e: host logits in, tokens out, every step, through psmc_step_host ----
    Ke = min(K, args.e2e_steps)
    host_blocks = [b.cpu().pin_memory() for b in blocks]
    tok_host = torch.empty(R, dtype=torch.int32).pin_memory()
    reset_all()
    for t in range(1, Wm + 1):
        before_step()
        ps.step_host(host_blocks[(t - 1) % N_BLOCKS], tok_host)
        move_cache()
    barrier()
    e0.record()
    for t in range(Wm + 1, Wm + Ke + 1):
        before_step()
        ps.step_host(host_blocks[(t - 1) % N_BLOCKS], tok_host)
        move_cache()
    e1.record()
    torch.cuda.synchronize(dev)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1))
    e2e_value = sum_over_ranks(float(np.sum(live_rows[Wm:Wm + Ke]))) / (ms_e2e * 1e-3)
    assert ps.sync_status() == B.OK

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": "%s: %d prompts x %d particles, V=%d, KV %dx%dx%d max_len %d (%s)" % (
                       cfg.name, G, N, cfg.V, cfg.n_layers, cfg.n_kv_heads, cfg.head_dim, cfg.max_len, cfg.dtype),
                   "prompts_per_gpu": G, "rows_per_gpu": R, "alpha": cfg.alpha, "tau": cfg.tau, "kappa": cfg.kappa,
                   "ramp": cfg.ramp, "l2": "inputs larger than L2: %d logit blocks of %.0f MB rotated, KV %.1f GB" % (
                       N_BLOCKS, R * cfg.logit_bytes_per_row / 1e6, G * per_group / 1e9),
                   "kv_reindex": ("paged cache, blocks of %d positions, copy on write" % PAGE) if args.paged_kv else
                                 ("prompt positions left in place" if args.skip_shared_prompt else "whole live prefix copied"),
                   "proposal": ("top-k %d" % args.top_k) if args.top_k else ("nucleus %.3g" % args.top_p) if args.top_p
                               else "softmax(beta l) over the whole vocabulary (Corollary 1)",
                   "parallelism": "replicas only (prompts sharded, no collective)"},
        "clocks": clk.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": R * cfg.logit_bytes_per_row,
                "d2h_bytes_per_step": R * 4, "steps": Ke, "ms_per_step": ms_e2e / Ke},
        # per step: logit pass + finish/weights/resampling (two kernels on this workload) + the cache move (one bulk
        # reindex kernel per 64 layers, or release + acquire (which also prepares the next token's blocks) + copy for the paged cache)
        "gpu_launches": int(K * (2 + (3 if args.paged_kv else (cfg.n_layers + 63) // 64))),
        "roofline": roofline,
        "kernels": roofs,
        # the whole step against the HBM roofline: algorithmic bytes of all its kernels over the headline time
        "step_roofline": {"bound": "hbm", "bytes_per_step": (k1_bytes + k3_bytes) / K,
                          "achieved": (k1_bytes + k3_bytes) * world / (ms_total * 1e-3) / 1e9 / world, "peak": hbm_peak,
                          "unit": "GB/s", "frac": (k1_bytes + k3_bytes) / (ms_total * 1e-3) / 1e9 / hbm_peak},
        "kv_reindex": {"gb_per_s": k3_gbs, "frac_of_hbm_peak": k3_gbs / hbm_peak,
                       "slots_moved_per_step": float(np.mean(moved_slots[Wm:])),
                       "gb_moved_per_step": k3_bytes / K / 1e9},
        "step_without_kv": {"particle_tokens_per_s": float(np.sum(live_rows[Wm:])) / (cms[0] * 1e-3) if cms[0] > 0 else 0.0,
                            "us_per_step": step_us, "logit_gb_per_s": step_gbs, "frac_of_hbm_peak": step_gbs / hbm_peak,
                            "how": "one CUDA-event bracket around each psmc_step (logit pass + finish/weights/resampling)"},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(cfg, wl, blocks, G, float(np.mean(kv_bytes[Wm:])))
    ps.destroy()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def oracle_step_rate(cfg, seed, G, logits_host_blocks, prompt_len, n_steps):
    """Times the CPU oracle (as it stands) on n_steps of the given blocks; returns (rows/s, seconds, rows)."""
    from oracle import oracle as O
    o = O.Oracle(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, cfg.ramp, seed, cfg.eos_id, G=G, T_max=n_steps,
                 prompt_len=prompt_len)
    rows = 0
    t0 = time.perf_counter()
    for t in range(n_steps):
        rows += G * cfg.N - int(o.done.sum())
        o.step(logits_host_blocks[t % len(logits_host_blocks)])
    return rows / (time.perf_counter() - t0), time.perf_counter() - t0, rows


def oracle_copy_rate(cfg):
    """GB/s (read + write) of the oracle's KV reindex loop on a 4-row slice of one layer tensor."""
    from oracle import oracle as O
    rng = np.random.default_rng(0)
    t = rng.integers(0, 2**16, size=(4, cfg.n_kv_heads, cfg.max_len, cfg.head_dim), dtype=np.uint16)
    if cfg.dtype == "f32":
        t = t.astype(np.float32)
    idx = np.array([1, 1, 3, 3], dtype=np.int32)
    O.reindex_tensor(t, t, idx, None)  # touch
    reps = 20
    t0 = time.perf_counter()
    for _ in range(reps):
        O.reindex_tensor(t, t, idx, None)
    dt = time.perf_counter() - t0
    return reps * 2 * 2 * t[0].nbytes / dt / 1e9


def cpu_baseline(cfg, wl, blocks, G, kv_bytes_per_step, n_steps=24):
    """The oracle as it stands on the host cores: every row of the workload for n_steps tokens (the logit blocks
    the CUDA path was timed on, downloaded), plus the rate of its KV reindex loop applied to one step's moves."""
    cores = len(os.sched_getaffinity(0))
    host = [logits_to_numpy(b) for b in blocks]
    rate, secs, rows = oracle_step_rate(cfg, wl.seed, G, host, wl.prompt_len, n_steps)
    copy_gbs = oracle_copy_rate(cfg)
    # one full step on the CPU = the oracle's step for all rows + its memcpy loop over the step's KV bytes
    t_step = (G * cfg.N) / rate + kv_bytes_per_step / (copy_gbs * 1e9)
    return {"value": (G * cfg.N) / t_step, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "oracle step on all %d prompts (%d rows) for %d tokens: %.0f rows/s in %.1f s wall on %d threads; "
                      "oracle KV reindex loop on a 4-row slice of one layer: %.1f GB/s; combined for one full step of "
                      "%d rows and %.2f GB of KV moves" % (G, G * cfg.N, n_steps, rate, secs, cores, copy_gbs,
                                                          G * cfg.N, kv_bytes_per_step / 1e9),
            "oracle_rows_per_s": rate, "oracle_copy_gb_per_s": copy_gbs}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg = gen.CONFIGS[args.workload]
    seed = 1
    G = cfg.G if args.groups is None else args.groups
    Gs = min(G, 8)                      # each step is a bounded sample: the first 8 prompts
    bias = gen.vocab_bias(seed, cfg.V, cfg.slope)
    plen = gen.prompt_lengths(seed, G, cfg.prompt_lo, cfg.prompt_hi)
    prev = np.repeat(gen.prompt_last_token(seed, G, plen, cfg.V), cfg.N)[: Gs * cfg.N]
    groups = np.repeat(np.arange(Gs), cfg.N)
    host = [gen.logits_block(seed, t, groups, prev, cfg.V, cfg.scale, bias, cfg.dtype) for t in (1, 2)]
    K, Wm = args.steps, args.warmup
    from oracle import oracle as O
    o = O.Oracle(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, cfg.ramp, seed, cfg.eos_id, G=Gs, T_max=K + Wm,
                 prompt_len=plen[:Gs])
    copy_gbs = oracle_copy_rate(cfg)
    for t in range(Wm):
        o.step(host[t % 2])
    rows, kv_b = 0, 0.0
    t0 = time.perf_counter()
    for t in range(K):
        rows += Gs * cfg.N - int(o.done.sum())
        o.step(host[(Wm + t) % 2])
        b, _ = moved_bytes(o.slot_map, o.lens, Gs, cfg.N, cfg.kv_bytes_per_pos_per_row)
        kv_b += b
    secs = time.perf_counter() - t0 + kv_b / (copy_gbs * 1e9)
    value = rows / secs
    cores = len(os.sched_getaffinity(0))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": Wm, "ms_per_step": 1e3 * secs / K * (G / Gs), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s (CPU oracle on the first %d of %d prompts per step)" % (cfg.name, Gs, G)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "oracle step on %d prompts (%d rows) per step plus its KV reindex loop rate "
                                   "(%.1f GB/s on a 4-row slice) applied to the step's moved bytes" % (
                                       Gs, Gs * cfg.N, copy_gbs)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="batched_prompts", choices=sorted(gen.CONFIGS))
    ap.add_argument("--groups", type=int, default=None, help="override the number of prompts (default: the workload's)")
    ap.add_argument("--e2e-steps", type=int, default=24)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--paged-kv", action="store_true",
                    help="supplementary run: paged cache with copy-on-write resampling instead of the dense cache")
    ap.add_argument("--skip-shared-prompt", action="store_true",
                    help="supplementary run: the KV reindex leaves each group's prompt positions in place (not the "
                         "headline configuration, which copies whole live prefixes)")
    ap.add_argument("--top-k", type=int, default=0, help="supplementary run: proposal restricted to the top-k tokens")
    ap.add_argument("--top-p", type=float, default=0.0, help="supplementary run: proposal restricted to a nucleus")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 1016 if args.steps is None else args.steps  # with the warm-up: all 1024 tokens of the workload
        args.warmup = 8 if args.warmup is None else args.warmup
        if args.warmup < 3:
            args.warmup = 3
        run_ours(args)


if __name__ == "__main__":
    main()
