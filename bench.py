#!/usr/bin/env python
"""Benchmark of the Power-SMC hot path on B200: one "step" = one decoded token for every particle =
psmc_step (logit pass, token draw, Eq. 7, weights, ESS, resampling: one kernel) + psmc_reindex_kv (the
cache reorder), on synthetic inputs shaped like the paper's.

  python bench.py --gpus 1 --steps 1016 --warmup 8           # this repository's CUDA path (the defaults)
  python bench.py --impl reference --steps 3 --warmup 1      # the CPU oracle as the reference arm

Prints ONE JSON line.  `value` is particle-tokens/s with every input resident in HBM; `e2e` is the
same metric through psmc_step_host (pinned host logits copied in, tokens copied out, every step).
Multi-GPU (torchrun): every rank runs its own set of prompts (no data-path collective; weak scaling);
time is the max over ranks of the device time of the K timed steps.

What is timed, in order (every pass restarts the run from its reset, so all of them do the same work):
  record   the K steps once with a host read-back per step: bytes each cache move carries, rows alive
  A        the headline: K steps between one pair of events, repeated --repeats times (median, min, max)
  B        the same K steps with a pair of events around every kernel  -> `kernels`, `roofline`
  C        the same K steps with a pair of events around every psmc_step call  -> `step_in_loop`
  D        the K steps without the cache moves: per-kernel pairs, then back to back between one pair of
           events (rotating logit blocks: L2-cold) and on one block (L2-hot)  -> `step_without_kv`
  kv_fixed_event   the cache move of a fixed event: half the slots of every group rewritten, len = max_len / 2
  e2e      a few of the K steps through psmc_step_host
  other_configs    the step alone on the four smaller named configurations, and with the paper's 64 particles
  cpu_baseline     the oracle, as it stands, on a slice of the same workload
Supplementary runs: --paged-kv, --skip-shared-prompt, --top-k K, --top-p P (see their help lines).
"""
from __future__ import annotations

import argparse
import json
import os
import re
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
L2_BYTES = 126 << 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def load_traffic_ratios():
    """DRAM bytes (read + write counters of an ncu capture) per algorithmic byte, per kernel, from the table in
    profiles/dram_traffic_ratios.md; a kernel whose row says `stale` (changed since its counters were taken) or
    that has no row gets no traffic figure."""
    out = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic_ratios.md")
    if not os.path.exists(path):
        return out
    for line in open(path):
        m = re.match(r"\|\s*`?([A-Za-z0-9_]+)`?\s*\|\s*([0-9.]+|stale)\s*\|", line)
        if m and m.group(2) != "stale":
            out[m.group(1)] = float(m.group(2))
    return out


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML while a region runs (read-only)."""

    def __init__(self, local_index: int, period_s: float = 0.01):
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


def events():
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def step_alone(name, hbm_peak, steps=200, seed=1):
    """The step (one kernel) alone on a named configuration, `steps` launches back to back between one pair of events.
    The logit blocks are generated once along a short run and rotated; small configurations cannot leave L2 that way
    (64 blocks at most) and are labelled L2-hot."""
    from paper_2602_10273_b200 import binding as B
    from paper_2602_10273_b200.workload import cuda as WC
    cfg = gen.CONFIGS[name] if isinstance(name, str) else name
    wl = WC.DeviceWorkload(cfg, seed)
    block_bytes = wl.R * cfg.logit_bytes_per_row
    n_buf = int(min(64, max(2, -(-2 * L2_BYTES // block_bytes))))
    T = steps + 8
    ps = B.Psmc(cfg.N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, cfg.ramp, seed, cfg.eos_id, G=cfg.G, T_max=T,
                prompt_len=wl.prompt_len)
    bufs = [wl.new_logits() for _ in range(n_buf)]
    prev = wl.first_prev.clone()
    last = ps.device_view("psmc_last_tokens", wl.R)
    for i, b in enumerate(bufs):
        wl.fill(b, 1 + i, prev)
        if i < 8:
            ps.step(b)
            prev.copy_(last)
    ps.reset(seed)
    for i in range(4):
        ps.step(bufs[i % n_buf])
    e0, e1 = events()
    torch.cuda.synchronize()
    live0 = wl.R - int(ps.done.numpy().sum())
    e0.record()
    for i in range(steps):
        ps.step(bufs[(4 + i) % n_buf])
    e1.record()
    torch.cuda.synchronize()
    assert ps.sync_status() == B.OK
    live1 = wl.R - int(ps.done.numpy().sum())
    us = e0.elapsed_time(e1) * 1e3 / steps
    ps.destroy()
    live = 0.5 * (live0 + live1)
    return {"rows": wl.R, "vocab": cfg.V, "logit_bytes_per_step": block_bytes, "us_per_step": us,
            "particle_tokens_per_s": live / (us * 1e-6), "logit_gb_per_s": block_bytes / (us * 1e-6) / 1e9,
            "frac_of_hbm_peak": block_bytes / (us * 1e-6) / 1e9 / hbm_peak,
            "l2": "cold (%d blocks rotated)" % n_buf if n_buf * block_bytes > L2_BYTES else
                  "hot (%d blocks of %.1f MB fit L2)" % (n_buf, block_bytes / 1e6),
            "steps": steps, "how": "launches back to back between one pair of CUDA events, exponent ramp as configured"}


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
    ratios = load_traffic_ratios()

    K, Wm = args.steps, args.warmup
    T_total = K + Wm
    if cfg.prompt_hi + T_total > cfg.max_len:
        raise SystemExit("steps + warmup exceed the cache length of the workload")
    # shrink the number of prompts only if the cache does not fit this GPU (never the shapes)
    G = cfg.G if args.groups is None else args.groups
    if args.split_prompts:  # strong scaling: the workload's prompts are split over the ranks instead of multiplied
        lo, hi = replicas.shard_groups(G, world, rank)
        G = max(1, hi - lo)
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
    masked = bool(args.top_k or args.top_p)
    if masked:  # supplementary run: proposal restricted to the top of each row
        ps.set_proposal_mask(args.top_k, args.top_p)
    skip = wl.prompt_len if args.skip_shared_prompt else None
    PAGE = 16  # positions per block in the supplementary paged run
    ks = vs = None
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

        def move_cache():
            ps.reindex_kv_paged(pdesc)
    else:
        ks, vs = wl.new_kv()
        desc = ps.make_kv_desc(ks, vs, skip_shared_prompt=args.skip_shared_prompt)

        def reset_all():
            ps.reset(seed)

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

    def one_pass(n_steps, first_t=1, moves=True, hot=False):
        for t in range(first_t, first_t + n_steps):
            ps.step(blocks[0 if hot else (t - 1) % N_BLOCKS])
            if moves:
                move_cache()

    # ---- recording pass: per-step algorithmic KV bytes and live rows (deterministic, so the timed passes repeat it)
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

    # ---- pass A: the headline.  K steps, device-resident inputs, one pair of events around all of them; repeated,
    # the clocks sampled across all repeats ----
    e0, e1 = events()
    ms_runs = []
    with ClockSampler(local) as clk:
        for rep in range(max(1, args.repeats)):
            reset_all()
            one_pass(Wm, 1)
            barrier()
            e0.record()
            one_pass(K, Wm + 1)
            e1.record()
            torch.cuda.synchronize(dev)
            barrier()
            ms_runs.append(max_over_ranks(e0.elapsed_time(e1)))
    assert ps.sync_status() == B.OK
    ms_total = float(np.median(ms_runs))
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
        r = ratios.get(kernel)
        return None if r is None or launches < 1 else r * algorithmic_bytes / launches

    kv_name = "paged_release_acquire_copy_kernels" if args.paged_kv else "reindex_bulk_kernel"
    # with a restricted proposal the logit pass and the group update are two other kernels, bracketed together;
    # a step that cannot run as one kernel (N > 32, unaligned rows) would show a second bracket kind
    k1_name = "masked_rows_kernel+rows_weights_kernel" if masked else "psmc_step_kernel"
    roofs = {
        k1_name: {"bound": "hbm", "achieved": k1_gbs, "peak": hbm_peak, "unit": "GB/s",
                  "frac": k1_gbs / hbm_peak, "traffic": traffic(k1_name, k1_bytes, kn[0]),
                  "peak_kind": peak_kind,
                  "avg_launch_us": 1e3 * kms[0] / max(kn[0], 1), "time_share": shares[0],
                  "bytes_per_launch": k1_bytes / max(kn[0], 1), "launches": int(kn[0]),
                  "what": "the whole psmc_step: logit sweep, token draw, Eq. 7, weights, ESS, resampling"},
        kv_name: {"bound": "hbm", "achieved": k3_gbs, "peak": hbm_peak, "unit": "GB/s",
                  "frac": k3_gbs / hbm_peak, "traffic": traffic(kv_name, k3_bytes, kn[2]),
                  "peak_kind": peak_kind,
                  "avg_launch_us": 1e3 * kms[2] / max(kn[2], 1), "time_share": shares[2],
                  "bytes_per_launch": k3_bytes / max(kn[2], 1), "launches": int(kn[2])},
    }
    if kn[1] > 0:
        roofs["finish_weights_resample_kernel"] = {"bound": "latency", "avg_launch_us": 1e3 * kms[1] / kn[1],
                                                   "time_share": shares[1], "launches": int(kn[1])}
    dominant = kv_name if kms[2] >= kms[0] else k1_name
    roofline = dict(roofs[dominant])
    roofline["kernel"] = dominant

    # ---- pass C: the same K steps with one bracket around each psmc_step ----
    reset_all()
    one_pass(Wm, 1)
    torch.cuda.synchronize(dev)
    ps.timing_enable(2)
    one_pass(K, Wm + 1)
    cms, cn = ps.timing_read()
    ps.timing_enable(False)
    loop_us = 1e3 * cms[0] / max(cn[0], 1)
    loop_gbs = k1_bytes / (cms[0] * 1e-3) / 1e9 if cms[0] > 0 else 0.0

    # ---- pass D: the same K steps without the cache moves between them (the particle state does not depend on the
    # caches): per-kernel brackets, then back to back between one pair of events, L2-cold and L2-hot ----
    reset_all()
    one_pass(Wm, 1, moves=False)
    torch.cuda.synchronize(dev)
    ps.timing_enable(True)
    one_pass(K, Wm + 1, moves=False)
    dms, dn = ps.timing_read()
    ps.timing_enable(False)
    if dms[0] > 0:
        alone_gbs = k1_bytes / (dms[0] * 1e-3) / 1e9
        roofs[k1_name]["without_cache_moves"] = {"avg_launch_us": 1e3 * dms[0] / max(dn[0], 1), "achieved": alone_gbs,
                                                 "frac": alone_gbs / hbm_peak}

    def steps_back_to_back(hot):
        runs = []
        for rep in range(max(1, min(args.repeats, 5))):
            reset_all()
            one_pass(Wm, 1, moves=False, hot=hot)
            barrier()
            e0.record()
            one_pass(K, Wm + 1, moves=False, hot=hot)
            e1.record()
            torch.cuda.synchronize(dev)
            runs.append(max_over_ranks(e0.elapsed_time(e1)))
        return runs

    cold_runs, hot_runs = steps_back_to_back(False), steps_back_to_back(True)
    assert ps.sync_status() == B.OK
    cold_ms, hot_ms = float(np.median(cold_runs)), float(np.median(hot_runs))
    cold_gbs = k1_bytes / (cold_ms * 1e-3) / 1e9

    # ---- the cache move of a fixed event: in every group four slots rewritten by the other four, every row half full
    kv_fixed = None
    if not args.paged_kv and not args.skip_shared_prompt and N % 2 == 0:
        half = cfg.max_len // 2
        lw = np.tile(np.concatenate([np.linspace(0.0, -0.01, N // 2), np.full(N - N // 2, -60.0)]), G)
        lens = np.full(R, half, dtype=np.int32)
        # nothing is added to the weights but a log omega of a few units at most: the heavy half keeps all offspring
        ev_ms, ev_bytes = [], []
        reps = 5
        pe = B.Psmc(N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, 0, seed, cfg.eos_id, G=G, T_max=reps + 2,
                    prompt_len=wl.prompt_len)
        edesc = pe.make_kv_desc(ks, vs)
        for rep in range(reps):
            pe.set_state(log_w=lw, cum_logp=np.zeros(R), done=np.zeros(R, dtype=np.uint8), lens=lens)
            pe.step(blocks[rep % N_BLOCKS])
            b, mv = moved_bytes(pe.slot_map.numpy(), pe.lens.numpy(), G, N, cfg.kv_bytes_per_pos_per_row)
            torch.cuda.synchronize(dev)
            pe.timing_enable(True)
            pe.reindex_kv(edesc)
            ems, en = pe.timing_read()
            pe.timing_enable(False)
            ev_ms.append(ems[2])
            ev_bytes.append((b, mv))
        assert pe.sync_status() == B.OK
        pe.destroy()
        b_med, mv_med = ev_bytes[len(ev_bytes) // 2]
        gbs = [b / (m * 1e-3) / 1e9 for (b, _), m in zip(ev_bytes, ev_ms) if m > 0]
        kv_fixed = {"slots_rewritten": mv_med, "of_slots": R, "len": half + 1, "bytes": b_med,
                    "ms_median": float(np.median(ev_ms)), "gb_per_s_median": float(np.median(gbs)),
                    "frac_of_hbm_peak": float(np.median(gbs)) / hbm_peak, "events": reps}

    # ---- e2e: host logits in, tokens out, every step, through psmc_step_host ----
    Ke = min(K, args.e2e_steps)
    host_blocks = [b.cpu().pin_memory() for b in blocks]
    tok_host = torch.empty(R, dtype=torch.int32).pin_memory()
    reset_all()
    for t in range(1, Wm + 1):
        ps.step_host(host_blocks[(t - 1) % N_BLOCKS], tok_host)
        move_cache()
    barrier()
    e0.record()
    for t in range(Wm + 1, Wm + Ke + 1):
        ps.step_host(host_blocks[(t - 1) % N_BLOCKS], tok_host)
        move_cache()
    e1.record()
    torch.cuda.synchronize(dev)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1))
    e2e_value = sum_over_ranks(float(np.sum(live_rows[Wm:Wm + Ke]))) / (ms_e2e * 1e-3)
    assert ps.sync_status() == B.OK

    live_k = float(np.sum(live_rows[Wm:]))
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "strong" if args.split_prompts else "weak", "vs_baseline": None,
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
        "repeats": {"n": len(ms_runs), "ms_per_step_median": ms_total / K, "ms_per_step_min": min(ms_runs) / K,
                    "ms_per_step_max": max(ms_runs) / K, "timed_region_ms_median": ms_total,
                    "how": "every repeat: reset, W warm-up steps, K steps between one pair of events; value from the median"},
        "clocks": clk.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": R * cfg.logit_bytes_per_row,
                "d2h_bytes_per_step": R * 4, "steps": Ke, "ms_per_step": ms_e2e / Ke},
        # per step: the step kernel (two kernels when the proposal is restricted) + the cache move (one bulk reindex
        # kernel per 64 layers, or release + acquire + copy for the paged cache)
        "gpu_launches": int(K * ((2 if masked else 1) + (3 if args.paged_kv else (cfg.n_layers + 63) // 64))),
        "roofline": roofline,
        "kernels": roofs,
        # the whole step against the HBM roofline: algorithmic bytes of all its kernels over the headline time
        "step_roofline": {"bound": "hbm", "bytes_per_step": (k1_bytes + k3_bytes) / K,
                          "achieved": (k1_bytes + k3_bytes) / (ms_total * 1e-3) / 1e9, "peak": hbm_peak,
                          "unit": "GB/s", "frac": (k1_bytes + k3_bytes) / (ms_total * 1e-3) / 1e9 / hbm_peak},
        "kv_reindex": {"gb_per_s": k3_gbs, "frac_of_hbm_peak": k3_gbs / hbm_peak,
                       "slots_moved_per_step": float(np.mean(moved_slots[Wm:])),
                       "gb_moved_per_step": k3_bytes / K / 1e9, "fixed_event": kv_fixed},
        # metric (i): particle-tokens/s of the step alone = live rows / time of the step's kernel(s)
        "step_without_kv": {"particle_tokens_per_s": live_k / (cold_ms * 1e-3), "us_per_step": 1e3 * cold_ms / K,
                            "logit_gb_per_s": cold_gbs, "frac_of_hbm_peak": cold_gbs / hbm_peak,
                            "us_per_step_min": 1e3 * min(cold_runs) / K, "us_per_step_max": 1e3 * max(cold_runs) / K,
                            "repeats": len(cold_runs),
                            "l2_hot": {"us_per_step": 1e3 * hot_ms / K, "particle_tokens_per_s": live_k / (hot_ms * 1e-3),
                                       "how": "the same launches on one logit block (%.0f MB against %d MB of L2)" % (
                                           R * cfg.logit_bytes_per_row / 1e6, L2_BYTES >> 20)},
                            "how": "K psmc_step launches back to back between one pair of CUDA events, no cache moves, "
                                   "logit blocks rotated (L2-cold); median of the repeats"},
        "step_in_loop": {"us_per_step": loop_us, "particle_tokens_per_s": live_k / (cms[0] * 1e-3) if cms[0] > 0 else 0.0,
                         "logit_gb_per_s": loop_gbs, "frac_of_hbm_peak": loop_gbs / hbm_peak,
                         "how": "one CUDA-event bracket around each psmc_step between the cache moves of the headline loop: "
                                "includes the launch gap of a bracketed launch and the write-back of the preceding cache "
                                "move's dirty L2 lines, which drain while the step streams its logits"},
    }
    if rank == 0 and world == 1 and not args.no_other_configs and not masked and not args.paged_kv:
        out["other_configs"] = {n: step_alone(n, hbm_peak) for n in ("tiny", "llama2_7b", "qwen25_7b", "resample_stress")}
        # the particle count of the paper's own runs (Section 6: N = 64) on the largest vocabulary of the named shapes:
        # a group one warp cannot update, so the step is the one kernel followed by the group-update kernel
        import dataclasses
        out["other_configs"]["qwen25_7b_64_particles"] = step_alone(
            dataclasses.replace(gen.CONFIGS["qwen25_7b"], name="qwen25_7b_64_particles", N=64), hbm_peak)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(cfg, wl.seed, wl.prompt_len, [logits_to_numpy(b) for b in blocks], G)
    ps.destroy()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def oracle_slice_run(cfg, seed, prompt_len, block_of, Gs, n_steps, n_warm=0, budget_s=None):
    """The oracle, as it stands, on the first Gs prompts of the workload with their WHOLE cache (every layer, K and
    V, every head, max_len positions, held in host memory): each step is its step function on the slice's rows of the
    logit block followed by its reindex loop over every cache tensor with that step's slot map and lengths.
    block_of(t, oracle) hands out the logits of step t (not timed).  Returns (rows, seconds, moved bytes) over the
    timed steps."""
    from oracle import oracle as O
    N = cfg.N
    rows = Gs * N
    o = O.Oracle(N, cfg.V, cfg.alpha, cfg.tau, cfg.kappa, cfg.ramp, seed, cfg.eos_id, G=Gs, T_max=n_steps + n_warm,
                 prompt_len=prompt_len[:Gs])
    np_dt = np.uint16 if cfg.dtype == "bf16" else np.float32
    cache = [np.ones((rows, cfg.n_kv_heads, cfg.max_len, cfg.head_dim), dtype=np_dt) for _ in range(2 * cfg.n_layers)]
    done_rows, moved, secs = 0, 0, 0.0
    for t in range(n_steps + n_warm):
        blk = block_of(t, o)
        live = rows - int(o.done.sum())
        t0 = time.perf_counter()
        o.step(blk)
        idx = (o.slot_map.reshape(Gs, N) + (np.arange(Gs) * N)[:, None]).reshape(-1).astype(np.int32)
        ln = o.lens
        for c in cache:
            O.reindex_tensor(c, c, idx, ln)
        dt = time.perf_counter() - t0
        if t >= n_warm:
            secs += dt
            done_rows += live
            moved += moved_bytes(o.slot_map, ln, Gs, N, cfg.kv_bytes_per_pos_per_row)[0]
            if budget_s is not None and secs > budget_s:
                break
    return done_rows, secs, moved


def cpu_baseline(cfg, seed, prompt_len, host_blocks, G, n_steps=600, Gs=4):
    """One real oracle step (rows + its reindex loop over the same moves), timed as it stands on the host cores, on
    a slice of the workload: Gs of the G prompts, every layer of their cache."""
    cores = len(os.sched_getaffinity(0))
    Gs = min(Gs, G)
    n_rows = Gs * cfg.N
    rows, secs, moved = oracle_slice_run(cfg, seed, prompt_len, lambda t, o: host_blocks[t % len(host_blocks)][:n_rows],
                                         Gs, n_steps, n_warm=1, budget_s=20.0)
    return {"value": rows / secs, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d of the %d prompts (%d rows) with their whole cache (%d layers, K and V, %d heads, max_len %d), "
                      "up to %d tokens or 20 s: oracle step + its reindex loop over the step's moves, %d live rows in "
                      "%.1f s wall on %d threads, %.2f GB of cache moved" % (
                          Gs, G, Gs * cfg.N, cfg.n_layers, cfg.n_kv_heads, cfg.max_len, n_steps, rows, secs, cores,
                          moved / 1e9),
            "seconds": secs, "rows": rows, "kv_bytes_moved": moved}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only).  Each step is a bounded
    sample of the workload: the first 4 prompts with their whole cache."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg = gen.CONFIGS[args.workload]
    seed = 1
    G = cfg.G if args.groups is None else args.groups
    Gs = min(G, 4)
    bias = gen.vocab_bias(seed, cfg.V, cfg.slope)
    plen = gen.prompt_lengths(seed, G, cfg.prompt_lo, cfg.prompt_hi)
    first_prev = np.repeat(gen.prompt_last_token(seed, G, plen, cfg.V), cfg.N)[: Gs * cfg.N]
    groups = np.repeat(np.arange(Gs), cfg.N)

    def block_of(t, o):  # the synthetic LM along the oracle's own run: logits of step t+1 given each slot's last token
        prev = first_prev if t == 0 else o.last_tokens
        return gen.logits_block(seed, t + 1, groups, prev, cfg.V, cfg.scale, bias, cfg.dtype)

    K, Wm = args.steps, args.warmup
    rows, secs, moved = oracle_slice_run(cfg, seed, plen, block_of, Gs, K, n_warm=Wm)
    value = rows / secs
    cores = len(os.sched_getaffinity(0))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": K, "warmup": Wm, "ms_per_step": 1e3 * secs / K * (G / Gs), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s (CPU oracle on the first %d of %d prompts per step, whole cache; ms_per_step scaled "
                               "to all prompts)" % (cfg.name, Gs, G)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "oracle step on %d prompts (%d rows) per step + its reindex loop over every layer of "
                                   "their cache (%.2f GB moved in %d steps)" % (Gs, Gs * cfg.N, moved / 1e9, K)},
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
    ap.add_argument("--split-prompts", action="store_true",
                    help="with several ranks: split the workload's prompts over them (strong scaling) instead of giving "
                         "every rank the whole set (weak scaling, the default)")
    ap.add_argument("--repeats", type=int, default=10, help="how often the headline pass is repeated (median reported)")
    ap.add_argument("--e2e-steps", type=int, default=24)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the step-alone figures of the smaller configurations")
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
