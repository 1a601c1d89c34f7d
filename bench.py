#!/usr/bin/env python
"""Benchmark of the CoWA hot path on B200.

One step = one pass of the whole hot path on seeded synthetic inputs:
  training forward + backward at the 128K configuration (B=1, T=131072, Hq=32, Hkv=8, D=128,
  sink 128, near 4096) followed by one split-KV decode step of the 128K decode configuration
  (batch 8, lengths in [96K, 128K]).
`value` is TFLOP/s over visited tiles of forward + backward (4*D resp. 10*D FLOPs per visited
query-key pair and QO head); the decode phase is reported beside it (us per step, GB/s).

    python bench.py [--gpus N] [--steps K] [--warmup W]          # the CUDA library
    python bench.py --impl reference [...]                       # the CPU oracle, bounded sample

Under torchrun every rank runs the same workload on its own GPU (independent replicas: the
operator has no exchange step); rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import itertools
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

TRAIN_CFG, DECODE_CFG = "128k", "decode128k"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic():
    """DRAM bytes per launch of the kernels, from the tracked ncu summary profiles/traffic.json:
    {kernel name: {workload: {"bytes_per_launch": ..., "source": ...}}}."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        return json.load(f)


def traffic_for(table, kernel, workload):
    """The recorded figure for this kernel name and workload, or None: a renamed kernel or a workload that was
    never captured gets no number."""
    e = table.get(kernel)
    if not isinstance(e, dict) or workload not in e:
        return None
    return e[workload].get("bytes_per_launch")


def tp_shards(rank, world, tp):
    """KV-head shards of a TP group of `tp` ranks that process `rank` of `world` times: its own shard when
    world == tp, every world-th shard when fewer processes than shards run, none for surplus processes."""
    return list(range(rank, tp, world))


def duplicated_windows(windows, m):
    """Control layout of the collective-coverage study: head h gets the band of head h mod m of the default
    layout (every head keeps the shared sink and near windows)."""
    return [windows[h % m] for h in range(len(windows))]


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def barrier(world):
    import torch
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x, world):
    """Largest value of x over the ranks (device timings are reported as the slowest rank's)."""
    import torch
    if world == 1:
        return x
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------------------------------
# CPU oracle timing (bounded sample of the 128K forward), used by cpu_baseline and --impl reference
# ------------------------------------------------------------------------------------------

def oracle_sample(budget_s, seed_tiles=0):
    """Times the oracle on units of the 128K training configuration until about budget_s seconds are spent.
    A unit is one (KV head, 128-row query tile): its forward (O, LSE) and the backward terms that belong to
    those query rows (recompute of S and P, dP, dS, dQ); the dK / dV sums of a unit's keys run over every query
    row of the sequence and are left out of the sample.  Returns the FLOPs the oracle actually performed over
    legal pairs (4*D per pair forward, 6*D per pair for S, dP and dQ of the backward), the seconds used and the
    number of units."""
    import numpy as np
    import torch
    import cowa_inputs
    from oracle import cowa_oracle as orc
    c = cowa_inputs.CONFIGS[TRAIN_CFG]
    T, Hq, Hkv, D = c["T"], c["Hq"], c["Hkv"], c["D"]
    ws = orc.default_windows(T, Hkv, c["sink"], c["local"])
    scale = cowa_inputs.softmax_scale(D)
    g = torch.Generator().manual_seed(c["index"] * 1000 + 7)
    # one head's tensors (synthetic N(0,1), bf16-rounded like the GPU inputs), reused by every unit
    flops, secs, units = 0.0, 0.0, 0
    rng = np.random.default_rng(seed_tiles)
    k = torch.randn(1, T, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    v = torch.randn(1, T, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    q = torch.randn(1, T, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    d_o = torch.randn(1, T, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    while secs < budget_s:
        hk = int(rng.integers(0, Hkv))
        tile = int(rng.integers(0, T // 128))
        rows = np.arange(tile * 128, tile * 128 + 128)
        t0 = time.perf_counter()
        orc.forward_rows(q, k, v, [ws[hk]], scale, 0, rows)
        orc.backward_dq_rows(q, k, v, d_o, [ws[hk]], scale, 0, rows)
        secs += time.perf_counter() - t0
        pairs = int(orc.visible_mask(T, T, ws[hk], rows).sum())
        flops += (4.0 + 6.0) * D * pairs
        units += 1
    return flops, secs, units


def oracle_decode_sample(reps=3):
    """Times the oracle's decode of one (sequence, KV head) of the 128K decode configuration: visible K/V bytes
    per second of host time (what the GPU path reports for the whole batch)."""
    import numpy as np
    import torch
    import cowa_inputs
    from oracle import cowa_oracle as orc
    c = cowa_inputs.CONFIGS[DECODE_CFG]
    D, G = c["D"], c["Hq"] // c["Hkv"]
    n_k = (c["len_lo"] + c["len_hi"]) // 2
    g = torch.Generator().manual_seed(c["index"] * 1000 + 9)
    kc = torch.randn(1, 1, n_k, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    vc = torch.randn(1, 1, n_k, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    qd = torch.randn(1, G, D, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    lens = np.array([n_k])
    win = orc.default_windows(n_k, c["Hkv"], c["sink"], c["local"])[3]
    vis = int(orc.visible_mask(1, n_k, win).sum())
    t0 = time.perf_counter()
    for _ in range(reps):
        orc.decode(qd, kc, vc, lens, c["sink"], c["local"], cowa_inputs.softmax_scale(D), h_k_global=c["Hkv"], hk_offset=3)
    dt = (time.perf_counter() - t0) / reps
    return vis * D * 2 * 2 / dt / 1e9, dt


def count_legal_pairs(T, windows):
    """Legal (query, key) pairs summed over the KV heads for N_q = N_k = T (accounting only: the
    second FLOP figure beside the visited-tile one).  Per query row the sink, band and near
    intervals of keys are clipped to the causal prefix and their union is measured."""
    import numpy as np
    iq = np.arange(T, dtype=np.int64)
    total = 0
    for s_, n_, g_, l_ in windows:
        near_lo = np.maximum(iq - n_ + 1, 0)                      # near: [near_lo, iq]
        band_lo = np.maximum(iq - (n_ + g_ + l_) + 1, 0)          # band: [band_lo, band_hi]
        band_hi = iq - (n_ + g_)
        band = np.where(l_ > 0, np.maximum(band_hi - band_lo + 1, 0), 0)
        sink_hi = np.minimum(s_ - 1, iq)                          # sink: [0, sink_hi]
        # the three intervals are ordered sink <= band <= near; subtract the overlaps of neighbours
        sink = np.maximum(sink_hi + 1, 0)
        top_of_lower = np.where(band > 0, band_hi, -1)
        near = iq - np.maximum(near_lo, np.maximum(top_of_lower, sink_hi) + 1) + 1
        band_eff = np.where(band > 0, np.maximum(band_hi - np.maximum(band_lo, sink_hi + 1) + 1, 0), 0)
        total += int(sink.sum() + band_eff.sum() + np.maximum(near, 0).sum())
    return total


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def workload_config(args, world):
    """The `config` object of the JSON line; both arms print the same one."""
    import cowa_inputs
    ct = cowa_inputs.CONFIGS[args.train_cfg]
    cd = cowa_inputs.CONFIGS[DECODE_CFG]
    return {"workload": args.train_cfg, "decode_workload": DECODE_CFG, "decode_batch": args.decode_batch or cd["B"],
            "B": ct["B"], "T": ct["T"], "Hq": ct["Hq"], "Hkv": ct["Hkv"], "D": ct["D"], "sink": ct["sink"], "near": ct["local"],
            "deterministic_dq": bool(args.deterministic), "windows": args.windows, "phases": ["fwd", "bwd", "decode"],
            "l2": "inputs larger than L2 (2.6 GB training tensors, 0.57 GB visible KV cache)",
            "parallelism": "independent replicas" if world > 1 else "single GPU"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy  # noqa: F401  (loads BLAS so that the thread count can be read)
    per_step = 6.0
    for _ in range(args.warmup):
        oracle_sample(0.5)
    flops, secs = 0.0, 0.0
    for s in range(args.steps):
        f, t, _ = oracle_sample(per_step, seed_tiles=s)
        flops, secs = flops + f, secs + t
    val = flops / secs / 1e12
    sample = (f"oracle forward + the backward terms of the same query rows (S, P, dP, dS, dQ; dK/dV not sampled) on "
              f"random (KV head, 128-row query tile) units of the 128K configuration, ~{per_step:.0f} s per step; "
              f"FLOPs as performed over legal pairs (10*D per pair)")
    line = {
        "impl": "reference", "metric": "cowa_train_tflops_visited_tiles_128k", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(argparse.Namespace(**{**vars(args), "train_cfg": TRAIN_CFG}), args.gpus), "config_note": "float64 CPU oracle, legal-pair FLOPs of the sampled tiles",
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# CUDA library
# ------------------------------------------------------------------------------------------

def run_cuda(args):
    import torch
    import cowa_inputs
    import paper_2609_32704_b200 as cowa

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", torch.cuda.current_device())
    peaks, peak_src = load_peaks()

    ct = cowa_inputs.CONFIGS[args.train_cfg]
    cd = dict(cowa_inputs.CONFIGS[DECODE_CFG])
    if args.decode_batch:
        cd["B"] = args.decode_batch
    B, T, Hq, Hkv, D = ct["B"], ct["T"], ct["Hq"], ct["Hkv"], ct["D"]
    scale = cowa_inputs.softmax_scale(D)
    train_windows = None
    if args.windows != "default":  # duplicated-window control: the first m bands repeated over the heads
        m = int(args.windows[3:])
        train_windows = duplicated_windows(cowa.cowa_default_windows(T, Hkv, 0, Hkv, ct["sink"], ct["local"]), m)
    p_train = cowa.make_params(sink=ct["sink"], local=ct["local"], softmax_scale=scale, windows=train_windows,
                               deterministic=args.deterministic)
    p_full = cowa.make_params(softmax_scale=scale, full_attn=True, deterministic=args.deterministic)
    p_dec = cowa.make_params(sink=cd["sink"], local=cd["local"], softmax_scale=scale)

    # ---- inputs resident in HBM ----
    q, k, v, d_o = cowa_inputs.make_train_inputs(ct["index"], B, T, Hq, Hkv, D, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, T), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws_bwd = torch.empty(max(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, p_train), 16), dtype=torch.uint8,
                         device=dev)
    qd, kc, vc, lens = cowa_inputs.make_decode_inputs(cd["index"], cd["B"], cd["Tmax"], cd["Hq"], cd["Hkv"], cd["D"],
                                                      cd["len_lo"], cd["len_hi"], device=dev)
    od = torch.empty_like(qd)
    lsed = torch.empty((cd["B"], cd["Hq"]), dtype=torch.float32, device=dev)
    ws_dec = torch.empty(cowa.cowa_decode_workspace_bytes(cd["B"], cd["Tmax"], cd["Hq"], cd["Hkv"], cd["D"], p_dec),
                         dtype=torch.uint8, device=dev)

    # ---- work counts ----
    cnt = cowa.cowa_tile_counts(T, T, Hkv, p_train)
    cnt_full = cowa.cowa_tile_counts(T, T, Hkv, p_full)
    G = Hq // Hkv
    legal_pairs = count_legal_pairs(T, train_windows or cowa.cowa_default_windows(T, Hkv, 0, Hkv, ct["sink"], ct["local"]))
    fwd_flops = cnt["visited"] * 128 * 128 * 4 * D * G * B
    bwd_flops = 2.5 * fwd_flops
    full_fwd_flops = cnt_full["visited"] * 128 * 128 * 4 * D * G * B
    lens_h = lens.cpu().tolist()
    vis_rows = 0
    for n in lens_h:
        for w_ in cowa.cowa_default_windows(n, cd["Hkv"], 0, cd["Hkv"], cd["sink"], cd["local"]):
            vis_rows += min(n, w_[0] + w_[1] + w_[3])
    dec_bytes = vis_rows * cd["D"] * 2 * 2

    have_bwd = True  # every phase is part of the step; a failing call raises
    cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, p_train, ws_bwd)
    torch.cuda.synchronize()

    main_evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    for pair in main_evs:
        for e_ in pair:
            e_.record()  # creates the underlying CUDA event

    def step(params, ev=None, main_ev=None):
        if ev: ev[0].record()
        cowa.cowa_fwd(q, k, v, o, lse, params)
        if ev: ev[1].record()
        if have_bwd:
            pb = cowa.with_bwd_events(params, main_ev[0], main_ev[1]) if main_ev else params
            cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, pb, ws_bwd)
        if ev: ev[2].record()
        cowa.cowa_decode(qd, kc, vc, lens, od, lsed, p_dec, ws_dec)
        if ev: ev[3].record()

    for _ in range(args.warmup):
        step(p_train)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(torch.cuda.current_device())
    if rank == 0:
        sampler.start()
    barrier(world)
    for s in range(args.steps):
        step(p_train, evs[s], main_evs[s])
    barrier(world)
    clocks = sampler.stop() if rank == 0 else None
    cowa.cowa_check_device_status()

    fwd_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    bwd_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    dec_ms = sum(e[2].elapsed_time(e[3]) for e in evs) / args.steps
    fwd_min = max_over_ranks(min(e[0].elapsed_time(e[1]) for e in evs), world)
    bwd_min = max_over_ranks(min(e[1].elapsed_time(e[2]) for e in evs), world)
    dec_min = max_over_ranks(min(e[2].elapsed_time(e[3]) for e in evs), world)
    total_ms = evs[0][0].elapsed_time(evs[-1][3]) / args.steps
    fwd_ms, bwd_ms, dec_ms, total_ms = (max_over_ranks(x, world) for x in (fwd_ms, bwd_ms, dec_ms, total_ms))

    # main backward kernel alone (the call also enqueues a memset, the preprocess and the dQ conversion)
    bwd_main_ms = None
    if have_bwd:
        bwd_main_ms = max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in main_evs) / args.steps, world)
    train_flops = fwd_flops + (bwd_flops if have_bwd else 0.0)
    train_ms = fwd_ms + (bwd_ms if have_bwd else 0.0)
    value = world * train_flops / (train_ms * 1e-3) / 1e12

    # ---- decode alone, calls queued back to back (no long kernel in front of it) ----
    eb = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    n_dec = 20
    barrier(world)
    eb[0].record()
    for _ in range(n_dec):
        cowa.cowa_decode(qd, kc, vc, lens, od, lsed, p_dec, ws_dec)
    eb[1].record()
    barrier(world)
    dec_b2b_ms = max_over_ranks(eb[0].elapsed_time(eb[1]) / n_dec, world)

    # ---- decode variants on the same cache: several newest tokens per call, paged cache ----
    dec_var = None
    if not args.no_varlen:
        def b2b(fn):
            for _ in range(3):
                fn()
            ev3 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev3[0].record()
            for _ in range(n_dec):
                fn()
            ev3[1].record()
            torch.cuda.synchronize()
            return max_over_ranks(ev3[0].elapsed_time(ev3[1]) / n_dec, world)

        dec_var = {}
        Bd, Hqd, Hkvd, Dd, Tm = cd["B"], cd["Hq"], cd["Hkv"], cd["D"], cd["Tmax"]
        for nq in (2, 4):
            qm = cowa_inputs.make_train_inputs(9, Bd, nq, Hqd, Hkvd, Dd, device=dev)[0].permute(0, 2, 1, 3).contiguous()
            om = torch.empty_like(qm)
            wsm = torch.empty(cowa.cowa_decode_multi_workspace_bytes(Bd, nq, Tm, Hqd, Hkvd, Dd, p_dec),
                              dtype=torch.uint8, device=dev)
            ms = b2b(lambda: cowa.cowa_decode_multi(qm, kc, vc, lens, om, None, p_dec, wsm))
            dec_var[f"multi_nq{nq}"] = {"us_per_call": ms * 1e3, "us_per_token": ms * 1e3 / (Bd * nq),
                                        "visible_kv_gbs": dec_bytes / (ms * 1e-3) / 1e9}
        ps = 64
        mp = Tm // ps
        perm = torch.randperm(Bd * mp, generator=torch.Generator().manual_seed(5)).to(dev)
        table = perm.view(Bd, mp).to(torch.int32).contiguous()
        def to_pages(x):
            pages = x.view(Bd, Hkvd, mp, ps, Dd).permute(0, 2, 1, 3, 4).reshape(Bd * mp, Hkvd, ps, Dd)
            out = torch.empty_like(pages)
            out[perm] = pages
            return out
        kp, vp = to_pages(kc), to_pages(vc)
        q1 = qd.view(Bd, 1, Hqd, Dd)
        o1 = torch.empty_like(q1)
        wsp = torch.empty(cowa.cowa_decode_multi_workspace_bytes(Bd, 1, Tm, Hqd, Hkvd, Dd, p_dec), dtype=torch.uint8,
                          device=dev)
        ms = b2b(lambda: cowa.cowa_decode_paged(q1, kp, vp, table, lens, o1, None, p_dec, wsp))
        dec_var[f"paged_{ps}"] = {"us_per_call": ms * 1e3, "visible_kv_gbs": dec_bytes / (ms * 1e-3) / 1e9,
                                  "max_abs_diff_vs_contiguous": float((o1.view_as(od).float() - od.float()).abs().max())}
        cowa.cowa_check_device_status()
        del kp, vp

    # ---- yardstick for the decode numbers: a plain streaming read of exactly as many bytes as the decode's
    # visible K/V rows (a library reduction over a buffer of that size), timed in the same two situations: right
    # behind a training backward, as inside the step, and back to back.  It shows what the GPU lets a pure read
    # of these bytes do in that state (SM clock under the power cap, dirty L2 lines left by the backward).
    yard = torch.ones(dec_bytes // 4, dtype=torch.float32, device=dev)
    for _ in range(3):
        yard.sum()
    ey = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(4)]
    for e_ in ey[:3]:
        cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, p_train, ws_bwd)
        e_[0].record(); yard.sum(); e_[1].record()
    ey[3][0].record()
    for _ in range(n_dec):
        yard.sum()
    ey[3][1].record()
    torch.cuda.synchronize()
    yard_step_ms = max_over_ranks(sum(e_[0].elapsed_time(e_[1]) for e_ in ey[:3]) / 3, world)
    yard_b2b_ms = max_over_ranks(ey[3][0].elapsed_time(ey[3][1]) / n_dec, world)
    del yard

    # ---- FullAttn path of the same library: the same step (forward, backward, decode in that order), one
    # warm-up step and three timed ones (it is ~5.4x the work), so that every ratio compares like with like ----
    full = {}
    if rank == 0 and not args.no_fullattn:
        ws_df = torch.empty(cowa.cowa_decode_workspace_bytes(cd["B"], cd["Tmax"], cd["Hq"], cd["Hkv"], cd["D"], p_full),
                            dtype=torch.uint8, device=dev)
        n_full = 3

        def full_step(ev=None):
            if ev: ev[0].record()
            cowa.cowa_fwd(q, k, v, o, lse, p_full)
            if ev: ev[1].record()
            cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, p_full, ws_bwd)
            if ev: ev[2].record()
            cowa.cowa_decode(qd, kc, vc, lens, od, lsed, p_full, ws_df)
            if ev: ev[3].record()

        full_step()
        torch.cuda.synchronize()
        fe = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_full)]
        for e_ in fe:
            full_step(e_)
        torch.cuda.synchronize()
        f_ms = sum(e_[0].elapsed_time(e_[1]) for e_ in fe) / n_full
        b_ms = sum(e_[1].elapsed_time(e_[2]) for e_ in fe) / n_full
        fd_step_ms = sum(e_[2].elapsed_time(e_[3]) for e_ in fe) / n_full
        e2 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for _ in range(2):
            cowa.cowa_decode(qd, kc, vc, lens, od, lsed, p_full, ws_df)
        e2[0].record()
        for _ in range(5):
            cowa.cowa_decode(qd, kc, vc, lens, od, lsed, p_full, ws_df)
        e2[1].record()
        torch.cuda.synchronize()
        fd_b2b_ms = e2[0].elapsed_time(e2[1]) / 5
        tile_ratio = cnt_full["visited"] / cnt["visited"]
        byte_ratio = sum(lens_h) * cd["Hkv"] / vis_rows
        # the bar of the speed-up criterion: CoWA time <= FullAttn time x (visited / causal work) x 1.2
        full = {"fullattn_iterations": n_full,
                "fullattn_fwd_ms": f_ms, "fullattn_fwd_tflops": full_fwd_flops / f_ms / 1e9,
                "fullattn_bwd_ms": b_ms, "fullattn_bwd_tflops": 2.5 * full_fwd_flops / b_ms / 1e9,
                "speedup_fwd": f_ms / fwd_ms, "speedup_bwd": b_ms / bwd_ms, "work_ratio_tiles": tile_ratio,
                "bar_fwd_ms": 1.2 * f_ms / tile_ratio, "bar_bwd_ms": 1.2 * b_ms / tile_ratio,
                "meets_bar_fwd": fwd_ms <= 1.2 * f_ms / tile_ratio, "meets_bar_bwd": bwd_ms <= 1.2 * b_ms / tile_ratio,
                "fullattn_decode_us_in_step": fd_step_ms * 1e3, "fullattn_decode_us_back_to_back": fd_b2b_ms * 1e3,
                "speedup_decode_in_step": fd_step_ms / dec_ms, "speedup_decode_back_to_back": fd_b2b_ms / dec_b2b_ms,
                "byte_ratio_decode": byte_ratio,
                "bar_decode_us_in_step": 1.2e3 * fd_step_ms / byte_ratio,
                "bar_decode_us_back_to_back": 1.2e3 * fd_b2b_ms / byte_ratio,
                "meets_bar_decode_in_step": dec_ms <= 1.2 * fd_step_ms / byte_ratio,
                "meets_bar_decode_back_to_back": dec_b2b_ms <= 1.2 * fd_b2b_ms / byte_ratio}
        del ws_df

    # ---- prefill over a packed batch of mixed lengths (one launch) against one call per sequence ----
    varlen = None
    if not args.no_varlen:
        mix = [65536, 32768, 16384, 16384, 8192, 8192, 4096, 2048, 1000, 333]  # N_q = N_k per sequence
        tot = sum(mix)
        pq, pk, pv, _ = cowa_inputs.make_train_inputs(7, 1, tot, Hq, Hkv, D, device=dev)
        pq, pk, pv = pq[0], pk[0], pv[0]
        po = torch.empty_like(pq)
        plse = torch.empty((Hq, tot), dtype=torch.float32, device=dev)
        cu = torch.tensor([0] + list(itertools.accumulate(mix)), dtype=torch.int32, device=dev)
        p_mix = cowa.make_params(sink=ct["sink"], local=ct["local"], softmax_scale=scale)
        v_flops = sum(cowa.cowa_tile_counts(n, n, Hkv, p_mix)["visited"] for n in mix) * 128 * 128 * 4 * D * G

        def packed():
            cowa.cowa_prefill_varlen(pq, pk, pv, po, plse, cu, cu, p_mix)

        def one_by_one():
            a0 = 0
            for n in mix:
                # a sequence's rows are not contiguous per head inside the packed tensors: time on copies
                cowa.cowa_prefill(seq_q[a0], seq_k[a0], seq_v[a0], seq_o[a0], seq_l[a0], p_mix)
                a0 += n

        seq_q, seq_k, seq_v, seq_o, seq_l = {}, {}, {}, {}, {}
        a0 = 0
        for n in mix:
            seq_q[a0] = pq[:, a0:a0 + n].contiguous()[None]
            seq_k[a0] = pk[:, a0:a0 + n].contiguous()[None]
            seq_v[a0] = pv[:, a0:a0 + n].contiguous()[None]
            seq_o[a0] = torch.empty_like(seq_q[a0])
            seq_l[a0] = torch.empty((1, Hq, n), dtype=torch.float32, device=dev)
            a0 += n
        times = {}
        for name, fn in (("packed", packed), ("one_by_one", one_by_one)):
            for _ in range(2):
                fn()
            ev2 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev2[0].record()
            for _ in range(5):
                fn()
            ev2[1].record()
            torch.cuda.synchronize()
            times[name] = max_over_ranks(ev2[0].elapsed_time(ev2[1]) / 5, world)
        cowa.cowa_check_device_status()
        varlen = {"lengths": mix, "ms": times["packed"], "tflops": v_flops / times["packed"] / 1e9,
                  "one_call_per_sequence_ms": times["one_by_one"]}
        del seq_q, seq_k, seq_v, seq_o, seq_l
        if have_bwd:  # backward over the same packed batch (N_q = N_k per sequence)
            pdo = cowa_inputs.make_train_inputs(8, 1, tot, Hq, Hkv, D, device=dev)[3][0]
            pdq, pdk, pdv = torch.empty_like(pq), torch.empty_like(pk), torch.empty_like(pv)
            wsv = torch.empty(cowa.cowa_bwd_varlen_workspace_bytes(len(mix), tot, Hq, Hkv, D, p_mix), dtype=torch.uint8,
                              device=dev)
            fn = lambda: cowa.cowa_bwd_varlen(pq, pk, pv, po, plse, pdo, pdq, pdk, pdv, cu, p_mix, wsv)
            for _ in range(2):
                fn()
            ev2 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev2[0].record()
            for _ in range(3):
                fn()
            ev2[1].record()
            torch.cuda.synchronize()
            cowa.cowa_check_device_status()
            b_ms = max_over_ranks(ev2[0].elapsed_time(ev2[1]) / 3, world)
            varlen.update({"bwd_ms": b_ms, "bwd_tflops": 2.5 * v_flops / b_ms / 1e9})
            del pdo, pdq, pdk, pdv, wsv
        del pq, pk, pv, po, plse

    # ---- the other training configurations beside FullAttn, and the slowest TP=8 shard at 128K ----
    table, tp_row = None, None
    if rank == 0 and not args.no_table:
        table = [train_config_row(cowa, cowa_inputs, name, mode, dev)
                 for name, mode in (("tiny", "default"), ("8k", "default"), ("8k", "dup1"), ("32k", "default"))]
        tp_row = tp_replica_rows(cowa, cowa_inputs, dev, [131072], 0, 1, 3, 3)[0]
        tp_row["note"] = ("TP=8 shards of the paper's benchmark shape (Hq=64, Hkv=8, D=128, sink+near=128+896), timed "
                          "one after another on this GPU; slowest shard per phase")

    # ---- end to end: host buffers in, results back to the host, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        hq, hk_, hv, hdo = (x.cpu().pin_memory() for x in (q, k, v, d_o))
        ho = torch.empty_like(hq).pin_memory()
        hlse = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        hdq, hdk, hdv = (torch.empty_like(x).pin_memory() for x in (hq, hk_, hv))
        # decode step of the same pass: the query tokens come from the host and the outputs go back; the KV
        # cache stays resident, as it does in a serving loop
        hqd = qd.cpu().pin_memory()
        hod = torch.empty_like(hqd).pin_memory()
        qd2 = [torch.empty_like(qd) for _ in range(2)]
        od2 = [torch.empty_like(od) for _ in range(2)]
        h2d = sum(x.numel() * x.element_size() for x in (hq, hk_, hv, hdo, hqd))
        d2h = sum(x.numel() * x.element_size() for x in (ho, hlse, hdq, hdk, hdv, hod))

        # Three streams (inputs, compute, results) and two sets of device buffers: PCIe is full duplex, and
        # as in a training loop that prefetches its next batch, the inputs of step s+1 come in while step s
        # computes and the results of step s leave while step s+1 computes.  Every step's copies are issued
        # and finished inside the timed region (the closing event waits for all three streams); the first
        # step's input copy and the last step's result copy have nothing to hide behind and are paid in full.
        s_main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        sets = [dict(q=q, k=k, v=v, d_o=d_o, o=o, lse=lse, dq=dq, dk=dk, dv=dv)]
        sets.append({n_: torch.empty_like(t_) for n_, t_ in sets[0].items()})

        def e2e_run(n_steps):
            computed = [None, None]   # event: the compute that last used buffer set i has finished
            drained = [None, None]    # event: the results of that compute have reached the host
            s_in.wait_stream(s_main); s_out.wait_stream(s_main)
            for s_ in range(n_steps):
                d = sets[s_ & 1]
                ev_qkv, ev_do, ev_fwd, ev_bwd = (torch.cuda.Event() for _ in range(4))
                with torch.cuda.stream(s_in):
                    if computed[s_ & 1] is not None:
                        s_in.wait_event(computed[s_ & 1]); s_in.wait_event(drained[s_ & 1])
                    # the decode step's query tokens first: 64 KB that must not queue behind gigabytes on the copy engine
                    qd2[s_ & 1].copy_(hqd, non_blocking=True)
                    d["q"].copy_(hq, non_blocking=True); d["k"].copy_(hk_, non_blocking=True)
                    d["v"].copy_(hv, non_blocking=True)
                    ev_qkv.record()
                    if have_bwd:
                        d["d_o"].copy_(hdo, non_blocking=True)
                        ev_do.record()
                s_main.wait_event(ev_qkv)
                cowa.cowa_fwd(d["q"], d["k"], d["v"], d["o"], d["lse"], p_train)
                ev_fwd.record()
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_fwd)
                    ho.copy_(d["o"], non_blocking=True); hlse.copy_(d["lse"], non_blocking=True)
                if have_bwd:
                    s_main.wait_event(ev_do)
                    cowa.cowa_bwd(d["q"], d["k"], d["v"], d["o"], d["lse"], d["d_o"], d["dq"], d["dk"], d["dv"],
                                  p_train, ws_bwd)
                    ev_bwd.record()
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(ev_bwd)
                        hdq.copy_(d["dq"], non_blocking=True); hdk.copy_(d["dk"], non_blocking=True)
                        hdv.copy_(d["dv"], non_blocking=True)
                # decode on the resident cache; its 64 KB of output leave on the result stream with the gradients
                cowa.cowa_decode(qd2[s_ & 1], kc, vc, lens, od2[s_ & 1], lsed, p_dec, ws_dec)
                ev_step = torch.cuda.Event()
                ev_step.record()
                computed[s_ & 1] = ev_step
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_step)
                    hod.copy_(od2[s_ & 1], non_blocking=True)
                    drained[s_ & 1] = torch.cuda.Event()
                    drained[s_ & 1].record()
            s_main.wait_stream(s_in); s_main.wait_stream(s_out)

        e2e_run(2)
        barrier(world)
        n_e2e = max(2, min(args.steps, 50))  # the timed steps of the device-resident measurement, as far as a bound allows
        ee = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        ee[0].record()
        e2e_run(n_e2e)
        ee[1].record()
        barrier(world)
        e_ms = max_over_ranks(ee[0].elapsed_time(ee[1]) / n_e2e, world)
        e2e = {"value": world * train_flops / (e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "phases": ["fwd", "bwd", "decode"],
               "note": "value = forward + backward FLOPs over the whole step time, decode step and all copies included"}
        del hq, hk_, hv, hdo, ho, hlse, hdq, hdk, hdv, sets, hqd, hod, qd2, od2

    if rank != 0:
        return

    # ---- roofline of the dominant kernel ----
    k_fwd, k_bwd, k_dec = f"cowa_fwd_kernel<{D}, 0>", f"cowa_bwd_kernel<{D}, 0>", f"cowa_decode_split_kernel<{cd['D']}, {cd['Hq'] // cd['Hkv']}, 0>"
    if bwd_ms >= fwd_ms:
        dom, dom_flops, dom_ms = k_bwd, bwd_flops, bwd_main_ms
    else:
        dom, dom_flops, dom_ms = k_fwd, fwd_flops, fwd_ms
    peak_tf = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    achieved = dom_flops / dom_ms / 1e9
    # DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of an ncu capture) come from the
    # tracked summary profiles/traffic.json, keyed by kernel name and workload; no entry, no number.
    traffic = load_traffic()
    wl = args.train_cfg if args.windows == "default" else None
    roofline = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": achieved / peak_tf, "peak_source": f"{peak_src} bf16 sustained (kernel timed inside a long step)",
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0,
                "traffic": traffic_for(traffic, dom, wl),
                "traffic_unit": "bytes per launch (ncu; see profiles/traffic.json for the capture it comes from)"}
    dec_gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
    b2b_gbs = dec_bytes / (dec_b2b_ms * 1e-3) / 1e9
    decode = {"us_per_step": dec_ms * 1e3, "us_per_token": dec_ms * 1e3 / cd["B"], "visible_kv_bytes": dec_bytes,
              "achieved_gbs": dec_gbs, "hbm_peak_gbs": peaks["hbm_gbs"], "frac_hbm": dec_gbs / peaks["hbm_gbs"],
              "frac_nominal_8tbs": dec_gbs / 8000.0, "us_per_step_min": dec_min * 1e3,
              "back_to_back": {"us_per_call": dec_b2b_ms * 1e3, "achieved_gbs": b2b_gbs,
                               "frac_hbm": b2b_gbs / peaks["hbm_gbs"], "frac_nominal_8tbs": b2b_gbs / 8000.0,
                               "calls": n_dec},
              "plain_read_of_same_bytes": {"after_backward_us": yard_step_ms * 1e3, "back_to_back_us": yard_b2b_ms * 1e3,
                                           "decode_over_read_in_step": dec_ms / yard_step_ms,
                                           "decode_over_read_back_to_back": dec_b2b_ms / yard_b2b_ms,
                                           "what": "torch.sum over a float32 buffer of visible_kv_bytes"}}

    cpu = None
    if not args.no_cpu_baseline and world == 1:  # the oracle is timed on one-GPU runs only
        f, t, units = oracle_sample(args.cpu_seconds)
        dec_gbs_cpu, dec_s_cpu = oracle_decode_sample()
        cpu = {"value": f / t / 1e12, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle",
               "sample": f"oracle forward + the backward terms of the same query rows (S, P, dP, dS, dQ; dK/dV sums run "
                         f"over all query rows and are not sampled) of {units} random (KV head, 128-row query tile) units "
                         f"of the 128K configuration, {t:.1f} s; FLOPs as performed over legal pairs (10*D per pair)",
               "decode": {"value": dec_gbs_cpu, "unit": "GB/s of visible K/V", "seconds_per_sequence_and_kv_head": dec_s_cpu,
                          "sample": "oracle decode of one (sequence, KV head) of the 128K decode configuration"}}

    line = {
        "metric": "cowa_train_tflops_visited_tiles_" + args.train_cfg, "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(args, world),
        "fwd_ms": fwd_ms, "fwd_ms_min": fwd_min, "fwd_tflops": fwd_flops / fwd_ms / 1e9,
        "fwd_tflops_legal_pairs": legal_pairs * 4 * D * G * B / fwd_ms / 1e9,
        "bwd_ms_min": bwd_min if have_bwd else None,
        "bwd_tflops_legal_pairs": legal_pairs * 10 * D * G * B / bwd_ms / 1e9 if have_bwd else None,
        "bwd_ms": bwd_ms if have_bwd else None, "bwd_tflops": bwd_flops / bwd_ms / 1e9 if have_bwd else None,
        "bwd_main_kernel_ms": bwd_main_ms,
        "visited_tiles": cnt["visited"], "causal_tiles": cnt["causal"],
        "decode": decode, "prefill_varlen": varlen, "decode_variants": dec_var, "roofline": roofline,
        "roofline_other_kernels": [
            {"kernel": k_fwd, "bound": "tensor", "achieved": fwd_flops / fwd_ms / 1e9, "peak": peak_tf,
             "unit": "TFLOP/s", "frac": fwd_flops / fwd_ms / 1e9 / peak_tf,
             "frac_of_burst_peak": fwd_flops / fwd_ms / 1e9 / peaks["bf16_tflops"],
             "traffic": traffic_for(traffic, k_fwd, wl)},
            {"kernel": k_dec + " + merge", "bound": "hbm", "achieved": b2b_gbs,
             "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": b2b_gbs / peaks["hbm_gbs"],
             "frac_nominal_8tbs": b2b_gbs / 8000.0,
             "traffic": traffic_for(traffic, k_dec, DECODE_CFG if not args.decode_batch else None)}],
        "configs_table": table, "tp_replica": tp_row, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": args.steps * (1 + (BWD_LAUNCHES if have_bwd else 0) + 2),
    }
    line.update(full)
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# The paper's operator benchmark re-staged: TP=8 shards of Hq=64, Hkv=8, D=128, batch 1
# ------------------------------------------------------------------------------------------

# Latency table of the paper (8 x H100, TP=8), ms: T -> (FullAttn fwd, CoWA fwd, FullAttn bwd, CoWA bwd,
# FullAttn decode, CoWA decode).  Context for the reader, never a target.
PAPER_TP8_MS = {
    1024: (0.015, 0.015, 0.055, 0.041, 0.003, 0.003), 2048: (0.043, 0.040, 0.149, 0.106, 0.004, 0.003),
    4096: (0.153, 0.098, 0.468, 0.253, 0.007, 0.004), 8192: (0.572, 0.237, 1.699, 0.600, 0.009, 0.004),
    16384: (2.179, 0.616, 6.455, 1.564, 0.012, 0.005), 32768: (8.570, 1.807, 24.449, 4.358, 0.018, 0.006),
    65536: (36.431, 5.573, 99.664, 14.150, 0.027, 0.009), 131072: (159.987, 21.758, 441.230, 51.509, 0.045, 0.015),
}


def timed_ms(torch, fn, warmup, iters, flush=None):
    for _ in range(warmup):
        fn()
    tot = 0.0
    for _ in range(iters):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1)
    return tot / iters


def train_config_row(cowa, cowa_inputs, name, mode, dev, warmup=2, iters=5):
    """Forward and backward of one training configuration, CoWA (or the duplicated-window control) beside
    FullAttn at the same shape: ms, speed-up, and the visited / causal tile ratio the speed-up is held against."""
    import torch
    c = cowa_inputs.CONFIGS[name]
    B, T, Hq, Hkv, D = c["B"], c["T"], c["Hq"], c["Hkv"], c["D"]
    scale = cowa_inputs.softmax_scale(D)
    wins = None
    if mode != "default":
        wins = duplicated_windows(cowa.cowa_default_windows(T, Hkv, 0, Hkv, c["sink"], c["local"]), int(mode[3:]))
    p = cowa.make_params(sink=c["sink"], local=c["local"], softmax_scale=scale, windows=wins)
    pf = cowa.make_params(softmax_scale=scale, full_attn=True)
    q, k, v, d_o = cowa_inputs.make_train_inputs(c["index"], B, T, Hq, Hkv, D, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, T), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(max(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, p), cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, pf), 16),
                     dtype=torch.uint8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if q.numel() * 2 < (128 << 20) else None
    row = {"config": name, "windows": mode, "B": B, "T": T, "Hq": Hq, "Hkv": Hkv, "D": D,
           "l2": "flushed before every timed call" if flush is not None else "inputs larger than L2"}
    cnt, cntf = cowa.cowa_tile_counts(T, T, Hkv, p), cowa.cowa_tile_counts(T, T, Hkv, pf)
    flops = cnt["visited"] * 128 * 128 * 4 * D * (Hq // Hkv) * B
    for tag, par in (("cowa", p), ("fullattn", pf)):
        row[tag + "_fwd_ms"] = timed_ms(torch, lambda: cowa.cowa_fwd(q, k, v, o, lse, par), warmup, iters, flush)
        row[tag + "_bwd_ms"] = timed_ms(torch, lambda: cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, par, ws), warmup, iters, flush)
    cowa.cowa_check_device_status()
    row.update({"fwd_tflops": flops / row["cowa_fwd_ms"] / 1e9, "bwd_tflops": 2.5 * flops / row["cowa_bwd_ms"] / 1e9,
                "speedup_fwd": row["fullattn_fwd_ms"] / row["cowa_fwd_ms"],
                "speedup_bwd": row["fullattn_bwd_ms"] / row["cowa_bwd_ms"],
                "tile_ratio": cntf["visited"] / cnt["visited"], "visited_tiles": cnt["visited"], "causal_tiles": cnt["causal"],
                "iterations": iters})
    return row


def tp_replica_rows(cowa, cowa_inputs, dev, lengths, rank, world, warmup, iters):
    """Per sequence length: the slowest TP=8 shard per phase and layout among the shards this process owns."""
    import torch
    TP, Hq_r, D, sink, near = 8, 8, 128, 128, 896
    scale = cowa_inputs.softmax_scale(D)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for _ in range(500):  # ~50 ms of memory traffic: the first microsecond-scale calls must not meet an idle GPU's clocks
        flush.fill_(1)
    rows = []
    for T in lengths:
        q, k, v, d_o = cowa_inputs.make_train_inputs(11, 1, T, Hq_r, 1, D, device=dev)
        o = torch.empty_like(q)
        lse = torch.empty((1, Hq_r, T), dtype=torch.float32, device=dev)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        qd, od = q[:, :, -1].contiguous(), torch.empty((1, Hq_r, D), dtype=torch.bfloat16, device=dev)
        lsed = torch.empty((1, Hq_r), dtype=torch.float32, device=dev)
        lens = torch.tensor([T], dtype=torch.int32, device=dev)
        worst = {}
        for layout in ("cowa", "eq", "full"):  # default equal-width bands, equal-area bands, dense
            for r in tp_shards(rank, world, TP):
                if layout == "eq":
                    p = cowa.make_params(windows=cowa.cowa_equal_area_windows(T, T, TP, r, 1, sink, near),
                                         softmax_scale=scale)
                else:
                    p = cowa.make_params(sink=sink, local=near, softmax_scale=scale, full_attn=(layout == "full"),
                                         hkv_global=TP, hkv_offset=r)
                ws = torch.empty(max(cowa.cowa_bwd_workspace_bytes(1, T, Hq_r, 1, D, p), 16), dtype=torch.uint8,
                                 device=dev)
                wsd = torch.empty(max(cowa.cowa_decode_workspace_bytes(1, T, Hq_r, 1, D, p), 16), dtype=torch.uint8,
                                  device=dev)
                t = {"fwd": timed_ms(torch, lambda: cowa.cowa_fwd(q, k, v, o, lse, p), warmup, iters, flush),
                     "bwd": timed_ms(torch, lambda: cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, p, ws), warmup, iters, flush)}
                if layout != "eq":  # decode keeps the equal-width rule (Sec. 2.1), so there is no third variant
                    t["dec"] = timed_ms(torch, lambda: cowa.cowa_decode(qd, k, v, lens, od, lsed, p, wsd), warmup, iters, flush)
                for ph, ms in t.items():
                    key = layout + "_" + ph
                    worst[key] = max(worst.get(key, 0.0), ms)
                if layout == "full":
                    break  # dense shards are identical on every rank
        cowa.cowa_check_device_status()
        rows.append({"T": T, **{k_ + "_ms": v_ for k_, v_ in sorted(worst.items())}})
        del q, k, v, d_o, o, lse, dq, dk, dv
    return rows


def reduce_worst(rows, world):
    """Slowest shard over all ranks, per phase (every rank passes the rows of its own shards)."""
    return [{k_: (max_over_ranks(v_, world) if k_.endswith("_ms") else v_) for k_, v_ in sorted(r.items())} for r in rows]


def run_tp_replica(args):
    """Each rank of a TP=8 group owns one KV head and its 8 QO heads and runs the operator on its
    shard without any exchange; the group's latency is the slowest rank's.  With fewer than 8 GPUs
    the shards are timed one after another on the GPUs at hand (rank r takes shards r, r+world, ...):
    every launch is exactly what that rank's GPU would run.  L2 is flushed before every timed call."""
    import torch
    import cowa_inputs
    import paper_2609_32704_b200 as cowa

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    rank, world, _ = dist_setup(args.gpus)
    dev = torch.device("cuda", torch.cuda.current_device())
    iters, warm = max(args.steps, 3), max(args.warmup, 3)
    rows = reduce_worst(tp_replica_rows(cowa, cowa_inputs, dev, sorted(PAPER_TP8_MS), rank, world, warm, iters), world)
    for r in rows:
        pf, pc, pfb, pcb, pfd, pcd = PAPER_TP8_MS[r["T"]]
        r.update({"speedup_fwd": r["full_fwd_ms"] / r["cowa_fwd_ms"], "speedup_bwd": r["full_bwd_ms"] / r["cowa_bwd_ms"],
                  "speedup_fwd_equal_area": r["full_fwd_ms"] / r["eq_fwd_ms"],
                  "speedup_bwd_equal_area": r["full_bwd_ms"] / r["eq_bwd_ms"],
                  "speedup_dec": r["full_dec_ms"] / r["cowa_dec_ms"],
                  "paper_h100_ms": {"full_fwd": pf, "cowa_fwd": pc, "full_bwd": pfb, "cowa_bwd": pcb,
                                    "full_dec": pfd, "cowa_dec": pcd}})
    if rank != 0:
        return
    last = rows[-1]
    print(json.dumps({
        "metric": "cowa_tp8_shard_fwd_bwd_ms_128k", "value": last["cowa_fwd_ms"] + last["cowa_bwd_ms"], "unit": "ms",
        "n_gpus": world, "steps": iters, "warmup": warm, "higher_is_better": False,
        "scaling": "strong", "vs_baseline": (last["cowa_fwd_ms"] + last["cowa_bwd_ms"]) / (21.758 + 51.509),
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "TP=8 shards of B=1, Hq=64, Hkv=8, D=128, sink+near=128+896, T=1K..128K",
                   "shards_per_gpu": 8 // world if world <= 8 else 1, "l2": "flushed before every timed call",
                   "latency": "slowest shard (max over the 8 ranks' launches)"},
        "rows": rows}))


BWD_LAUNCHES = 3  # preprocess, main kernel, dq conversion


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-fullattn", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-varlen", action="store_true")
    ap.add_argument("--tp-replica", action="store_true",
                    help="time the TP=8 shards of the paper's operator benchmark shape instead of the default step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-table", action="store_true",
                    help="skip the rows of the other configurations (tiny, 8K, 8K control, 32K) and the TP=8 shard row")
    ap.add_argument("--windows", default="default", choices=["default", "dup1", "dup2"],
                    help="dup<m>: duplicated-window control, the first m bands repeated over the KV heads")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--train-cfg", default=TRAIN_CFG, choices=["tiny", "8k", "32k", "128k"],
                    help="training configuration (default: the 128K headline; smaller ones are for profiling)")
    ap.add_argument("--decode-batch", type=int, default=0, help="override the decode batch (profiling)")
    ap.add_argument("--deterministic", action="store_true",
                    help="backward with fixed-point dQ accumulation (bitwise reproducible dQ)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.tp_replica:
        run_tp_replica(args)
    else:
        run_cuda(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
