#!/usr/bin/env python
"""Benchmark of one Slim-DP communication round on B200.

A step is one whole round (score, select, K x explore, K x pack, merge,
K x pull) over the VGG-16-shaped synthetic workload, every step a C-ABI call
sequence of the CUDA library.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

N > 1 (under torchrun): the round does not shard (K workers are buffers on one
GPU, there is no exchange step), so every rank runs an independent replica of
the same workload; value = N * params / max-over-ranks time ("weak").
--impl reference times the CPU oracle on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "Gparams/s per Slim-DP round (score+select+pack+merge) and % of HBM roofline"
UNIT = "Gparams/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
CPU_BASELINE_SAMPLE = 1 << 25      # leading parameters of the workload for the cpu_baseline leg
REFERENCE_BUDGET_S = 120.0         # wall-clock target of a whole --impl reference run


# ------------------------------------------------------------ byte model ---

def model_bytes(N: int, K: int, k_core: int, k_exp: int) -> dict:
    """Algorithmic bytes per step: every input element the method must examine
    read once, every output written once, gathers / scatters at 4 B per element."""
    m = k_core + k_exp
    b = {
        "score": 4 * N * (K + 1) + 4 * N,
        "select": 4 * N + 4 * k_core + N // 8,
        "explore": K * (N // 8 + 4 * k_exp),
        "pack": K * 12 * m,
        "merge": 4 * k_core + 8 * k_core + 4 * K * k_core + K * 16 * k_exp,
        "pull": K * 12 * m,
    }
    b["round"] = sum(b.values())
    b["round_without_score"] = b["round"] - b["score"]
    # what the one-call round must move: the scores are neither written (4N) nor read back by the selection (4N)
    b["round_fused"] = b["round"] - 8 * N
    return b


def fused_pass_kernel_name(K: int, staging: bool):
    """Which kernel slimdp_round's pass over all parameters is for K workers (the library's own rule:
    a ring of 2..8 stages of 8 x (K + 1) x 512 bytes within 112 KB, or two stages within 160 KB;
    K = 4 and K = 8 have instantiations of their own).  None: the round does not fuse for this K."""
    stage = 8 * (K + 1) * 512
    stages = (112 * 1024) // stage
    if stages < 2 and 2 * stage <= 160 * 1024:
        stages = 2
    stages = min(stages, 8)
    if stages < 2 or stages * stage < 64 * 1024:
        return None
    kt = K if (K, stages) in ((8, 3), (4, 5)) else 0
    return f"score_bracket_async_kernel<{stages}, {kt}, {'true' if staging else 'false'}>"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "MEASURED_PEAKS.json hbm_gbs (of measured)"
    except Exception:
        return FALLBACK_HBM_GBS, "profiling-recipe fallback 6.65 TB/s (of fallback)"


# --------------------------------------------------------- clock sampling ---

_REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
            0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, torch_device_index: int, period_s: float = 0.01):
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.handle = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_device_index).uuid)
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = int(vis.split(",")[torch_device_index]) if vis else torch_device_index
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.handle = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                for bit, name in _REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.handle is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self) -> dict:
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------- multi-rank glue ---

def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value_ms: float, world: int, device=None) -> float:
    """Max of a per-rank duration over all ranks (the job is as slow as its slowest replica)."""
    if world == 1:
        return value_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([value_ms], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(params_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job Gparams/s: all ranks' parameters over the slowest rank's step time."""
    return params_per_rank * world / (ms_per_step * 1e-3) / 1e9


# ------------------------------------------------------------ CPU oracle ---

def time_oracle(cfg, n_sample: int, steps: int, warmup: int):
    import oracle
    from workloads import all_inputs, scaled_config
    sample = scaled_config(cfg, n_sample) if n_sample < cfg.N else cfg
    w, gs = all_inputs(sample)
    times = []
    for s in range(warmup + steps):
        t0 = time.perf_counter()
        r = oracle.run_round(w, gs, sample.c, sample.k_core, sample.k_exp, sample.seed, s, sample.eta)
        dt = time.perf_counter() - t0
        w = r["w"]
        if s >= warmup:
            times.append(dt)
    return sample, times


def oracle_round_threaded(w, gs, c, k_core, k_exp, seed, rnd, eta, threads: int):
    """The oracle's round with its loops spread over host threads, the "multi-thread scanning" of
    Section 3.5: scoring over index chunks, explorers / extraction / pull over workers.  The sort of
    the selection and the worker-ordered merge stay serial.  Same results as oracle.run_round."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    import oracle
    n, K = w.size, len(gs)
    cuts = [n * i // threads for i in range(threads + 1)]
    S = np.empty(n, np.float32)

    def score_chunk(i):
        a, b = cuts[i], cuts[i + 1]
        if b > a:
            S[a:b] = oracle.score(w[a:b], [g[a:b] for g in gs], c)

    with ThreadPoolExecutor(max_workers=threads) as pool:
        list(pool.map(score_chunk, range(threads)))
        core = oracle.select_core(S, k_core)
        exp = list(pool.map(lambda k: oracle.sample_explore(core, n, k_exp, seed, k, rnd), range(K)))
        val = list(pool.map(lambda k: oracle.pack(gs[k], core, exp[k]), range(K)))
        merged = oracle.merge(w, core, exp, val, eta)
        pulled = list(pool.map(lambda k: oracle.pull(merged, core, exp[k]), range(K)))
    return {"scores": S, "core_idx": core, "exp_idx": exp, "val": val, "w": merged, "pulled": pulled}


def time_oracle_threaded(cfg, n_sample: int, threads: int):
    from workloads import all_inputs, scaled_config
    sample = scaled_config(cfg, n_sample) if n_sample < cfg.N else cfg
    w, gs = all_inputs(sample)
    t0 = time.perf_counter()
    oracle_round_threaded(w, gs, sample.c, sample.k_core, sample.k_exp, sample.seed, 0, sample.eta, threads)
    return sample, time.perf_counter() - t0


def dominant_traffic(kernel: str, n: int):
    """DRAM bytes of one launch of `kernel` over n parameters, from the tracked summary of its ncu
    capture (bytes per parameter on a small case; traffic grows in proportion to n).  None when the
    summary is for another kernel: counters of a kernel that has changed since are not reported."""
    path = os.path.join(ROOT, "profiles", "dominant_kernel_traffic.txt")
    try:
        with open(path) as f:
            for line in f:
                if line.startswith("#") or not line.strip():
                    continue
                name, per_param, date = [x.strip() for x in line.split("|")][:3]
                if name == kernel:
                    return {"bytes": int(float(per_param) * n), "bytes_per_parameter": float(per_param),
                            "captured": date, "source": "profiles/dominant_kernel_traffic.txt"}
    except Exception:
        pass
    return None


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from workloads import CONFIGS
    cfg = CONFIGS[args.config]
    # size the per-step sample from a short probe so that warmup + steps rounds fit the budget
    probe, probe_t = time_oracle(cfg, 1 << 20, 1, 0)
    per_step = REFERENCE_BUDGET_S / (args.steps + args.warmup)
    n_sample = 1 << 16
    while n_sample * 2 <= min(cfg.N, 1 << 25) and (n_sample * 2) * 1.3 * probe_t[0] / probe.N <= per_step:
        n_sample *= 2
    sample, times = time_oracle(cfg, n_sample, args.steps, args.warmup)
    ms = 1e3 * sum(times) / len(times)
    value = sample.N / (ms * 1e-3) / 1e9
    desc = (f"leading {sample.N} parameters of the {cfg.name}-shaped workload (K={sample.K}, "
            f"k_core={sample.k_core}, k_exp={sample.k_exp}), one oracle round per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ ours ---

def timed_rounds(P, torch, cfg, w, grads, buf, steps: int, warmup: int, t0: int, flush=None, mark=True):
    """`steps` one-call rounds after `warmup` untimed ones, device-timed.  Returns the time of the whole
    timed region, every step's own time (between events recorded on the caller's stream after each
    round), the pass's times (events the library records around its dominant kernel) and the next round
    index.  flush: a buffer larger than L2 that is overwritten before every timed round; its time is
    not counted (each round is then bracketed by its own pair of events)."""
    def one_round(t):
        P.slimdp_round(w, grads, cfg.c, cfg.seed, t, cfg.eta, buf.scores, buf.core_idx, buf.core_aux, buf.exp_idx,
                       buf.val, buf.pulled, buf.select_ws, buf.explore_ws, buf.stage)
    t = t0
    for _ in range(warmup):
        one_round(t)
        t += 1
    torch.cuda.synchronize()
    P.read_status(buf.select_ws)
    P.read_status(buf.explore_ws)
    new_ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = [(new_ev(), new_ev()) for _ in range(steps)]
    for a, b in marks:      # torch creates the CUDA event at the first record
        a.record()
        b.record()
    begins = [new_ev() for _ in range(steps)]
    ends = [new_ev() for _ in range(steps)]
    ev_start, ev_end = new_ev(), new_ev()
    torch.cuda.synchronize()
    ev_start.record()
    for s in range(steps):
        if flush is not None:
            flush.zero_()
        begins[s].record()
        if mark:
            P.mark_dominant_kernel(marks[s][0], marks[s][1])
        one_round(t)
        ends[s].record()
        t += 1
    ev_end.record()
    torch.cuda.synchronize()
    P.read_status(buf.select_ws)
    P.read_status(buf.explore_ws)
    per_step = [begins[s].elapsed_time(ends[s]) for s in range(steps)]
    pass_ms = [a.elapsed_time(b) for a, b in marks] if mark else []
    return ev_start.elapsed_time(ev_end), per_step, pass_ms, t


def parity_with_oracle(P, torch, cfg, w_host, g_host, staging: bool) -> bool:
    """One one-call round on a fresh copy of the inputs against the CPU oracle, bit for bit."""
    import numpy as np
    import oracle
    ref = oracle.run_round(w_host, g_host, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    d_w = torch.from_numpy(w_host).cuda()
    d_g = [torch.from_numpy(g).cuda() for g in g_host]
    buf = P.RoundBuffers(cfg.N, cfg.K, cfg.k_core, cfg.k_exp, staging=staging)
    P.slimdp_round(d_w, d_g, cfg.c, cfg.seed, 0, cfg.eta, buf.scores, buf.core_idx, buf.core_aux, buf.exp_idx, buf.val,
                   buf.pulled, buf.select_ws, buf.explore_ws, buf.stage)
    P.read_status(buf.select_ws)
    P.read_status(buf.explore_ws)
    same = lambda t, a: np.array_equal(t.cpu().numpy().view(np.uint32), np.ascontiguousarray(a).view(np.uint32))
    ok = same(buf.core_idx, ref["core_idx"]) and same(d_w, ref["w"])
    for k in range(cfg.K):
        ok = ok and same(buf.exp_idx[k], ref["exp_idx"][k]) and same(buf.val[k], ref["val"][k]) \
            and same(buf.pulled[k], ref["pulled"][k])
    return bool(ok)


def config_report(P, torch, name: str, args, device, peak: float):
    """Short report for one of the other configs: warm and L2-flushed round times, both roofline
    fractions, and parity with the oracle re-checked on the spot."""
    from workloads import CONFIGS, all_inputs
    cfg = CONFIGS[name]
    N, K = cfg.N, cfg.K
    w_host, g_host = all_inputs(cfg)
    parity = parity_with_oracle(P, torch, cfg, w_host, g_host, args.staging) if N <= (1 << 26) else None
    w = torch.from_numpy(w_host).to(device)
    grads = [torch.from_numpy(g).to(device) for g in g_host]
    buf = P.RoundBuffers(N, K, cfg.k_core, cfg.k_exp, device, staging=args.staging)
    steps = max(20, min(args.steps, 50))
    _, warm, pass_ms, t = timed_rounds(P, torch, cfg, w, grads, buf, steps, 5, 0)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
    _, cold, _, t = timed_rounds(P, torch, cfg, w, grads, buf, steps, 3, t, flush=flush, mark=False)
    bm = model_bytes(N, K, cfg.k_core, cfg.k_exp)
    med = statistics.median(warm)
    out = {"N": N, "K": K, "k_core": cfg.k_core, "k_exp": cfg.k_exp,
           "us_per_round_median": round(med * 1e3, 1), "us_per_round_min": round(min(warm) * 1e3, 1),
           "us_per_round_l2_flushed_median": round(statistics.median(cold) * 1e3, 1),
           "us_per_round_l2_flushed_min": round(min(cold) * 1e3, 1),
           "gparams_per_s": N / (med * 1e-3) / 1e9,
           "frac_of_8TBs": bm["round"] / (med * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
           "frac_of_measured": bm["round"] / (med * 1e-3) / 1e9 / peak,
           "pass_us_median": round(statistics.median(pass_ms) * 1e3, 1) if pass_ms else None,
           "inputs_fit_l2": 4 * N * (K + 1) <= 126e6, "parity_with_oracle": parity}
    del buf, w, grads, flush
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import numpy as np
    import torch

    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl")
    torch.cuda.set_device(local_rank if world > 1 else 0)
    device = torch.device("cuda", torch.cuda.current_device())

    import paper_1709_09393_b200 as P
    from workloads import CONFIGS, all_inputs

    cfg = CONFIGS[args.config]
    if args.core_pct:
        cfg = cfg.with_core_pct(args.core_pct)   # another point of the core-ratio sweep
    if args.scale:
        from workloads import scaled_config
        cfg = scaled_config(cfg, args.scale)     # leading parameters only: a small case for profiling
    N, K, k_core, k_exp, m = cfg.N, cfg.K, cfg.k_core, cfg.k_exp, cfg.m
    w_host, g_host = all_inputs(cfg)
    w = torch.from_numpy(w_host).to(device)
    grads = [torch.from_numpy(g).to(device) for g in g_host]
    buf = P.RoundBuffers(N, K, k_core, k_exp, device, staging=args.staging)
    bytes_model = model_bytes(N, K, k_core, k_exp)

    def barrier():
        if world > 1:
            torch.distributed.barrier()

    # ---- timed region: exactly `steps` rounds (successive rounds t = 0, 1, ... on the evolving model, as
    # in training), each the ONE C-ABI call slimdp_round; device-timed
    sampler = ClockSampler(torch.cuda.current_device())
    launches0 = P.launch_count()
    barrier()
    sampler.start()
    total_ms, per_step, pass_ms, t = timed_rounds(P, torch, cfg, w, grads, buf, args.steps, args.warmup, 0)
    clocks = sampler.stop()
    barrier()
    launches = P.launch_count() - launches0
    total_ms = max_over_ranks(total_ms, world, device)
    ms_per_step = total_ms / args.steps
    dominant_ms = sum(pass_ms) / args.steps
    value = aggregate_value(N, world, ms_per_step)

    def one_round(tt):
        P.slimdp_round(w, grads, cfg.c, cfg.seed, tt, cfg.eta, buf.scores, buf.core_idx, buf.core_aux, buf.exp_idx,
                       buf.val, buf.pulled, buf.select_ws, buf.explore_ws, buf.stage)

    # ---- optional: kernel timeline of three more rounds (CUPTI through torch.profiler) ----
    # Start, duration and stream of every kernel, relative to the first: shows which kernels of the
    # one-call round run side by side, which a serialising profiler cannot.  Not a timing source.
    if args.timeline and rank == 0:
        from torch.profiler import ProfilerActivity, profile
        with profile(activities=[ProfilerActivity.CUDA]) as prof:
            for _ in range(3):
                one_round(t)
                t += 1
            torch.cuda.synchronize()
        trace = args.timeline + ".trace.json"
        prof.export_chrome_trace(trace)
        with open(trace) as f:
            events = [e for e in json.load(f)["traceEvents"] if e.get("cat") in ("kernel", "gpu_memset")]
        os.remove(trace)
        events.sort(key=lambda e: e["ts"])
        with open(args.timeline, "w") as f:
            f.write("# start_us duration_us stream kernel   (three consecutive slimdp_round calls)\n")
            for e in events:
                name = e["name"].replace("slimdp::(anonymous namespace)::", "").split("(")[0]
                f.write(f'{e["ts"] - events[0]["ts"]:10.1f} {e["dur"]:8.1f} s{e["args"].get("stream")} {name}\n')

    # ---- per-call breakdown (untimed for the headline; 5 more rounds) -------
    # the steps as separate C-ABI calls on one stream ("exchange" is the fused pack + merge + pull; the
    # three separate calls follow for comparison), then the steps either side of the path
    names = ["score", "select", "explore", "exchange", "pack_alone", "merge_alone", "pull_alone", "worker_merge",
             "dense_merge_score"]
    acc = {nm: [] for nm in names}
    breakdown_us = {"round_one_call": round(ms_per_step * 1e3, 1), "dominant_kernel": round(dominant_ms * 1e3, 1)}
    if not args.no_breakdown:
        local = [w.clone() for _ in range(K)]
        for _ in range(5):
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(10)]
            marks[0].record()
            P.slimdp_score(w, grads, cfg.c, buf.scores); marks[1].record()
            P.slimdp_select_core(buf.scores, k_core, buf.core_idx, buf.core_aux, buf.select_ws); marks[2].record()
            P.slimdp_sample_explore_batched(buf.core_aux, N, k_core, k_exp, cfg.seed, 0, t, buf.exp_idx, buf.explore_ws)
            marks[3].record()
            P.slimdp_exchange(w, grads, buf.core_idx, buf.exp_idx, cfg.eta, buf.val, buf.pulled); marks[4].record()
            P.slimdp_pack_batched(grads, buf.core_idx, buf.exp_idx, buf.val); marks[5].record()
            P.slimdp_merge(w, buf.core_idx, buf.exp_idx, buf.val, cfg.eta); marks[6].record()
            P.slimdp_pull_batched(w, buf.core_idx, buf.exp_idx, buf.pulled); marks[7].record()
            P.slimdp_worker_merge_batched(local, buf.core_idx, buf.exp_idx, buf.pulled); marks[8].record()
            P.slimdp_dense_merge_score(w, grads, cfg.eta, cfg.c, buf.scores); marks[9].record()
            torch.cuda.synchronize()
            t += 1
            for i, nm in enumerate(names):
                acc[nm].append(marks[i].elapsed_time(marks[i + 1]) * 1e3)
        breakdown_us.update({nm: round(statistics.median(v), 1) for nm, v in acc.items()})
        del local

    peak, peak_src = measured_peak()
    fused_kernel = fused_pass_kernel_name(K, buf.stage is not None)
    fused = N >= (1 << 21) and k_core > 0 and fused_kernel is not None   # the round scores inside the selection's pass
    if fused:
        # per parameter: K + 1 fp32 values read, one bit in each of the two bitmaps written (the
        # candidates, about 1 % of the parameters at 8 B each, are not counted)
        dominant = {"kernel": fused_kernel, "bytes": 4 * N * (K + 1) + 2 * (N // 8)}
    else:
        dominant = {"kernel": f"score_vec4_kernel<{K}>", "bytes": bytes_model["score"]}
    traffic = dominant_traffic(dominant["kernel"], N)
    achieved = dominant["bytes"] / (dominant_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dominant["kernel"], "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "traffic": traffic["bytes"] if traffic else None,
                "traffic_source": traffic, "algorithmic_bytes_per_launch": dominant["bytes"],
                "avg_launch_ms": dominant_ms, "peak_source": peak_src}
    round_gbs = bytes_model["round"] / (ms_per_step * 1e-3) / 1e9
    fused_gbs = bytes_model["round_fused"] / (ms_per_step * 1e-3) / 1e9
    # "round without score": the model's bytes of select + explore + pack + merge + pull against the
    # round's time less the score step's share of the fused pass (that pass's time scaled by the score
    # step's part of its bytes: an attribution), and, beside it, against the round's time less the
    # separately timed slimdp_score call (a measurement; that call also writes the scores)
    score_ms = dominant_ms * (4 * N * (K + 1) / dominant["bytes"]) if fused else dominant_ms
    rest_ms = ms_per_step - score_ms
    rest_gbs = bytes_model["round_without_score"] / (rest_ms * 1e-3) / 1e9
    without = {"model_bytes": bytes_model["round_without_score"], "ms": rest_ms, "achieved_gbs": rest_gbs,
               "frac_of_8TBs": rest_gbs / NOMINAL_HBM_GBS, "frac_of_measured": rest_gbs / peak,
               "how": "round time less the score step's byte share of the fused pass"}
    if "score" in breakdown_us and ms_per_step * 1e3 > breakdown_us["score"]:
        alt_ms = ms_per_step - breakdown_us["score"] * 1e-3
        alt_gbs = bytes_model["round_without_score"] / (alt_ms * 1e-3) / 1e9
        without["less_separate_score_call"] = {"ms": alt_ms, "frac_of_8TBs": alt_gbs / NOMINAL_HBM_GBS,
                                               "frac_of_measured": alt_gbs / peak}
    if not args.no_breakdown:
        sep_ms = (breakdown_us["select"] + breakdown_us["explore"] + breakdown_us["exchange"]) * 1e-3
        sep_gbs = bytes_model["round_without_score"] / (sep_ms * 1e-3) / 1e9
        without["as_separate_calls"] = {"ms": sep_ms, "frac_of_8TBs": sep_gbs / NOMINAL_HBM_GBS,
                                        "frac_of_measured": sep_gbs / peak}
    round_roofline = {
        "model_bytes": bytes_model["round"], "achieved_gbs": round_gbs,
        "frac_of_8TBs": round_gbs / NOMINAL_HBM_GBS, "frac_of_measured": round_gbs / peak,
        "label": "unfused model bytes (scores written and read back) over the one-call round's time",
        "moved_bytes": {"model_bytes": bytes_model["round_fused"], "achieved_gbs": fused_gbs,
                        "frac_of_8TBs": fused_gbs / NOMINAL_HBM_GBS, "frac_of_measured": fused_gbs / peak,
                        "label": "bytes the one-call round must move (no score write, no re-read)"},
        "without_score": without,
    }
    step_stats = {"median_ms": statistics.median(per_step), "min_ms": min(per_step), "max_ms": max(per_step),
                  "note": "per step, between events recorded around each round; ms_per_step is the whole timed "
                          "region over the step count"}
    # ---- end to end: host buffers through the C ABI, copies inside the timed region
    e2e = None
    if (rank == 0 or world > 1) and not args.no_e2e:
        pin = lambda a: torch.from_numpy(a).pin_memory()
        w_pin = pin(w_host.copy())
        g_pin = [pin(g) for g in g_host]
        core_pin = torch.empty(k_core, dtype=torch.int32).pin_memory()
        exp_pin = [torch.empty(k_exp, dtype=torch.int32).pin_memory() for _ in range(K)]
        pulled_pin = [torch.empty(m, dtype=torch.float32).pin_memory() for _ in range(K)]
        del buf
        torch.cuda.empty_cache()
        arena = torch.empty(P.round_arena_bytes(N, K, k_core, k_exp), dtype=torch.uint8, device=device)
        e2e_steps = max(1, min(args.steps, 5))
        P.slimdp_round_host(w_pin, g_pin, cfg.c, k_core, k_exp, cfg.seed, 0, cfg.eta, core_pin, exp_pin, pulled_pin,
                            arena)      # warm-up
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        e0.record()
        for s in range(e2e_steps):
            P.slimdp_round_host(w_pin, g_pin, cfg.c, k_core, k_exp, cfg.seed, 1 + s, cfg.eta, core_pin, exp_pin,
                                pulled_pin, arena)
        e1.record()
        torch.cuda.synchronize()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, device) / e2e_steps
        e2e = {"value": aggregate_value(N, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "h2d_bytes_per_step": 4 * N * (K + 1),
               "d2h_bytes_per_step": 4 * N + 4 * k_core + K * (4 * k_exp + 4 * m)}
        del arena, w_pin, g_pin
        torch.cuda.empty_cache()

    # ---- the other configs (rank 0, one GPU): warm and L2-flushed times, parity re-checked
    per_config = None
    if rank == 0 and world == 1 and args.per_config != "none" and not args.scale:
        del w, grads
        torch.cuda.empty_cache()
        names_pc = ["tiny", "googlenet", "resnet50_ties", "vgg16"] + (["large"] if args.per_config == "all" else [])
        per_config = {nm: config_report(P, torch, nm, args, device, peak) for nm in names_pc if nm != args.config}

    cpu_baseline = cpu_baseline_mt = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_cpu = cfg.N if args.cpu_baseline_full else min(cfg.N, CPU_BASELINE_SAMPLE)
        sample, times = time_oracle(cfg, n_cpu, 1, 0)
        what = (f"one oracle round on {'all' if sample.N == cfg.N else 'the leading'} {sample.N} parameters of the "
                f"{cfg.name}-shaped workload (K={sample.K}, k_core={sample.k_core}, k_exp={sample.k_exp})")
        cpu_baseline = {"value": sample.N / times[0] / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "seconds": times[0], "sample": what}
        threads = os.cpu_count() or 1
        sample, secs = time_oracle_threaded(cfg, n_cpu, threads)
        cpu_baseline_mt = {"value": sample.N / secs / 1e9, "unit": UNIT, "cores": threads,
                           "kind": "oracle, its loops spread over host threads (scoring over index chunks; "
                                   "explorers, extraction and pull over workers; sort and merge serial)",
                           "seconds": secs, "sample": what}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{cfg.name}-shaped: N={N} fp32 parameters, K={K} workers, k_core={k_core} "
                                   f"({cfg.core_pct}%), k_exp={k_exp} ({cfg.explore_pct}% of the non-core)",
                       "N": N, "K": K, "k_core": k_core, "k_exp": k_exp, "seed": cfg.seed,
                       "staging_area": bool(args.staging),
                       "l2": "inputs larger than L2 (no flush needed)" if 4 * N * (K + 1) > 4 * 126e6
                       else "inputs fit L2 (warm)",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks, "step_ms": step_stats, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
            "round_roofline": round_roofline, "breakdown_us": breakdown_us, "cpu_baseline": cpu_baseline,
            "cpu_baseline_threaded": cpu_baseline_mt, "per_config": per_config,
        }
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="vgg16")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-breakdown", action="store_true", help="skip the steps timed as separate calls")
    ap.add_argument("--per-config", default="default", choices=["default", "all", "none"],
                    help="short reports for the other configs: default = tiny, googlenet, resnet50_ties; "
                         "all = also the 10^9-parameter vector; none")
    ap.add_argument("--cpu-baseline-full", action="store_true",
                    help="time the CPU oracle on the whole workload instead of its leading 2^25 parameters")
    ap.add_argument("--staging", action="store_true",
                    help="give slimdp_round its optional staging area (the exchange then streams the core's values)")
    ap.add_argument("--timeline", default="",
                    help="also write the kernel timeline of three extra rounds (start, duration, stream) to this file")
    ap.add_argument("--core-pct", type=int, default=0, help="core ratio in percent (default: the config's own)")
    ap.add_argument("--scale", type=int, default=0,
                    help="run on the leading SCALE parameters of the config (small case for profiler captures)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
