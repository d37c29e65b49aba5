#!/usr/bin/env python
"""Benchmark of the G-KV hot path on B200.

A "step" is one eviction period of the decode loop in steady state: s decode-attention launches
over the compressed cache of every layer (the last w of them accumulating the window score)
followed by one eviction of every layer (normalise, merge with history, top-(b-w), compaction).
The default workload is the 7B-reasoning-model shape the paper's compression-time table is
quoted on (28 layers, batch 32, 28 q / 4 kv heads, d = 128, b = 1024, w = 32, s = 128).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg1|cfg3|cfg4] [--impl reference]

--workload cfg3 runs the eviction-step sweep (stages timed separately and fused) instead of the decode loop.

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange step.
One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "decode tok/s over the compressed cache incl. eviction (attention + eviction only)"
UNIT = "tok/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode kernel, from the ncu capture
# summarised in profiles/decode_kernel_cfg2.md: measured on a 4-layer stack (512 units) as 1.012 (plain
# steps) and 1.015 (window steps) x the algorithmic bytes of the captured launches, i.e. 1.013 over a
# period, scaled to the full 3584-unit launch at the period's average length (traffic grows in
# proportion to units). None where no capture exists.
NCU_TRAFFIC_BYTES = {"cfg2": 1.013 * 2.022e9, "cfg1": None, "cfg4": None}


def workload_shape(name: str) -> dict:
    from paper_2512_00504_b200 import synth
    idx = {"cfg0": 0, "cfg1": 1, "cfg2": 2, "cfg4": 4}[name]
    shape = {k: v for k, v in synth.CONFIGS[idx].items() if k != "steps"}
    return shape


def describe(name: str, sh: dict) -> str:
    return (f"config {name[3:]}: {sh['n_layers']} layers x batch {sh['batch']}, {sh['h_q']} q / {sh['h_kv']} kv heads, "
            f"d {sh['d']}, b={sh['b']}, buffer={sh['buffer']}, w={sh['w']}, s={sh['s']}; steady state len {sh['b']}..{sh['b'] + sh['s']}; "
            f"step = one eviction period ({sh['s']} all-layer decode-attention launches + 1 all-layer eviction)")


# ------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period: float = 0.1):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
            }
            get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
            while not self._stop_evt.is_set():
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                mask = get_reasons(h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
                time.sleep(self.period)
        except Exception as e:  # NVML missing: report that rather than fail the benchmark
            self.reasons.add(f"nvml_unavailable:{type(e).__name__}")

    def stop(self) -> dict:
        self._stop_evt.set()
        self.join(timeout=2)
        med = sorted(self.samples)[len(self.samples) // 2] if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(value: float) -> float:
    """Max of a per-rank scalar over the process group (identity without one). Works with any backend."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def replica_summary(tokens_per_rank_step: float, steps: int, max_ms: float, world: int) -> dict:
    """Whole-job throughput of `world` independent replicas timed as the max over ranks."""
    return {"value": world * tokens_per_rank_step * steps / (max_ms * 1e-3), "ms_per_step": max_ms / steps}


# ------------------------------------------------------------------------------------------
def algorithmic_bytes(sh: dict, n_keys: int, accum: bool) -> float:
    """Bytes one decode launch must move: every K and V row of every unit once, q / k_new / v_new in,
    out back, the appended rows written, and on window steps the read-modify-write of the sums."""
    units = sh["n_layers"] * sh["batch"] * sh["h_kv"]
    row = sh["d"] * 2
    per_unit = 2 * n_keys * row + 2 * row            # K, V stream + the appended rows written
    g = sh["h_q"] // sh["h_kv"]
    per_unit += 2 * g * row + 2 * row                # q in, out back, k_new / v_new in
    if accum:
        per_unit += 8 * n_keys
    return float(units * per_unit)


def evict_bytes(sh: dict, moved_rows: float) -> float:
    """Bytes of one eviction (window-sum path): sums read and cleared, F read and written, and each moved
    K and V row read and written once."""
    units = sh["n_layers"] * sh["batch"] * sh["h_kv"]
    C, l, b, w = sh["b"] + sh["buffer"], sh["b"] + sh["s"], sh["b"], sh["w"]
    per_unit = 4 * l + 4 * C + 4 * (b - w) + 4 * C + 4 * b   # sums read + cleared, F read + written, kept list
    return float(units * per_unit + moved_rows * 4 * sh["d"] * 2)


def redundancy_kwargs(args) -> dict:
    """Configuration of the redundancy term (appendix on combining the global score with other methods);
    off unless --redundancy LAMBDA is given. Threshold and protected recent tokens are the benchmark's choice."""
    if args.redundancy is None:
        return {}
    return dict(redundancy_lambda=args.redundancy, redundancy_threshold=args.redundancy_threshold)


def run_ours(args) -> dict:
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}: launch N > 1 with torch.distributed.run"
    dev = f"cuda:{local}"
    torch.cuda.set_device(local)
    gkv.build_library()

    sh = workload_shape(args.workload)
    if args.layers > 0:
        sh["n_layers"] = args.layers   # reduced stack for profiler captures; not a benchmark number
    L, B, Hq, H, d, b, w, s = (sh[k] for k in ("n_layers", "batch", "h_q", "h_kv", "d", "b", "w", "s"))
    C = b + sh["buffer"]
    cfg = gkv.make_config(**sh, alpha=0.8, mode=gkv.GKV_MODE_MAX, fuse_window_scores=True, **redundancy_kwargs(args))
    cache = gkv.GKVCache(cfg, dev, staging=True)

    # steady-state cache: b rows of N(0,1) keys/values, history on the first b-w rows
    gen = torch.Generator(device=dev).manual_seed(synth.BASE_SEED + 100 + rank)
    for layer in range(L):
        cache.k[layer, :, :, :b] = torch.randn((B, H, b, d), generator=gen, device=dev).to(torch.bfloat16)
        cache.v[layer, :, :, :b] = torch.randn((B, H, b, d), generator=gen, device=dev).to(torch.bfloat16)
        cache.f[layer, :, :, : b - w] = torch.rand((B, H, b - w), generator=gen, device=dev)
    cache.set_state(-1, b, b - w, 0)

    # one period of drifting per-step inputs, generated once (device ring + pinned host copy for e2e)
    ring = min(s, args.ring) if args.ring > 0 else s
    stream = synth.DecodeStream(synth.BASE_SEED + 2 + rank, n_layers=L, batch=B, h_q=Hq, h_kv=H, b=b, s=s, device=dev)
    steps_in = [stream.step() for _ in range(ring)]
    out = torch.empty((L, B, Hq, d), dtype=torch.bfloat16, device=dev)
    kept = torch.empty((L, B, H, b), dtype=torch.int32, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def period(timers=None):
        if timers is not None:
            timers[0].record()
        for t in range(s):
            if timers is not None and t == s - w:
                timers[1].record()
            q, kn, vn = steps_in[t % ring]
            cache.decode_attn(-1, q, kn, vn, out)
        if timers is not None:
            timers[2].record()
        cache.evict(-1, None, kept)
        if timers is not None:
            timers[3].record()

    for _ in range(max(args.warmup, 3)):
        period()
    cache.poll()
    moved = float((kept != torch.arange(b, device=dev, dtype=torch.int32)).sum().item())  # rows that moved in the last warm-up eviction

    sampler = ClockSampler(local)
    timers = [[ev() for _ in range(4)] for _ in range(args.steps)]
    launches0 = gkv.gkv_launch_count(cache.ctx)
    t0, t1 = ev(), ev()
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    t0.record()
    for k in range(args.steps):
        period(timers[k])
    t1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    launches = gkv.gkv_launch_count(cache.ctx) - launches0
    cache.poll()
    total_ms = t0.elapsed_time(t1)
    plain_ms = sum(t[0].elapsed_time(t[1]) for t in timers) / (args.steps * (s - w))
    window_ms = sum(t[1].elapsed_time(t[2]) for t in timers) / (args.steps * w)
    evict_ms = sum(t[2].elapsed_time(t[3]) for t in timers) / args.steps
    decode_ms = (plain_ms * (s - w) + window_ms * w) / s

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        host_in = [tuple(x.cpu().pin_memory() for x in st) for st in steps_in]
        host_out = torch.empty((L, B, Hq, d), dtype=torch.bfloat16).pin_memory()
        host_kept = torch.empty((L, B, H, b), dtype=torch.int32).pin_memory()
        e_steps = max(1, min(args.steps, args.e2e_steps))

        def period_host():
            for t in range(s):
                q, kn, vn = host_in[t % ring]
                gkv.gkv_decode_attn_host(cache.ctx, -1, q, kn, vn, host_out)
            gkv.gkv_evict_host(cache.ctx, -1, None, host_kept)

        period_host()
        e0, e1 = ev(), ev()
        barrier()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(e_steps):
            period_host()
        e1.record()
        torch.cuda.synchronize()
        barrier()
        e_ms = max_over_ranks(e0.elapsed_time(e1))
        h2d = sum(x.numel() * 2 for x in host_in[0]) * s
        d2h = host_out.numel() * 2 * s + host_kept.numel() * 4
        e2e = {"value": world * B * s * e_steps / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e_steps, "ms_per_step": e_ms / e_steps}
        cache.poll()

    max_ms = max_over_ranks(total_ms)
    summ = replica_summary(B * s, args.steps, max_ms, world)

    # ---- roofline of the dominant kernel (decode attention): algorithmic bytes / measured launch time
    peaks_path = ROOT / "MEASURED_PEAKS.json"
    if peaks_path.exists():
        peak_gbs, peak_src = float(json.loads(peaks_path.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak_gbs, peak_src = 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"
    n_plain = [b + t + 1 for t in range(s - w)]
    n_win = [b + t + 1 for t in range(s - w, s)]
    bytes_plain = sum(algorithmic_bytes(sh, n, False) for n in n_plain) / len(n_plain)
    bytes_win = sum(algorithmic_bytes(sh, n, True) for n in n_win) / len(n_win)
    bytes_avg = (bytes_plain * (s - w) + bytes_win * w) / s
    ach = bytes_avg / (decode_ms * 1e-3) / 1e9
    roofline = {"kernel": "gkv_decode_kernel", "bound": "hbm", "achieved": ach, "peak": peak_gbs, "unit": "GB/s",
                "frac": ach / peak_gbs, "peak_source": peak_src, "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                "algorithmic_bytes_per_launch": bytes_avg, "avg_launch_ms": decode_ms,
                "plain_steps": {"ms": plain_ms, "GBps": bytes_plain / (plain_ms * 1e-3) / 1e9},
                "window_steps": {"ms": window_ms, "GBps": bytes_win / (window_ms * 1e-3) / 1e9},
                "frac_of_nominal_8TBps": ach / 8000.0}
    eb = evict_bytes(sh, moved)
    units = L * B * H
    evict = {"kernel": "gkv_evict_fused_kernel", "ms": evict_ms, "eviction_steps_per_s": 1e3 / evict_ms,
             "scored_kv_tokens_per_s": units * (b + s) / (evict_ms * 1e-3), "moved_rows": moved,
             "algorithmic_bytes": eb, "achieved_GBps": eb / (evict_ms * 1e-3) / 1e9,
             "frac": eb / (evict_ms * 1e-3) / 1e9 / peak_gbs, "overhead_frac_of_step": evict_ms / (max_ms / args.steps)}
    if args.redundancy is not None:   # the eviction then has two more launches (key norms, similarity sums on tcgen05)
        evict["redundancy"] = {"lambda": args.redundancy, "threshold": args.redundancy_threshold,
                               "note": "ms includes gkv_keynorm_kernel and gkv_redundancy_tc_kernel; GB/s and frac do not describe them",
                               "gram_flop": 2.0 * units * (b + s) * (b + s) * d}

    result = {
        "metric": METRIC, "value": summ["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": summ["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": describe(args.workload, sh) + (" [REDUCED LAYER COUNT: profiling only]" if args.layers > 0 else ""),
                   "tokens_per_step": B * s,
                   "l2": "inputs larger than L2: every launch streams the whole resident cache "
                         f"({2 * units * C * d * 2 / 1e9:.2f} GB K+V)",
                   "input_ring": ring, "replicas": world},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "eviction": evict,
        "decode": {"ms_per_launch": decode_ms, "attention_only_tok_per_s": B / (decode_ms * 1e-3)},
    }
    if rank == 0 and world == 1 and not args.no_cpu:
        result["cpu_baseline"] = cpu_baseline(sh, budget_s=args.cpu_seconds)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return result if rank == 0 else None


# ------------------------------------------------------------------------------------------
def run_sweep(args) -> dict:
    """Eviction-step sweep (configuration 3): 32 q / 8 kv heads, one layer, b x batch x w cells, l = b + 128.
    Per cell the stages (score, merge, select, compact) are timed as separate launches, then the step as it
    runs in production: one fused launch reading the window sums, and the recompute path (score launch +
    fused launch). The JSON line carries the largest cell; `sweep` holds every cell."""
    import math
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    dev = "cuda:0"
    torch.cuda.set_device(0)
    gkv.build_library()
    c3 = synth.CONFIGS[3]
    peaks_path = ROOT / "MEASURED_PEAKS.json"
    peaks = json.loads(peaks_path.read_text()) if peaks_path.exists() else {}
    peak_gbs = float(peaks.get("hbm_gbs", 6650.0))
    peak_tf = float(peaks.get("bf16_tflops", 1590.0))
    peak_src = "measured (MEASURED_PEAKS.json)" if peaks else "fallback (6.65 TB/s, 1.59 PFLOP/s)"
    ev = lambda: torch.cuda.Event(enable_timing=True)
    reps = max(3, args.steps)
    cells = []
    sampler = ClockSampler(0)
    sampler.start()
    launches = 0
    pick = lambda arg, sweep: tuple(int(x) for x in arg.split(",")) if arg else sweep
    for b in pick(args.sweep_b, c3["b_sweep"]):
        for batch in pick(args.sweep_batch, c3["batch_sweep"]):
            for w in pick(args.sweep_w, c3["w_sweep"]):
                sh = dict(n_layers=1, batch=batch, h_q=c3["h_q"], h_kv=c3["h_kv"], d=128, b=b, buffer=c3["buffer"], w=w, s=c3["s"])
                H, g, C = sh["h_kv"], sh["h_q"] // sh["h_kv"], b + sh["buffer"]
                l, n_h, units = C, b - w, batch * sh["h_kv"]
                cfg = gkv.make_config(**sh, alpha=0.8, mode=gkv.GKV_MODE_MAX, fuse_window_scores=True, **redundancy_kwargs(args))
                cache = gkv.GKVCache(cfg, dev)
                red = args.redundancy is not None
                case = synth.eviction_case(synth.BASE_SEED + 3, batch=batch, h_q=sh["h_q"], h_kv=H, b=b, buffer=sh["buffer"],
                                           w=w, n_planted=math.ceil(0.01 * l), device=dev)
                cache.k[0].copy_(case.k); cache.v[0].copy_(case.v); cache.f[0].copy_(case.f_prev)
                q_win = case.q_win.unsqueeze(0).contiguous()
                del case
                cache.set_state(0, l, n_h, sh["s"], False)
                cache.evict_stage(0, gkv.GKV_STAGE_SCORE, q_win)          # the window sums of this state (w * S)
                sums0, f0 = cache.sacc.clone(), cache.f.clone()
                kept = torch.empty((1, batch, H, b), dtype=torch.int32, device=dev)

                def restore():
                    cache.sacc.copy_(sums0); cache.f.copy_(f0)
                    cache.set_state(0, l, n_h, sh["s"], True)

                t = {k: [] for k in ("score", "merge", "select", "compact", "fused", "recompute", "redundancy")}
                moved = 0.0
                l0 = gkv.gkv_launch_count(cache.ctx)
                for it in range(reps + 3):
                    e = [ev() for _ in range(11)]
                    restore()
                    e[0].record(); cache.evict_stage(0, gkv.GKV_STAGE_SCORE, q_win)
                    e[9].record()
                    if red:
                        cache.evict_stage(0, gkv.GKV_STAGE_REDUNDANCY)
                    e[10].record()
                    e[1].record(); cache.evict_stage(0, gkv.GKV_STAGE_MERGE)
                    e[2].record(); cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept)
                    e[3].record(); cache.evict_stage(0, gkv.GKV_STAGE_COMPACT)
                    e[4].record()
                    restore()
                    e[5].record(); cache.evict(0, None, kept); e[6].record()
                    moved = float((kept != torch.arange(b, device=dev, dtype=torch.int32)).sum().item())
                    restore()
                    e[7].record(); cache.evict(0, q_win, kept); e[8].record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        for k, (a, z) in zip(t, ((0, 9), (1, 2), (2, 3), (3, 4), (5, 6), (7, 8), (9, 10))):
                            t[k].append(e[a].elapsed_time(e[z]))
                cache.poll()
                launches += gkv.gkv_launch_count(cache.ctx) - l0
                med = {k: sorted(v)[len(v) // 2] for k, v in t.items()}
                eb = evict_bytes(sh, moved)
                flops = 2.0 * 2.0 * units * g * w * 128 * l        # two passes over the keys (statistics, then weights)
                kbytes = 2.0 * units * l * 256 + units * g * w * 256
                cells.append({"b": b, "batch": batch, "w": w, "units": units, "ms": med, "moved_rows": moved,
                              "fused_GBps": eb / (med["fused"] * 1e-3) / 1e9, "fused_frac": eb / (med["fused"] * 1e-3) / 1e9 / peak_gbs,
                              "fused_bytes": eb, "kv_bytes_resident": 2.0 * units * C * 256,
                              "score_TFLOPs": flops / (med["score"] * 1e-3) / 1e12, "score_K_GBps": kbytes / (med["score"] * 1e-3) / 1e9,
                              "redundancy_TFLOPs": (2.0 * units * l * l * 128 / (med["redundancy"] * 1e-3) / 1e12) if red else None,
                              "scored_kv_tokens_per_s": units * l / (med["recompute"] * 1e-3),
                              "scored_kv_tokens_per_s_window_sums": units * l / (med["fused"] * 1e-3)})
                del cache, sums0, f0, kept, q_win
                torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = cells[-1]
    return {"metric": "scored KV tokens/s of one eviction step (score from the window queries + merge + top-(b-w) + compaction)",
            "value": top["scored_kv_tokens_per_s"], "unit": "tok/s", "n_gpus": 1, "steps": reps, "warmup": 3,
            "ms_per_step": top["ms"]["recompute"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config 3 sweep, largest cell: 1 layer, batch {top['batch']}, 32 q / 8 kv heads, d 128, b={top['b']}, "
                                   f"buffer=128, w={top['w']}, l={top['b'] + 128}; step = one eviction step",
                       "l2": "cells with batch >= 64 hold more K+V than L2; smaller cells are L2-resident, as they are right after a decode step"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
            "roofline": {"kernel": "gkv_evict_fused_kernel", "bound": "hbm", "achieved": top["fused_GBps"], "peak": peak_gbs,
                         "unit": "GB/s", "frac": top["fused_frac"], "peak_source": peak_src, "traffic": None,
                         "algorithmic_bytes_per_launch": top["fused_bytes"], "avg_launch_ms": top["ms"]["fused"]},
            "score_kernel": {"TFLOPs": top["score_TFLOPs"], "frac_of_bf16_peak": top["score_TFLOPs"] / peak_tf, "peak_TFLOPs": peak_tf},
            "sweep": cells}


# ------------------------------------------------------------------------------------------
def run_perlayer(args) -> dict:
    """Decode attention launched one layer at a time, the way a model calls it (7B head geometry, b = 1024, w = 32,
    cache at 1064 tokens): the 28 per-layer launches of a step are captured in a CUDA graph and replayed, so the
    figure is device time per launch without host issue overhead. Batch 1, 8, 32, 128; plain and window steps."""
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    dev = "cuda:0"
    torch.cuda.set_device(0)
    gkv.build_library()
    base = {k: v for k, v in synth.CONFIGS[2].items() if k != "steps"}
    peaks_path = ROOT / "MEASURED_PEAKS.json"
    peak_gbs = float(json.loads(peaks_path.read_text())["hbm_gbs"]) if peaks_path.exists() else 6650.0
    reps = max(3, args.steps)
    cells, launches = [], 0
    sampler = ClockSampler(0)
    sampler.start()
    for batch in (1, 8, 32, 128):
        sh = dict(base, batch=batch)
        L, B, Hq, H, d, b, w, s = (sh[k] for k in ("n_layers", "batch", "h_q", "h_kv", "d", "b", "w", "s"))
        cache = gkv.GKVCache(gkv.make_config(**sh, fuse_window_scores=True), dev)
        gen = torch.Generator(device=dev).manual_seed(synth.BASE_SEED + 11)
        cache.k.copy_(torch.randn(cache.k.shape, generator=gen, device=dev).to(torch.bfloat16))
        cache.v.copy_(torch.randn(cache.v.shape, generator=gen, device=dev).to(torch.bfloat16))
        q = torch.randn((L, B, Hq, d), generator=gen, device=dev).to(torch.bfloat16)
        kn = torch.randn((L, B, H, d), generator=gen, device=dev).to(torch.bfloat16)
        vn = torch.randn((L, B, H, d), generator=gen, device=dev).to(torch.bfloat16)
        out = torch.empty_like(q)
        cell = {"batch": batch, "units_per_launch": B * H}
        for name, since in (("plain", 40), ("window", s - w)):
            n0 = b + since
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                cache.set_state(-1, n0, b - w, since)
                for layer in range(L):                              # warm-up outside the capture
                    cache.decode_attn(layer, q[layer], kn[layer], vn[layer], out[layer])
                cache.set_state(-1, n0, b - w, since)
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for layer in range(L):
                        cache.decode_attn(layer, q[layer], kn[layer], vn[layer], out[layer])
            launches += 2 * L
            ts = []
            for _ in range(reps + 3):
                cache.set_state(-1, n0, b - w, since)               # the replay advances the device lengths only
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); graph.replay(); e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) / L)
            launches += (reps + 3) * L
            ms = sorted(ts[3:])[len(ts[3:]) // 2]
            cell[name + "_us"] = ms * 1e3
            cell[name + "_GBps"] = algorithmic_bytes(dict(sh, n_layers=1), n0 + 1, name == "window") / (ms * 1e-3) / 1e9
        cache.poll()
        cells.append(cell)
        del cache, graph
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = cells[2]
    L = base["n_layers"]
    return {"metric": "decode tok/s with attention launched one layer at a time (28 launches per token step, attention only)",
            "value": top["batch"] / (L * top["plain_us"] * 1e-6), "unit": "tok/s", "n_gpus": 1, "steps": reps, "warmup": 3,
            "ms_per_step": L * top["plain_us"] * 1e-3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "per-layer decode launches: 28 layers, 28 q / 4 kv heads, d 128, b=1024, w=32, cache at 1064 "
                                   "tokens; headline cell batch 32 (128 units per launch); step = the 28 launches of one token step",
                       "l2": "the 28 layers' K+V (0.55 MB per unit) exceed L2 from batch 8 on; each launch reads its own layer"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
            "roofline": {"kernel": "gkv_decode_kernel (key split)", "bound": "hbm", "achieved": top["plain_GBps"], "peak": peak_gbs,
                         "unit": "GB/s", "frac": top["plain_GBps"] / peak_gbs, "traffic": None,
                         "avg_launch_ms": top["plain_us"] * 1e-3},
            "sweep": cells}


# ------------------------------------------------------------------------------------------
def run_prompt(args) -> dict:
    """First compression of a prefilled prompt (one layer of the 7B shape: batch 32, 28 q / 4 kv heads, b = 1024,
    w = 32) for prompt lengths 2048, 4096, 8192 and 32768: scoring of the prompt's window over all its keys,
    selection and gather into the cache. The JSON line carries the longest prompt; `sweep` every length."""
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    dev = "cuda:0"
    torch.cuda.set_device(0)
    gkv.build_library()
    sh = {k: v for k, v in synth.CONFIGS[2].items() if k != "steps"}
    sh["n_layers"] = 1
    B, Hq, H, b, w = sh["batch"], sh["h_q"], sh["h_kv"], sh["b"], sh["w"]
    peaks_path = ROOT / "MEASURED_PEAKS.json"
    peak_gbs = float(json.loads(peaks_path.read_text())["hbm_gbs"]) if peaks_path.exists() else 6650.0
    ev = lambda: torch.cuda.Event(enable_timing=True)
    reps = max(3, args.steps)
    cells, launches = [], 0
    sampler = ClockSampler(0)
    sampler.start()
    for P in (2048, 4096, 8192, 32768):
        cfg = gkv.make_config(**sh, fuse_window_scores=True, max_prompt=P)
        cache = gkv.GKVCache(cfg, dev)
        gen = torch.Generator(device=dev).manual_seed(synth.BASE_SEED + 9)
        kp = torch.randn((B, H, P, 128), generator=gen, device=dev).to(torch.bfloat16)
        vp = torch.randn((B, H, P, 128), generator=gen, device=dev).to(torch.bfloat16)
        qw = torch.randn((B, Hq, w, 128), generator=gen, device=dev).to(torch.bfloat16)
        kept = torch.empty((B, H, b), dtype=torch.int32, device=dev)
        ts = []
        l0 = gkv.gkv_launch_count(cache.ctx)
        for it in range(reps + 3):
            e0, e1 = ev(), ev()
            e0.record(); cache.compress_prompt(0, kp, vp, qw, [P] * B, kept); e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1))
        cache.poll()
        launches += gkv.gkv_launch_count(cache.ctx) - l0
        ms = sorted(ts)[len(ts) // 2]
        units = B * H
        bytes_ = units * (P * 256 + 2 * b * 256 * 2 + 8 * P)     # K once (second pass from L2), gather of b K and V rows, sums
        cells.append({"prompt_len": P, "ms": ms, "prompt_tokens_per_s": B * P / (ms * 1e-3), "algorithmic_bytes": bytes_,
                      "GBps": bytes_ / (ms * 1e-3) / 1e9, "score_flop": 2.0 * 2.0 * units * (Hq // H) * w * 128 * P,
                      "score_TFLOPs": 2.0 * 2.0 * units * (Hq // H) * w * 128 * P / (ms * 1e-3) / 1e12})
        del cache, kp, vp, qw, kept
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = cells[-1]
    return {"metric": "prompt tokens/s compressed into the cache (first compression of a prefilled prompt, one layer)",
            "value": top["prompt_tokens_per_s"], "unit": "tok/s", "n_gpus": 1, "steps": reps, "warmup": 3,
            "ms_per_step": top["ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"prompt compression: 1 layer, batch {B}, {Hq} q / {H} kv heads, d 128, b={b}, w={w}, "
                                   f"prompt {top['prompt_len']} tokens per sequence; step = scoring + selection + gather",
                       "l2": "the prompt's K (268 MB at 8192 tokens, 1.07 GB at 32768) exceeds L2"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
            "roofline": {"kernel": "gkv_score_tc_kernel + gkv_prompt_compress_kernel", "bound": "hbm", "achieved": top["GBps"],
                         "peak": peak_gbs, "unit": "GB/s", "frac": top["GBps"] / peak_gbs, "traffic": None,
                         "algorithmic_bytes_per_launch": top["algorithmic_bytes"], "avg_launch_ms": top["ms"]},
            "sweep": cells}


# ------------------------------------------------------------------------------------------
def cpu_baseline(sh: dict, budget_s: float = 20.0, n_units: int = 64) -> dict:
    """The oracle, as it stands, timed on the host cores on a bounded sample of the workload:
    `n_units` (layer, sequence) pairs, a few decode steps plus one eviction; extrapolated to a period."""
    import numpy as np
    import oracle

    rng = np.random.default_rng(7)
    Hq, H, d, b, w, s = (sh[k] for k in ("h_q", "h_kv", "d", "b", "w", "s"))
    C = b + sh["buffer"]
    total_units = sh["n_layers"] * sh["batch"]
    n_units = min(n_units, total_units)
    rb = lambda *shape: (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    K, V = rb(n_units, H, C, d), rb(n_units, H, C, d)
    q = rb(n_units, Hq, d)
    F = rng.random((n_units, H, C)).astype(np.float32)
    n_keys = b + s // 2
    t0 = time.perf_counter()
    oracle.decode_batch(q, K, V, n_keys)
    one = time.perf_counter() - t0
    reps = int(max(1, min(16, (budget_s * 0.6) / max(one, 1e-3))))
    sacc = np.zeros((n_units, H, C), np.float64)
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.decode_batch(q, K, V, n_keys, Sacc=sacc)
    t_dec = (time.perf_counter() - t0) / reps
    S = np.ascontiguousarray(sacc.astype(np.float32))
    t0 = time.perf_counter()
    oracle.evict_batch(None, S, K, V, F, h_q=Hq, l=b + s, n_h=b - w, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, want_kv=True)
    t_ev = time.perf_counter() - t0
    period = (total_units / n_units) * (s * t_dec + t_ev)
    return {"value": sh["batch"] * s / period, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n_units} of {total_units} (layer, sequence) pairs: {reps + 1} decode steps at {n_keys} keys "
                      f"({t_dec * 1e3:.1f} ms each) + 1 eviction with compaction ({t_ev * 1e3:.1f} ms); "
                      "period time extrapolated linearly in pairs and steps",
            "decode_step_s_full_workload": (total_units / n_units) * t_dec,
            "eviction_s_full_workload": (total_units / n_units) * t_ev}


def run_reference(args) -> dict | None:
    """The oracle arm: the same metric and configuration computed by the CPU oracle on the host cores,
    each step a bounded sample of the workload. Rank 0 only."""
    if int(os.environ.get("RANK", 0)) != 0:
        return None
    import oracle
    oracle.build()
    sh = workload_shape(args.workload)
    for _ in range(min(args.warmup, 1)):
        cpu_baseline(sh, budget_s=2.0, n_units=8)
    vals = []
    t0 = time.perf_counter()
    steps = max(1, min(args.steps, 4))
    for _ in range(steps):
        vals.append(cpu_baseline(sh, budget_s=max(4.0, args.cpu_seconds / steps)))
    wall = time.perf_counter() - t0
    base = vals[-1]
    value = sum(v["value"] for v in vals) / len(vals)
    B, s = sh["batch"], sh["s"]
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * B * s / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(args.workload, sh), "tokens_per_step": B * s,
                       "note": "CPU oracle on the host cores; each step times a bounded sample and extrapolates"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": base["cores"], "kind": "oracle", "sample": base["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "prompt", "perlayer"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiler captures only)")
    ap.add_argument("--ring", type=int, default=0, help="distinct per-step inputs kept on the device (0 = one period)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--sweep-b", default="", help="cfg3: comma-separated budgets instead of the full sweep")
    ap.add_argument("--sweep-batch", default="", help="cfg3: comma-separated batch sizes instead of the full sweep")
    ap.add_argument("--sweep-w", default="", help="cfg3: comma-separated windows instead of the full sweep")
    ap.add_argument("--redundancy", type=float, default=None, metavar="LAMBDA",
                    help="select on LAMBDA * F - (1 - LAMBDA) * R' (redundancy term on; adds two launches per eviction)")
    ap.add_argument("--redundancy-threshold", type=float, default=0.5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.workload in ("cfg3", "prompt", "perlayer"):
            args.workload = "cfg2"   # the oracle arm times the default workload only
        res = run_reference(args)
    elif args.workload == "cfg3":
        res = run_sweep(args)
    elif args.workload == "prompt":
        res = run_prompt(args)
    elif args.workload == "perlayer":
        res = run_perlayer(args)
    else:
        res = run_ours(args)
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
