#!/usr/bin/env python
"""Benchmark of the G-KV hot path on B200.

A "step" is one eviction period of the decode loop in steady state: s decode-attention launches
over the compressed cache of every layer (the last w of them accumulating the window score)
followed by one eviction of every layer (normalise, merge with history, top-(b-w), compaction).
The headline workload is the 7B-reasoning-model shape the paper's compression-time table is
quoted on (28 layers, batch 32, 28 q / 4 kv heads, d = 128, b = 1024, w = 32, s = 128).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg1|cfg3|cfg4|...] [--impl reference]

With the default workload on one GPU the JSON line also carries `configs`: the other benchmark
configurations (single eviction step, batch-1 decode loop, the eviction-step sweep's batch >= 64 cells,
the 32B-shaped 77 GB stress case), each with its time per launch, algorithmic bytes, fraction of the
measured peak, clock sample and a sampled CPU-oracle baseline (--no-configs leaves them out).
--workload cfg3 runs the whole eviction-step sweep (stages timed separately and fused).

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange step.
One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "decode tok/s over the compressed cache incl. eviction (attention + eviction only)"
UNIT = "tok/s"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the decode kernel as a multiple of its algorithmic
# bytes, from one ncu capture of a 4-layer stack of the same shape (512 units per launch): 1.012 on plain steps and
# 1.015 on window steps, 1.013 over a period; traffic grows in proportion to the units of a launch. The JSON line
# labels the figure as scaled from that capture, and drops it for any other shape.
NCU_TRAFFIC_RATIO = {"cfg2": 1.013}
L2_FLUSH_BYTES = 512 << 20


def load_peaks() -> dict:
    """Roofline denominators: the machine's measured copy rate and bf16 matmul rate, else the stated fallback."""
    path = ROOT / "MEASURED_PEAKS.json"
    if path.exists():
        p = json.loads(path.read_text())
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p.get("bf16_tflops", 1590.0)),
                "source": "measured (MEASURED_PEAKS.json: copy rate, cuBLAS bf16 burst rate)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback (6.65 TB/s, 1.59 PFLOP/s: earlier measurement on this pool)"}


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


def time_period_loop(sh: dict, dev: str, *, steps: int, warmup: int, ring: int, seed: int, gpu_index: int,
                     red_kwargs: dict, e2e_steps: int = 0, world: int = 1) -> dict:
    """Steady-state decode + eviction loop at shape `sh`: `warmup` untimed periods, then `steps` timed ones between
    barriers, CUDA events on the launching stream. Returns this rank's raw timings; the cache is freed on return."""
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    L, B, Hq, H, d, b, w, s = (sh[k] for k in ("n_layers", "batch", "h_q", "h_kv", "d", "b", "w", "s"))
    cfg = gkv.make_config(**sh, alpha=0.8, mode=gkv.GKV_MODE_MAX, fuse_window_scores=True, **red_kwargs)
    cache = gkv.GKVCache(cfg, dev, staging=e2e_steps > 0)
    # steady-state cache: b rows of N(0,1) keys/values, history on the first b-w rows
    gen = torch.Generator(device=dev).manual_seed(seed + 100)
    for layer in range(L):
        cache.k[layer, :, :, :b] = torch.randn((B, H, b, d), generator=gen, device=dev).to(torch.bfloat16)
        cache.v[layer, :, :, :b] = torch.randn((B, H, b, d), generator=gen, device=dev).to(torch.bfloat16)
        cache.f[layer, :, :, : b - w] = torch.rand((B, H, b - w), generator=gen, device=dev)
    cache.set_state(-1, b, b - w, 0)

    # one period of drifting per-step inputs, generated once (device ring + pinned host copy for e2e)
    ring = min(s, ring) if ring > 0 else s
    stream = synth.DecodeStream(seed + 2, n_layers=L, batch=B, h_q=Hq, h_kv=H, b=b, s=s, device=dev)
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

    for _ in range(warmup):
        period()
    cache.poll()
    moved = float((kept != torch.arange(b, device=dev, dtype=torch.int32)).sum().item())  # rows that moved in the last warm-up eviction

    sampler = ClockSampler(gpu_index)
    timers = [[ev() for _ in range(4)] for _ in range(steps)]
    launches0 = gkv.gkv_launch_count(cache.ctx)
    t0, t1 = ev(), ev()
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    t0.record()
    for k in range(steps):
        period(timers[k])
    t1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    launches = gkv.gkv_launch_count(cache.ctx) - launches0
    cache.poll()
    r = {"total_ms": t0.elapsed_time(t1),
         "plain_ms": sum(t[0].elapsed_time(t[1]) for t in timers) / (steps * (s - w)),
         "window_ms": sum(t[1].elapsed_time(t[2]) for t in timers) / (steps * w),
         "evict_ms": sum(t[2].elapsed_time(t[3]) for t in timers) / steps,
         "moved": moved, "launches": int(launches), "clocks": clocks, "ring": ring, "e2e": None}

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
    if e2e_steps > 0:
        host_in = [tuple(x.cpu().pin_memory() for x in st) for st in steps_in]
        host_out = torch.empty((L, B, Hq, d), dtype=torch.bfloat16).pin_memory()
        host_kept = torch.empty((L, B, H, b), dtype=torch.int32).pin_memory()

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
        for _ in range(e2e_steps):
            period_host()
        e1.record()
        torch.cuda.synchronize()
        barrier()
        e_ms = max_over_ranks(e0.elapsed_time(e1))
        h2d = sum(x.numel() * 2 for x in host_in[0]) * s
        d2h = host_out.numel() * 2 * s + host_kept.numel() * 4
        r["e2e"] = {"value": world * B * s * e2e_steps / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e_ms / e2e_steps}
        cache.poll()
        del host_in, host_out, host_kept
    cache.close()
    del cache, steps_in, out, kept
    torch.cuda.empty_cache()
    return r


def loop_report(name: str, sh: dict, r: dict, peaks: dict, redundancy=None) -> tuple[dict, dict, dict]:
    """Roofline of the decode kernel, eviction figures and decode summary from the timings of time_period_loop."""
    L, B, H, d, b, w, s = (sh[k] for k in ("n_layers", "batch", "h_kv", "d", "b", "w", "s"))
    peak_gbs = peaks["hbm_gbs"]
    decode_ms = (r["plain_ms"] * (s - w) + r["window_ms"] * w) / s
    n_plain = [b + t + 1 for t in range(s - w)]
    n_win = [b + t + 1 for t in range(s - w, s)]
    bytes_plain = sum(algorithmic_bytes(sh, n, False) for n in n_plain) / len(n_plain)
    bytes_win = sum(algorithmic_bytes(sh, n, True) for n in n_win) / len(n_win)
    bytes_avg = (bytes_plain * (s - w) + bytes_win * w) / s
    ach = bytes_avg / (decode_ms * 1e-3) / 1e9
    ratio = NCU_TRAFFIC_RATIO.get(name)
    roofline = {"kernel": "gkv_decode_kernel", "bound": "hbm", "achieved": ach, "peak": peak_gbs, "unit": "GB/s",
                "frac": ach / peak_gbs, "peak_source": peaks["source"],
                "traffic": ratio * bytes_avg if ratio else None,
                "traffic_source": ("not measured in this run: algorithmic bytes x 1.013, the ratio an ncu capture of a 4-layer "
                                   "stack of the same shape gave (traffic grows in proportion to units)") if ratio else None,
                "algorithmic_bytes_per_launch": bytes_avg, "avg_launch_ms": decode_ms,
                "plain_steps": {"ms": r["plain_ms"], "GBps": bytes_plain / (r["plain_ms"] * 1e-3) / 1e9},
                "window_steps": {"ms": r["window_ms"], "GBps": bytes_win / (r["window_ms"] * 1e-3) / 1e9},
                "frac_of_nominal_8TBps": ach / 8000.0}
    if ach > peak_gbs:
        roofline["note"] = ("achieved exceeds the peak: the peak is a read+write copy benchmark, not an upper bound for a "
                            "read-mostly stream; frac_of_nominal_8TBps is the conservative figure")
    resident = 2.0 * L * B * H * (b + sh["buffer"]) * d * 2
    if resident < 126e6:
        roofline["note_l2"] = "the resident K+V fits L2: the launch is latency-bound, the fraction says so"
    eb = evict_bytes(sh, r["moved"])
    units = L * B * H
    evict_ms = r["evict_ms"]
    evict = {"kernel": "gkv_evict_fused_kernel", "ms": evict_ms, "eviction_steps_per_s": 1e3 / evict_ms,
             "scored_kv_tokens_per_s": units * (b + s) / (evict_ms * 1e-3), "moved_rows": r["moved"],
             "algorithmic_bytes": eb, "achieved_GBps": eb / (evict_ms * 1e-3) / 1e9,
             "frac": eb / (evict_ms * 1e-3) / 1e9 / peak_gbs}
    if redundancy is not None:   # the eviction then has two more launches (key norms, similarity sums on tcgen05)
        evict["redundancy"] = {"lambda": redundancy[0], "threshold": redundancy[1],
                               "note": "ms includes gkv_keynorm_kernel and gkv_redundancy_tc_kernel; GB/s and frac do not describe them",
                               "gram_flop": 2.0 * units * (b + s) * (b + s) * d}
    decode = {"ms_per_launch": decode_ms, "attention_only_tok_per_s": B / (decode_ms * 1e-3)}
    return roofline, evict, decode


def l2_note(sh: dict) -> str:
    units = sh["n_layers"] * sh["batch"] * sh["h_kv"]
    gb = 2.0 * units * (sh["b"] + sh["buffer"]) * sh["d"] * 2 / 1e9
    if gb * 1e9 > 126e6:
        return f"inputs larger than L2: every launch streams the whole resident cache ({gb:.2f} GB K+V)"
    return (f"the whole resident cache ({gb * 1e3:.1f} MB K+V) fits L2, as it does in a decode loop of this shape; "
            "no flush between launches: the launches are latency-bound")


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
    peaks = load_peaks()

    sh = workload_shape(args.workload)
    if args.layers > 0:
        sh["n_layers"] = args.layers   # reduced stack for profiler captures; not a benchmark number
    B, s = sh["batch"], sh["s"]
    warmup = max(args.warmup, 3)
    r = time_period_loop(sh, dev, steps=args.steps, warmup=warmup, ring=args.ring, seed=synth.BASE_SEED + rank,
                         gpu_index=local, red_kwargs=redundancy_kwargs(args),
                         e2e_steps=0 if args.no_e2e else max(1, min(args.steps, args.e2e_steps)), world=world)
    max_ms = max_over_ranks(r["total_ms"])
    summ = replica_summary(B * s, args.steps, max_ms, world)
    red = (args.redundancy, args.redundancy_threshold) if args.redundancy is not None else None
    roofline, evict, decode = loop_report(args.workload if args.layers <= 0 else "", sh, r, peaks, red)
    evict["overhead_frac_of_step"] = evict["ms"] / (max_ms / args.steps)

    result = {
        "metric": METRIC, "value": summ["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": summ["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": describe(args.workload, sh) + (" [REDUCED LAYER COUNT: profiling only]" if args.layers > 0 else ""),
                   "tokens_per_step": B * s, "l2": l2_note(sh), "input_ring": r["ring"], "replicas": world},
        "clocks": r["clocks"], "e2e": r["e2e"], "gpu_launches": int(r["launches"]),
        "roofline": roofline, "eviction": evict, "decode": decode,
    }
    if rank == 0 and world == 1 and not args.no_cpu:
        result["cpu_baseline"] = cpu_baseline(sh, budget_s=args.cpu_seconds)
    if rank == 0 and world == 1 and args.workload == "cfg2" and args.layers <= 0 and not args.no_configs:
        result["configs"] = other_configs(args, dev, peaks)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return result if rank == 0 else None


# ------------------------------------------------------------------------------------------
def time_evict_cell(sh: dict, dev: str, *, reps: int, stages: bool, red_kwargs: dict, peaks: dict, n_planted: int,
                    seed: int, oracle_seconds: float = 0.0, group: int = 1) -> dict:
    """One eviction step of one layer at shape `sh` with the cache at l = b + buffer rows and n_h = b - w rows of
    history: the step as it runs (`fused`: one launch reading the window sums; `recompute`: scoring launch from the
    window queries + the fused launch), the scoring launch alone and, with `stages`, every stage as its own launch.
    L2 is flushed (a 512 MB memset) before every timed region; medians of `reps` after 3 warm-up rounds.
    group > 1: the cache holds `group` layers of the shape and a timed region is the `group` per-layer launches of the
    step back to back, the way a model compresses layer by layer (every layer's rows are cold: the flush precedes the
    group); the reported time is the region's divided by `group`. The stages are always timed on one layer."""
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    batch, H, b, w = sh["batch"], sh["h_kv"], sh["b"], sh["w"]
    g, C = sh["h_q"] // H, b + sh["buffer"]
    l, n_h, units = C, b - w, batch * H
    red = bool(red_kwargs)
    cfg = gkv.make_config(**dict(sh, n_layers=group), alpha=0.8, mode=gkv.GKV_MODE_MAX, fuse_window_scores=True, **red_kwargs)
    cache = gkv.GKVCache(cfg, dev)
    case = synth.eviction_case(seed, batch=batch, h_q=sh["h_q"], h_kv=H, b=b, buffer=sh["buffer"], w=w,
                               n_planted=n_planted, device=dev)
    for layer in range(group):
        cache.k[layer].copy_(case.k); cache.v[layer].copy_(case.v); cache.f[layer].copy_(case.f_prev)
    q_win = case.q_win.unsqueeze(0).contiguous()
    sample = None
    if oracle_seconds > 0:          # the oracle's inputs: the first sequences of the cell, the GPU's own bits
        n_s = min(batch, 16)
        sample = (synth.bits(case.q_win[:n_s]), synth.bits(case.k[:n_s]), synth.bits(case.v[:n_s]), case.f_prev[:n_s].cpu().numpy())
    del case
    cache.set_state(-1, l, n_h, sh["s"], False)
    for layer in range(group):
        cache.evict_stage(layer, gkv.GKV_STAGE_SCORE, q_win)  # the window sums of this state (w * S)
    sums0, f0 = cache.sacc.clone(), cache.f.clone()
    kept = torch.empty((group, batch, H, b), dtype=torch.int32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    layers = range(group)

    def restore():
        cache.sacc.copy_(sums0); cache.f.copy_(f0)
        cache.set_state(-1, l, n_h, sh["s"], True)
        flush.zero_()

    def timed(fn):
        e0, e1 = ev(), ev()
        e0.record(); fn(); e1.record()
        return e0, e1

    def each_layer(fn):
        def run():
            for layer in layers:
                fn(layer)
        return run

    names = ["score", "fused", "recompute"] + (["redundancy", "merge", "select", "compact"] if stages else [])
    per_group = {"score", "fused", "recompute"}
    t = {k: [] for k in names}
    moved = 0.0
    l0 = gkv.gkv_launch_count(cache.ctx)
    for it in range(reps + 3):
        pairs = {}
        restore()
        pairs["score"] = timed(each_layer(lambda layer: cache.evict_stage(layer, gkv.GKV_STAGE_SCORE, q_win)))
        if stages:
            if red:
                flush.zero_()
                pairs["redundancy"] = timed(lambda: cache.evict_stage(0, gkv.GKV_STAGE_REDUNDANCY))
            flush.zero_()
            pairs["merge"] = timed(lambda: cache.evict_stage(0, gkv.GKV_STAGE_MERGE))
            flush.zero_()
            pairs["select"] = timed(lambda: cache.evict_stage(0, gkv.GKV_STAGE_SELECT, None, kept[0]))
            flush.zero_()
            pairs["compact"] = timed(lambda: cache.evict_stage(0, gkv.GKV_STAGE_COMPACT))
        restore()
        pairs["fused"] = timed(each_layer(lambda layer: cache.evict(layer, None, kept[layer])))
        moved = float((kept[0] != torch.arange(b, device=dev, dtype=torch.int32)).sum().item())
        restore()
        pairs["recompute"] = timed(each_layer(lambda layer: cache.evict(layer, q_win, kept[layer])))
        torch.cuda.synchronize()
        if it >= 3:
            for k, (e0, e1) in pairs.items():
                t[k].append(e0.elapsed_time(e1) / (group if k in per_group else 1))
    cache.poll()
    launches = gkv.gkv_launch_count(cache.ctx) - l0
    med = {k: sorted(v)[len(v) // 2] for k, v in t.items() if v}
    hbm, tf = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops"] * 1e12
    eb = evict_bytes(sh, moved)                                   # window-sum path
    flop1 = 2.0 * units * g * w * 128 * l                         # one window x keys product
    score_bytes = units * (l * 256.0 + g * w * 256.0 + 4.0 * l)   # K once, the window queries, the sums written
    score_bound = max(score_bytes / hbm, flop1 / tf)
    rec_bound = max((score_bytes + eb) / hbm, flop1 / tf)
    cell = {"b": b, "batch": batch, "w": w, "units": units, "ms": med, "moved_rows": moved,
            "fused_bytes": eb, "fused_GBps": eb / (med["fused"] * 1e-3) / 1e9,
            "fused_frac": eb / (med["fused"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "kv_bytes_resident": 2.0 * units * C * 256,
            "score_bytes": score_bytes, "score_flop": flop1,
            "score_K_GBps": score_bytes / (med["score"] * 1e-3) / 1e9,
            "score_TFLOPs": flop1 / (med["score"] * 1e-3) / 1e12,
            "score_bound": "hbm" if score_bytes / hbm >= flop1 / tf else "tensor",
            "score_frac": score_bound / (med["score"] * 1e-3),
            "recompute_frac": rec_bound / (med["recompute"] * 1e-3),
            "scored_kv_tokens_per_s": units * l / (med["recompute"] * 1e-3),
            "scored_kv_tokens_per_s_window_sums": units * l / (med["fused"] * 1e-3),
            "launches_per_timed_region": group, "gpu_launches": int(launches)}
    if red and "redundancy" in med:
        cell["redundancy_TFLOPs"] = 2.0 * units * l * l * 128 / (med["redundancy"] * 1e-3) / 1e12
    if sample is not None:
        import oracle
        qb, kb, vb, fp = sample
        n_s = qb.shape[0]
        t0 = time.perf_counter()
        oracle.evict_batch(qb, None, kb, vb, fp, h_q=sh["h_q"], l=l, n_h=n_h, b=b, w=w, alpha=0.8, mode=oracle.MODE_MAX, want_kv=True)
        dt = time.perf_counter() - t0
        cell["cpu_baseline"] = {"value": n_s * H * l / dt, "unit": "scored KV tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": f"{n_s} of {batch} sequences of the cell, one eviction step from the window queries "
                                          f"with compaction ({dt * 1e3:.0f} ms)"}
    cache.close()
    del cache, sums0, f0, kept, q_win, flush
    torch.cuda.empty_cache()
    return cell


def other_configs(args, dev: str, peaks: dict) -> dict:
    """The benchmark configurations beside the headline one, each measured the same way on a smaller budget of time."""
    import torch
    from paper_2512_00504_b200 import synth

    out = {}
    # configuration 0: one eviction step, one layer, batch 1 (2 units): launch-latency bound by construction
    sampler = ClockSampler(0); sampler.start()
    sh0 = workload_shape("cfg0")
    c0 = time_evict_cell(sh0, dev, reps=20, stages=False, red_kwargs={}, peaks=peaks, n_planted=8, seed=synth.BASE_SEED,
                         oracle_seconds=0.0 if args.no_cpu else 1.0)
    out["cfg0"] = {"workload": "config 0: single eviction step, 1 layer, batch 1, 8 q / 2 kv heads, l = 640, b = 512, w = 16 (2 units)",
                   "eviction_steps_per_s": 1e3 / c0["ms"]["recompute"], "eviction_steps_per_s_window_sums": 1e3 / c0["ms"]["fused"],
                   "cell": c0, "l2": "flushed before every timed launch; 0.66 MB of K+V: launch-latency bound",
                   "roofline": {"kernel": "gkv_evict_fused_kernel", "bound": "hbm", "achieved": c0["fused_GBps"], "peak": peaks["hbm_gbs"],
                                "unit": "GB/s", "frac": c0["fused_frac"], "algorithmic_bytes_per_launch": c0["fused_bytes"],
                                "avg_launch_ms": c0["ms"]["fused"]},
                   "cpu_baseline": c0.pop("cpu_baseline", None), "clocks": sampler.stop()}
    # configuration 1: batch-1 decode loop of one layer (4 units per launch)
    sh1 = workload_shape("cfg1")
    r1 = time_period_loop(sh1, dev, steps=max(10, args.steps), warmup=3, ring=0, seed=synth.BASE_SEED + 1, gpu_index=0, red_kwargs={})
    roof1, ev1, dec1 = loop_report("cfg1", sh1, r1, peaks)
    out["cfg1"] = {"workload": describe("cfg1", sh1), "value": sh1["batch"] * sh1["s"] * max(10, args.steps) / (r1["total_ms"] * 1e-3),
                   "unit": UNIT, "l2": l2_note(sh1), "roofline": roof1, "eviction": ev1, "decode": dec1, "clocks": r1["clocks"],
                   "gpu_launches": r1["launches"],
                   "cpu_baseline": None if args.no_cpu else cpu_baseline(sh1, budget_s=4.0, n_units=1)}
    # configuration 3: the cells of the eviction-step sweep that hold more than a few MB (batch >= 64), w = 16 and 64
    sampler = ClockSampler(0); sampler.start()
    c3 = synth.CONFIGS[3]
    cells = []
    for b in c3["b_sweep"]:
        for batch in (64, 256):
            for w in c3["w_sweep"]:
                sh = dict(n_layers=1, batch=batch, h_q=c3["h_q"], h_kv=c3["h_kv"], d=128, b=b, buffer=c3["buffer"], w=w, s=c3["s"])
                cells.append(time_evict_cell(sh, dev, reps=5, stages=False, red_kwargs={}, peaks=peaks,
                                             n_planted=math.ceil(0.01 * (b + c3["buffer"])), seed=synth.BASE_SEED + 3,
                                             oracle_seconds=0.0 if args.no_cpu else 1.0, group=args.sweep_group))
    out["cfg3"] = {"workload": "config 3: eviction-step sweep, 1 layer, 32 q / 8 kv heads, l = b + 128; cells with batch >= 64 "
                               "(python bench.py --workload cfg3 runs all 32 cells with the stages timed one by one)",
                   "l2": "flushed (512 MB memset) before every timed region; a region is the per-layer launches of "
                         f"{args.sweep_group} layers of the cell's shape back to back (every layer's rows cold), time per launch = region / {args.sweep_group}",
                   "min_fused_frac": min(c["fused_frac"] for c in cells), "min_score_frac": min(c["score_frac"] for c in cells),
                   "cells": cells, "clocks": sampler.stop()}
    # configuration 4: the 32B-shaped stress case, 77 GB of K+V resident; 3 periods in steady state after 3 warm-up periods
    sh4 = workload_shape("cfg4")
    free, _ = torch.cuda.mem_get_info()
    if free > 95e9:
        r4 = time_period_loop(sh4, dev, steps=3, warmup=3, ring=4, seed=synth.BASE_SEED + 4, gpu_index=0, red_kwargs={})
        roof4, ev4, dec4 = loop_report("cfg4", sh4, r4, peaks)
        ev4["overhead_frac_of_step"] = ev4["ms"] / (r4["total_ms"] / 3)
        out["cfg4"] = {"workload": describe("cfg4", sh4) + "; 3 timed periods in steady state after 3 warm-up periods, not the full 32768-token run",
                       "value": sh4["batch"] * sh4["s"] * 3 / (r4["total_ms"] * 1e-3), "unit": UNIT, "ms_per_step": r4["total_ms"] / 3,
                       "l2": l2_note(sh4), "roofline": roof4, "eviction": ev4, "decode": dec4, "clocks": r4["clocks"],
                       "gpu_launches": r4["launches"],
                       "cpu_baseline": None if args.no_cpu else cpu_baseline(sh4, budget_s=4.0, n_units=4)}
    else:
        out["cfg4"] = {"skipped": f"needs ~80 GB of free device memory, {free / 1e9:.0f} GB free"}
    return out


# ------------------------------------------------------------------------------------------
def run_sweep(args) -> dict:
    """Eviction-step sweep (configuration 3): 32 q / 8 kv heads, one layer, b x batch x w cells, l = b + 128.
    Per cell the stages (score, merge, select, compact) are timed as separate launches, then the step as it
    runs in production: one fused launch reading the window sums, and the recompute path (score launch +
    fused launch). The JSON line carries the largest cell; `sweep` holds every cell."""
    import torch
    import paper_2512_00504_b200 as gkv
    from paper_2512_00504_b200 import synth

    dev = "cuda:0"
    torch.cuda.set_device(0)
    gkv.build_library()
    c3 = synth.CONFIGS[3]
    peaks = load_peaks()
    peak_gbs, peak_tf = peaks["hbm_gbs"], peaks["bf16_tflops"]
    reps = max(3, args.steps)
    cells = []
    sampler = ClockSampler(0)
    sampler.start()
    pick = lambda arg, sweep: tuple(int(x) for x in arg.split(",")) if arg else sweep
    for b in pick(args.sweep_b, c3["b_sweep"]):
        for batch in pick(args.sweep_batch, c3["batch_sweep"]):
            for w in pick(args.sweep_w, c3["w_sweep"]):
                sh = dict(n_layers=1, batch=batch, h_q=c3["h_q"], h_kv=c3["h_kv"], d=128, b=b, buffer=c3["buffer"], w=w, s=c3["s"])
                cells.append(time_evict_cell(sh, dev, reps=reps, stages=True, red_kwargs=redundancy_kwargs(args), peaks=peaks,
                                             n_planted=math.ceil(0.01 * (b + c3["buffer"])), seed=synth.BASE_SEED + 3,
                                             group=args.sweep_group))
    clocks = sampler.stop()
    top = cells[-1]
    return {"metric": "scored KV tokens/s of one eviction step (score from the window queries + merge + top-(b-w) + compaction)",
            "value": top["scored_kv_tokens_per_s"], "unit": "tok/s", "n_gpus": 1, "steps": reps, "warmup": 3,
            "ms_per_step": top["ms"]["recompute"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config 3 sweep, largest cell: 1 layer, batch {top['batch']}, 32 q / 8 kv heads, d 128, b={top['b']}, "
                                   f"buffer=128, w={top['w']}, l={top['b'] + 128}; step = one eviction step",
                       "l2": "flushed (512 MB memset) before every timed region; fused / recompute / score regions are the per-layer "
                             f"launches of {args.sweep_group} layers back to back, stages are single launches"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(sum(c["gpu_launches"] for c in cells)),
            "roofline": {"kernel": "gkv_evict_fused_kernel", "bound": "hbm", "achieved": top["fused_GBps"], "peak": peak_gbs,
                         "unit": "GB/s", "frac": top["fused_frac"], "peak_source": peaks["source"], "traffic": None,
                         "algorithmic_bytes_per_launch": top["fused_bytes"], "avg_launch_ms": top["ms"]["fused"]},
            "score_kernel": {"TFLOPs": top["score_TFLOPs"], "frac_of_bf16_peak": top["score_TFLOPs"] / peak_tf, "peak_TFLOPs": peak_tf,
                             "flop_counted": "one window x keys product (the kernel computes it twice)"},
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
    """The oracle arm: the same metric and configuration computed by the CPU oracle on the host cores. Every one of
    the --warmup + --steps steps times a bounded sample of the workload (a number of (layer, sequence) pairs, a few
    decode steps and one eviction) and extrapolates it to a period; the per-step sample is sized so that the whole run
    ends within a few minutes. Rank 0 only."""
    if int(os.environ.get("RANK", 0)) != 0:
        return None
    import oracle
    oracle.build()
    sh = workload_shape(args.workload)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    per_step = max(0.5, min(args.cpu_seconds, 120.0 / (steps + warmup)))
    n_units = 64 if per_step >= 4.0 else 16
    for _ in range(warmup):
        cpu_baseline(sh, budget_s=per_step, n_units=n_units)
    vals = []
    t0 = time.perf_counter()
    for _ in range(steps):
        vals.append(cpu_baseline(sh, budget_s=per_step, n_units=n_units))
    wall = time.perf_counter() - t0
    base = vals[-1]
    value = sum(v["value"] for v in vals) / len(vals)
    B, s = sh["batch"], sh["s"]
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": 1e3 * B * s / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(args.workload, sh), "tokens_per_step": B * s,
                       "note": f"CPU oracle on the host cores; each of the {warmup} + {steps} steps times a bounded sample "
                               f"({n_units} (layer, sequence) pairs, budget {per_step:.1f} s) and extrapolates it to a period: "
                               f"ms_per_step is the extrapolated period, the run itself took {wall:.0f} s"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": base["cores"], "kind": "oracle", "sample": base["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall, "wall_ms_per_step": 1e3 * wall / steps}


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
    ap.add_argument("--sweep-group", type=int, default=4,
                    help="cfg3: per-layer launches timed back to back between one pair of events (layers of the cell's shape)")
    ap.add_argument("--redundancy", type=float, default=None, metavar="LAMBDA",
                    help="select on LAMBDA * F - (1 - LAMBDA) * R' (redundancy term on; adds two launches per eviction)")
    ap.add_argument("--redundancy-threshold", type=float, default=0.5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="default workload only: leave the other configurations out")
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
