#!/usr/bin/env python
"""Benchmark of the ShotKV hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the prefill hot path (window scoring, per-shot reduce, shot selection,
K/V compaction) over one batch of the long-context workload (config 3: 4 prompts x 32 layers x
32,768 tokens, 8 KV heads, d=128, window 64, budget 10%).  `value` is prompt tokens compressed
per second with the inputs resident in HBM; `e2e` is the same through the host-buffer entry
point with the host<->device copies inside the timed region; `decode` reports decode steps/s on
config 4 (batch 8 x 32 layers, 1,024 steps, evict to 25% every 32 steps) starting from a
config-2-shaped compressed cache.  Rank 0 prints one JSON line.

Multi-GPU: (prompt, layer) units are independent, so each rank compresses its own batch of
prompts (weak scaling); the only communication is the barrier and the max-over-ranks of the
device-side time.

`--impl reference` times the fp64 CPU oracle on the host cores on a bounded sample of the same
workload and prints the same line shape.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2502_01941_b200 import workloads as wl

METRIC = "prompt tokens compressed/sec"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0            # an earlier burst measurement on this machine, used only without MEASURED_PEAKS.json
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0  # the same, back to back under the power cap
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, one ncu capture each) per algorithmic
# byte of the scoring kernel and of the two decode score kernels, taken on reduced copies of the
# workloads (config 3 with B=1, L=8; config 4 with B=2) and scaled by the bytes of a full launch.
# A ratio is set to None whenever its kernel has changed since its capture.
SCORE_TC_TRAFFIC_RATIO = 1.042
SCORE_FAST_TRAFFIC_RATIO = 1.021      # the 128-row kernel on config 2 at full size
DECODE_TRAFFIC_RATIO = 1.012
DECODE_ATTEND_TRAFFIC_RATIO = 1.006
NOMINAL_HBM_GBS = 8000.0
SUSTAIN_SECONDS = 2.5           # length of the sustained repeat of the step
SCORING_MODES = {"fast": 0, "exact": 1}


# ------------------------------------------------------------------ small utilities
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peaks():
    """Dense bf16 matmul throughput of this machine's B200s in TFLOP/s: (burst, sustained, source)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return float(p["bf16_tflops"]), float(p["bf16_tflops_sustained"]), "measured"
    except Exception:
        return FALLBACK_BF16_TFLOPS, FALLBACK_BF16_TFLOPS_SUSTAINED, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-i", str(self.idx), "-lms", "50"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self, t_begin: float | None = None, t_end: float | None = None) -> dict:
        """Ends sampling; keeps the samples whose timestamp lies in [t_begin, t_end] (wall clock)."""
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        import datetime
        sm, mx, pw, reasons = [], [], [], set()
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if t_begin is not None and not (t_begin - 0.05 <= ts <= t_end + 0.05):
                    continue
                sm.append(float(parts[1])); mx.append(float(parts[2]))
                pw.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus: int):
    """(rank, world, local_rank); initialises NCCL only when launched under torchrun with N > 1."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local))
    return rank, world, local


def max_over_ranks(ms: float, world: int, device) -> float:
    if world == 1:
        return ms
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


# ------------------------------------------------------------------ workloads
def rank_config(cfg: wl.PrefillConfig, rank: int) -> wl.PrefillConfig:
    return cfg if rank == 0 else cfg.replace(cfg_id=cfg.cfg_id + 1000 * rank)


def units_variant(cfg, kind: str, chunk_tokens: int = 16):
    """The workload with other semantic units: "sentences" = units of 10-40 tokens, "chunks" = fixed
    chunks of `chunk_tokens` tokens (the remainder joins the question), "shots" = as configured."""
    if kind == "sentences":
        return cfg.replace(S=(cfg.N - cfg.question_len) // 25, shot_dist="uniform", shot_lo=10, shot_hi=40,
                           name=cfg.name + "[sentence units]")
    if kind == "chunks":
        c = chunk_tokens
        S = (cfg.N - cfg.question_len) // c
        return cfg.replace(S=S, shot_dist="uniform", shot_lo=c, shot_hi=c, question_len=cfg.N - c * S,
                           name=cfg.name + f"[{c}-token chunks]")
    return cfg


def workload_config(cfg, world: int) -> dict:
    """The `config` entry of the JSON line: the same for the GPU arm and the reference arm."""
    k_bytes = cfg.B * cfg.L * cfg.Hkv * cfg.N * cfg.d * 2
    if fits_l2(cfg):
        l2 = ("K (%.1f MB) fits in the 126 MB L2: a %d MB buffer is written before every timed step, each step "
              "between its own pair of events" % (k_bytes / 1e6, L2_FLUSH_BYTES >> 20))
    else:
        l2 = "inputs (K alone %.1f GB) larger than the 126 MB L2; no flush" % (k_bytes / 1e9)
    return {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "H": cfg.H, "Hkv": cfg.Hkv, "d": cfg.d, "N": cfg.N,
            "W": cfg.W, "S": cfg.S, "r_p": cfg.r_p, "l2": l2,
            "parallelism": f"{world} independent replica(s), one batch of prompts each"}


L2_BYTES = 126 << 20
L2_FLUSH_BYTES = 256 << 20


def fits_l2(cfg) -> bool:
    """Would K of one step stay in L2 from one timed step to the next?  (Twice the L2 is the margin.)"""
    return cfg.B * cfg.L * cfg.Hkv * cfg.N * cfg.d * 2 < 2 * L2_BYTES


def algorithmic_bytes(cfg, kept_count: np.ndarray) -> dict:
    """Bytes the method itself must move per step: all of K read once, and the kept K and V rows
    read and written once each (actual kept counts)."""
    row = cfg.d * 2
    k_read = cfg.B * cfg.L * cfg.Hkv * cfg.N * row
    gathered = int(kept_count.sum()) * cfg.Hkv * row * 2 * 2          # K and V, read + write
    return {"k_read": k_read, "kv_gathered": gathered, "total": k_read + gathered}


# ------------------------------------------------------------------ our arm
def run_ours(args):
    import paper_2502_01941_b200 as skv
    from paper_2502_01941_b200.build import build_library
    build_library()
    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ctx = skv.Context(local)
    skv.shotkv_set_scoring_mode(ctx, SCORING_MODES[args.scoring])
    skv.shotkv_set_pipeline_groups(ctx, args.groups)
    peak, peak_src = measured_peaks()

    cfg = rank_config(wl.CONFIGS[args.workload], rank)
    if args.batch or args.layers:       # reduced copies of the workload, for profiler captures only
        cfg = cfg.replace(B=args.batch or cfg.B, L=args.layers or cfg.L,
                          name=f"{cfg.name}[B={args.batch or cfg.B},L={args.layers or cfg.L}]")
    cfg = units_variant(cfg, args.units, args.chunk_tokens)
    dims = skv.make_dims(cfg.B, cfg.L, cfg.H, cfg.Hkv, cfg.d, cfg.N, cfg.W, cfg.S)
    pol = skv.make_policy(r_p=cfg.r_p)
    Q, K, V, off = wl.prefill_batch(cfg, dev)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    out = skv.alloc_prefill_outputs(dims, Mcap, device=dev)

    def step():
        skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                    out["kept_count"], Mcap, out["Kc"], out["Vc"], None, 0, out["ws"])

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier(world)
    skv.shotkv_profile_enable(ctx, True)
    launches0 = skv.shotkv_launch_count(ctx)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    t_begin = time.time()
    if fits_l2(cfg):
        # a workload that would stay in L2: evict it before every step and time the steps one by one
        flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in pairs:
            flush.zero_()
            a.record()
            step()
            b.record()
        torch.cuda.synchronize()
        ms_own = sum(a.elapsed_time(b) for a, b in pairs)
        del flush
    else:
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        ms_own = e0.elapsed_time(e1)
    barrier(world)
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end)
    launches = skv.shotkv_launch_count(ctx) - launches0
    ms_total = max_over_ranks(ms_own, world, dev)
    ms_step = ms_total / args.steps
    stages = np.array([skv.shotkv_profile_read(ctx, i) for i in range(min(args.steps, 64))])   # [calls][4]
    skv.shotkv_profile_enable(ctx, False)
    kept = out["kept_count"].cpu().numpy()
    ab = algorithmic_bytes(cfg, kept)
    score_ms, reduce_ms, select_ms, compact_ms = [float(x) for x in stages.mean(axis=0)]
    tokens = cfg.B * cfg.N * world
    value = tokens / (ms_step * 1e-3)
    achieved = ab["k_read"] / (score_ms * 1e-3) / 1e9
    logits = cfg.B * cfg.L * cfg.H * cfg.W * cfg.N                       # one ex2 per window logit
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    tiles_per_sm = cfg.B * cfg.L * cfg.Hkv * ((cfg.N + 127) // 128) / sm_count
    # ---------------- the same step repeated for seconds: what the path sustains once the clock has
    # settled under the power cap (the --steps figure above may be a burst of a few tens of ms)
    sustained = None
    if not args.no_sustained and not fits_l2(cfg):       # a repeat without flushes would run out of L2
        sustained = sustained_leg(skv, ctx, step, ms_step, cfg, ab, peak, tiles_per_sm, world, dev, local)
    # host copies of prompt 0's results, for the parity record taken beside the CPU baseline
    gpu_prompt0 = None
    if rank == 0 and world == 1 and not args.no_cpu:
        gpu_prompt0 = {k: out[k][0].cpu() for k in ("shot_scores", "keep", "kept_idx", "kept_count")}
        gpu_prompt0["Kc"] = out["Kc"][0, :PARITY_ROW_UNITS].cpu()
        gpu_prompt0["Vc"] = out["Vc"][0, :PARITY_ROW_UNITS].cpu()
        # the very bytes the timed steps read: the oracle is given these, not a second draw
        gpu_prompt0["Q"], gpu_prompt0["K"], gpu_prompt0["V"] = Q[0].cpu(), K[0].cpu(), V[0].cpu()
    # the per-clock rate is taken at the clock of the sustained region when there is one (tens of
    # samples), else at the clock sampled during the --steps region
    sm_mhz = (sustained or {}).get("score_kernel_sm_mhz") or (sustained or {}).get("clocks", {}).get("sm_mhz") or clocks.get("sm_mhz") or 1965.0
    rate_ms = sustained["stage_ms"]["score"] if sustained else score_ms
    ex2_rate = logits / (rate_ms * 1e-3) / sm_count / (sm_mhz * 1e6)
    fast_name = "score_stream_kernel" if cfg.G * cfg.W > 128 else "score_fast_kernel"
    kernel_name = {"fast": fast_name, "exact": "score_tc_kernel"}[args.scoring] + \
        " (window QK^T on tcgen05 + softmax partials), one launch per step"
    # The scoring kernel is a contraction (Q K^T: 2 d flops per window logit) fed by one pass over K,
    # followed by one exponential per logit.  Its roofline is the slower of the two machine limits:
    # K bytes / copy bandwidth, or flops / the bf16 matmul rate this GPU sustains under its power cap
    # (the steps run back to back at the cap, so the sustained figure is the one that applies; the
    # fraction of the burst figure is given beside it).
    flops = 2.0 * logits * cfg.d
    traffic_ratio = {3: SCORE_TC_TRAFFIC_RATIO, 2: SCORE_FAST_TRAFFIC_RATIO}.get(args.workload)
    tf_burst, tf_sustained, tf_src = measured_tensor_peaks()
    achieved_tf = flops / (score_ms * 1e-3) / 1e12
    hbm_rec = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "peak_source": peak_src, "unit": "GB/s",
               "frac": round(achieved / peak, 4), "floor_ms": round(ab["k_read"] / peak / 1e6, 4)}
    tensor_rec = {"bound": "tensor", "achieved": round(achieved_tf, 1), "peak": tf_sustained,
                  "peak_source": tf_src + ", sustained bf16 matmul", "unit": "TFLOP/s",
                  "frac": round(achieved_tf / tf_sustained, 4), "frac_of_burst_peak": round(achieved_tf / tf_burst, 4),
                  "floor_ms": round(flops / tf_sustained / 1e9, 4)}
    # one exponential per logit: 16 per clock per SM is what the special-function unit alone delivers
    # (measured); the kernel takes 5 of every 16 column pairs on the FMA pipe instead, so this
    # fraction may pass 1
    alu_rec = {"bound": "alu", "unit": "exp/clk/SM", "achieved": round(ex2_rate, 2), "peak": 16.0,
               "frac": round(ex2_rate / 16.0, 4), "at_sm_mhz": sm_mhz,
               "cycles_per_tile": round(rate_ms * 1e-3 * sm_mhz * 1e6 / tiles_per_sm, 1),
               "region": "sustained" if sustained else "steps"}
    first, second = (tensor_rec, hbm_rec) if tensor_rec["floor_ms"] > hbm_rec["floor_ms"] else (hbm_rec, tensor_rec)
    roofline = dict(first)
    roofline.update({
        "kernel": kernel_name,
        # measured DRAM bytes per launch: the captured ratio times the K bytes of a full launch (captures
        # exist for config 3's shape and for config 2, with shots as units; null for anything else)
        "traffic": int(traffic_ratio * ab["k_read"]) if traffic_ratio and args.scoring == "fast" and args.units == "shots" else None,
        "algorithmic_bytes_per_launch": ab["k_read"], "algorithmic_flops_per_launch": int(flops),
        "ms_per_launch": round(score_ms, 4),
        "also": [second, alu_rec]})
    path = {"bytes_per_step": ab["total"], "k_read_bytes": ab["k_read"], "kv_gathered_bytes": ab["kv_gathered"],
            "achieved_gbs": round(ab["total"] / (ms_step * 1e-3) / 1e9, 1),
            "frac_of_measured_hbm": round(ab["total"] / (ms_step * 1e-3) / 1e9 / peak, 4),
            "frac_of_nominal_8tbs": round(ab["total"] / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 4),
            "stage_ms": {"score": round(score_ms, 4), "shot_reduce": round(reduce_ms, 4), "select": round(select_ms, 4),
                         "compact": round(compact_ms, 4)},
            "compact_gbs": round(ab["kv_gathered"] / (compact_ms * 1e-3) / 1e9, 1),
            "kept_tokens_mean": float(kept.mean()), "budget_tokens": skv.shotkv_budget_tokens(dims, pol)}

    result = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
        "config": workload_config(cfg, world),
        "roofline": roofline, "path": path, "clocks": clocks, "gpu_launches": int(launches),
    }
    if sustained:
        result["sustained"] = sustained

    # ---------------- the per-token form of the step (shotkv_prefill_score: a second pass over K
    # that normalises and column-sums, then selection from token importances, then compaction)
    if not args.no_tokens and not fits_l2(cfg):          # side legs repeat the step without flushes
        imp = torch.empty(cfg.B, cfg.L, cfg.Hkv, cfg.N, dtype=torch.float32, device=dev)
        def tok_step():
            skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                        out["kept_count"], Mcap, out["Kc"], out["Vc"], imp, skv.FLAG_TOKEN_IMPORTANCE, out["ws"])
        tok_step()
        barrier(world)
        n_tok = max(2, min(args.steps, 10))
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(n_tok):
            tok_step()
        t1.record()
        barrier(world)
        tok_ms = max_over_ranks(t0.elapsed_time(t1), world, dev) / n_tok
        result["token_importance_path"] = {
            "value": round(tokens / (tok_ms * 1e-3), 1), "unit": UNIT, "ms_per_step": round(tok_ms, 4), "steps": n_tok,
            "note": "same step with SHOTKV_FLAG_TOKEN_IMPORTANCE: per-token importance materialised (two passes over K)",
            "frac_of_measured_hbm_for_two_k_reads": round((ab["total"] + ab["k_read"]) / (tok_ms * 1e-3) / 1e9 / peak, 4)}
        del imp
    # ---------------- the same tensors with sentence-sized units and with fixed 16-token chunks as the
    # semantic units (only the boundaries change): the paper's document-QA adaptation and chunk-level
    # retention.  Short timed regions; the routes they take are chosen by the library.
    if not args.no_units and args.units == "shots" and not fits_l2(cfg):
        result["short_units"] = {}
        for kind in ("sentences", "chunks"):
            cu = units_variant(cfg, kind, args.chunk_tokens)
            off_u = wl.all_shot_offsets(cu)
            dims_u = skv.make_dims(cu.B, cu.L, cu.H, cu.Hkv, cu.d, cu.N, cu.W, cu.S)
            M_u = skv.shotkv_kept_capacity(dims_u, pol, off_u)
            out_u = skv.alloc_prefill_outputs(dims_u, M_u, device=dev)

            def unit_step():
                skv.shotkv_prefill_compress(ctx, dims_u, pol, Q, K, V, off_u, out_u["shot_scores"], out_u["keep"], out_u["kept_idx"],
                                            out_u["kept_count"], M_u, out_u["Kc"], out_u["Vc"], None, 0, out_u["ws"])
            for _ in range(3):
                unit_step()
            barrier(world)
            n_u = max(3, min(args.steps, 20))
            u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            u0.record()
            for _ in range(n_u):
                unit_step()
            u1.record()
            barrier(world)
            u_ms = max_over_ranks(u0.elapsed_time(u1), world, dev) / n_u
            ab_u = algorithmic_bytes(cu, out_u["kept_count"].cpu().numpy())
            result["short_units"][kind] = {"units_per_prompt": cu.S, "ms_per_step": round(u_ms, 4), "steps": n_u,
                                           "value": round(tokens / (u_ms * 1e-3), 1), "unit": UNIT,
                                           "path_frac_of_measured_hbm": round(ab_u["total"] / (u_ms * 1e-3) / 1e9 / peak, 4)}
            del out_u
        torch.cuda.empty_cache()
    # ---------------- end to end from host buffers (rank-local, same workload)
    if not args.no_e2e:
        result["e2e"] = e2e_leg(skv, ctx, cfg, dims, pol, Q, K, V, off, Mcap, world, dev, args)
    # ---------------- decode leg
    del Q, K, V, out
    torch.cuda.empty_cache()
    if not args.no_decode:
        result["decode"] = decode_leg(skv, ctx, rank, world, dev, peak, args)
    # ---------------- CPU baseline (rank 0, N = 1 only)
    if rank == 0 and world == 1 and not args.no_cpu:
        result["cpu_baseline"], result["parity"] = cpu_baseline(cfg, off, budget_s=args.cpu_seconds, gpu=gpu_prompt0)
    ctx.close()
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def sustained_leg(skv, ctx, step, ms_step, cfg, ab, peak, tiles_per_sm, world, dev, local) -> dict:
    """Repeats the step back to back for about SUSTAIN_SECONDS (at least 600 steps) with the clocks
    sampled every 50 ms; stage times are those of the last 64 steps."""
    n = int(min(4000, max(600, SUSTAIN_SECONDS * 1e3 / ms_step)))
    sampler = ClockSampler(local)
    sampler.start()
    skv.shotkv_profile_enable(ctx, True)
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.time()
    e0.record()
    for _ in range(n):
        step()
    e1.record()
    barrier(world)
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end)
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / n
    st = np.array([skv.shotkv_profile_read(ctx, i) for i in range(64)]).mean(axis=0)
    skv.shotkv_profile_enable(ctx, False)
    # the scoring kernel's own clock: cycles and nanoseconds its first CTA ran for in the last launch
    cyc, ns = skv.shotkv_last_scoring_clock(ctx)
    kernel_mhz = cyc / ns * 1e3 if ns > 0 else None
    mhz = kernel_mhz or clocks.get("sm_mhz") or 0.0
    gbs = ab["total"] / (ms * 1e-3) / 1e9
    return {"steps": n, "seconds": round(ms * n * 1e-3, 3), "ms_per_step": round(ms, 4),
            "value": round(cfg.B * cfg.N * world / (ms * 1e-3), 1), "unit": UNIT,
            "path_gbs": round(gbs, 1), "path_frac_of_measured_hbm": round(gbs / peak, 4),
            "stage_ms": {"score": round(float(st[0]), 4), "shot_reduce": round(float(st[1]), 4),
                         "select": round(float(st[2]), 4), "compact": round(float(st[3]), 4)},
            "score_gbs": round(ab["k_read"] / (float(st[0]) * 1e-3) / 1e9, 1),
            "score_frac_of_measured_hbm": round(ab["k_read"] / (float(st[0]) * 1e-3) / 1e9 / peak, 4),
            "score_cycles_per_tile": round(float(st[0]) * 1e-3 * mhz * 1e6 / tiles_per_sm, 1) if mhz else None,
            "score_kernel_sm_mhz": round(kernel_mhz, 1) if kernel_mhz else None,
            "clocks": clocks}


def e2e_leg(skv, ctx, cfg, dims, pol, Q, K, V, off, Mcap, world, dev, args) -> dict:
    """Same metric through shotkv_prefill_compress_host: pinned host inputs and outputs, the
    host->device copies of Q/K/V and the device->host copies of every result inside the timing."""
    try:
        hQ = torch.empty(Q.shape, dtype=Q.dtype, pin_memory=True); hQ.copy_(Q)
        hK = torch.empty(K.shape, dtype=K.dtype, pin_memory=True); hK.copy_(K)
        hV = torch.empty(V.shape, dtype=V.dtype, pin_memory=True); hV.copy_(V)
        ho = skv.alloc_prefill_outputs(dims, Mcap, device="cpu")
        for k in ("shot_scores", "keep", "kept_idx", "kept_count", "Kc", "Vc"):
            ho[k] = ho[k].pin_memory()
        arena = torch.empty(skv.shotkv_host_arena_bytes(dims, Mcap), dtype=torch.uint8, device=dev)
    except RuntimeError as e:
        return {"value": None, "unit": UNIT, "error": f"could not allocate pinned host buffers: {str(e)[:100]}"}
    # bytes that cross the bus per step: Q and K are copied whole; of V only the kept tokens' rows are
    # read (the compaction kernel gathers them from the page-locked host tensor); Kc and Vc rows are
    # written to the page-locked host outputs by that kernel; the small result arrays are copied
    row_bytes = cfg.d * 2
    kept_rows = None            # filled in after the first step, from its own kept counts
    h2d_fixed = sum(t.numel() * t.element_size() for t in (hQ, hK))
    d2h_fixed = sum(ho[k].numel() * ho[k].element_size() for k in ("shot_scores", "keep", "kept_idx", "kept_count"))

    def step():
        skv.shotkv_prefill_compress_host(ctx, dims, pol, hQ, hK, hV, off, ho["shot_scores"], ho["keep"], ho["kept_idx"],
                                         ho["kept_count"], Mcap, ho["Kc"], ho["Vc"], arena)
    steps = max(2, min(args.steps, args.e2e_steps))
    step()
    barrier(world)
    kept_rows = int(ho["kept_count"].to(torch.int64).sum()) * cfg.Hkv
    h2d = h2d_fixed + kept_rows * row_bytes
    d2h = d2h_fixed + 2 * kept_rows * row_bytes
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    barrier(world)
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / steps
    return {"value": round(cfg.B * cfg.N * world / (ms * 1e-3), 1), "unit": UNIT, "ms_per_step": round(ms, 3),
            "steps": steps, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "api": "shotkv_prefill_compress_host",
            "note": "page-locked host tensors: Q and K copied whole (K in up to four groups of units, each ahead of its scoring pass), V rows of kept tokens gathered in place, Kc/Vc written in place beside the next group's upload"}


def decode_leg(skv, ctx, rank, world, dev, peak, args) -> dict:
    """Config 4: batch 8 x 32 layers; the compressed prefill cache comes from running Phase 1 on a
    config-2-shaped batch of 8 prompts; then 1,024 decode steps, evicting to 25% every 32 steps."""
    dc = wl.DECODE_CONFIG
    if args.decode_steps or args.decode_batch:
        import dataclasses
        dc = dataclasses.replace(dc, steps=args.decode_steps or dc.steps, B=args.decode_batch or dc.B)
    pc = rank_config(wl.CONFIGS[2].replace(B=dc.B), rank)
    dims = skv.make_dims(pc.B, pc.L, pc.H, pc.Hkv, pc.d, pc.N, pc.W, pc.S)
    pol = skv.make_policy(r_p=pc.r_p, r_d=dc.r_d, recompress_every=dc.recompress_every)
    Q, K, V, off = wl.prefill_batch(pc, dev)
    Mcap = skv.shotkv_kept_capacity(dims, pol, off)
    out = skv.alloc_prefill_outputs(dims, Mcap, device=dev)
    skv.shotkv_prefill_compress(ctx, dims, pol, Q, K, V, off, out["shot_scores"], out["keep"], out["kept_idx"],
                                out["kept_count"], Mcap, out["Kc"], out["Vc"], None, 0, out["ws"])
    torch.cuda.synchronize()
    del Q, K, V
    torch.cuda.empty_cache()
    kept = out["kept_count"].cpu().numpy()
    Dcap = skv.shotkv_decode_capacity(pol, dc.steps)
    Kd = torch.zeros(dc.B, dc.L, dc.Hkv, Dcap, dc.d, dtype=torch.bfloat16, device=dev)
    Vd = torch.zeros_like(Kd)
    acc = torch.zeros(dc.B, dc.L, Dcap, device=dev)
    born = torch.zeros(dc.B, dc.L, Dcap, dtype=torch.int32, device=dev)
    ws = torch.empty(skv.shotkv_decode_workspace_bytes(dims, Dcap), dtype=torch.uint8, device=dev)
    # the step inputs are drawn before the timed region: one (q, k, v) triple per step
    n_in = 64
    ins = [wl.decode_step_inputs(dc, s, dev) for s in range(n_in)]

    attn_out = torch.empty(dc.B, dc.L, dc.H, dc.d, dtype=torch.float32, device=dev)

    def run(steps, attend=False):
        """`steps` decode steps from an empty decode region; returns the K bytes (and, for the
        fused attention-output step, the V bytes as well) the score kernel had to read."""
        st = skv.shotkv_decode_init(ctx, dims, pol, Dcap, Mcap, Kd, Vd, acc, born, ws)
        bytes_read = 0
        for s in range(steps):
            q, k, v = ins[s % n_in]
            bytes_read += (int(kept.sum()) + (st.n_dec + 1) * dc.B * dc.L) * dc.Hkv * dc.d * 2 * (2 if attend else 1)
            if attend:
                skv.shotkv_decode_step_attend(ctx, st, q, k, v, out["Kc"], out["Vc"], out["kept_count"], attn_out)
            else:
                skv.shotkv_decode_step(ctx, st, q, k, v, out["Kc"], out["kept_count"])
        return bytes_read

    def timed(steps, attend):
        barrier(world)
        skv.shotkv_profile_enable(ctx, True)
        l0 = skv.shotkv_launch_count(ctx)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        nbytes = run(steps, attend)
        e1.record()
        barrier(world)
        ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
        launches = skv.shotkv_launch_count(ctx) - l0
        st_ms = np.array([skv.shotkv_profile_read(ctx, i)[:2] for i in range(min(64, steps))])
        skv.shotkv_profile_enable(ctx, False)
        return ms, launches, nbytes / steps, float(st_ms[:, 0].mean())

    run(max(args.warmup, 3) * 8)
    ms, launches, per_step_bytes, score_ms = timed(dc.steps, False)
    # the same steps with the attention output fused into the score kernel (K and V both read)
    a_steps = min(dc.steps, 256)
    run(8, True)
    a_ms, a_launches, a_bytes, a_score_ms = timed(a_steps, True)
    attend = {"metric": "decode steps/sec, attention output fused", "value": round(a_steps * world / (a_ms * 1e-3), 1),
              "unit": "steps/s", "steps": a_steps, "ms_per_step": round(a_ms / a_steps, 4), "gpu_launches": int(a_launches),
              "roofline": {"bound": "hbm", "kernel": "decode_attend_kernel (last 64 steps)",
                           "achieved": round(a_bytes / (a_score_ms * 1e-3) / 1e9, 1), "peak": peak, "unit": "GB/s",
                           "frac": round(a_bytes / (a_score_ms * 1e-3) / 1e9 / peak, 4),
                           "traffic": int(DECODE_ATTEND_TRAFFIC_RATIO * a_bytes) if DECODE_ATTEND_TRAFFIC_RATIO else None,
                           "algorithmic_bytes_per_launch": int(a_bytes), "ms_per_launch": round(a_score_ms, 4)}}
    return {"metric": "decode steps/sec", "value": round(dc.steps * world / (ms * 1e-3), 1), "unit": "steps/s",
            "note": "one step = all 8 sequences x 32 layers of one replica; value sums the replicas",
            "steps": dc.steps, "ms_per_step": round(ms / dc.steps, 4), "gpu_launches": int(launches),
            "config": {"workload": dc.name, "B": dc.B, "L": dc.L, "H": dc.H, "Hkv": dc.Hkv, "d": dc.d,
                       "prefill_kept_mean": float(kept.mean()), "r_d": dc.r_d, "recompress_every": dc.recompress_every,
                       "Dcap": Dcap},
            "roofline": {"bound": "hbm", "kernel": "decode score kernel (last 64 steps)",
                         "achieved": round(per_step_bytes / (score_ms * 1e-3) / 1e9, 1), "peak": peak, "unit": "GB/s",
                         "frac": round(per_step_bytes / (score_ms * 1e-3) / 1e9 / peak, 4),
                         "traffic": int(DECODE_TRAFFIC_RATIO * per_step_bytes) if DECODE_TRAFFIC_RATIO else None,
                         "algorithmic_bytes_per_launch": int(per_step_bytes), "ms_per_launch": round(score_ms, 4)},
            "path_frac_of_measured_hbm": round(per_step_bytes / (ms / dc.steps * 1e-3) / 1e9 / peak, 4),
            "attend": attend}


# ------------------------------------------------------------------ the oracle, timed
def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_unit_seconds(cfg, b, l, off_b, keep_result: bool = False, inputs=None):
    """Times the oracle, as it stands, on one (prompt, layer) unit of the workload: on `inputs`
    (Q, K, V of that unit as bf16 host tensors) when given, else on a draw of its own."""
    from oracle import shotkv_oracle as O
    Q, K, V = inputs if inputs is not None else wl.prefill_unit(cfg, b, l, off_b, "cpu")
    q, k, v = wl.bf16_to_f64(Q), wl.bf16_to_f64(K), wl.bf16_bits(V)
    t0 = time.perf_counter()
    ref = O.prefill_compress(q, k, v, off_b, cfg.r_p)
    dt = time.perf_counter() - t0
    if not keep_result:
        return dt
    ref["Kc_bits"] = O.compact_kv(wl.bf16_bits(K), ref["kept_idx"])
    return dt, ref


PARITY_ROW_UNITS = 4       # units whose compacted K/V rows are compared bit for bit in the parity record
SCORE_RTOL, SCORE_ATOL = 2e-3, 1e-7


def parity_of_unit(ref: dict, gpu: dict, l: int, rec: dict) -> None:
    """Folds one (prompt 0, layer l) unit into the parity record: the oracle's result `ref` (just
    computed for the CPU baseline) against what the timed GPU steps left for the same unit."""
    S = len(ref["shot_scores"])
    g_sc = gpu["shot_scores"][l, :S].numpy().astype(np.float64)
    err = np.abs(g_sc - ref["shot_scores"]) / np.maximum(np.abs(ref["shot_scores"]), 1e-300)
    rec["max_rel_score_err"] = max(rec["max_rel_score_err"], float(err.max()) if S else 0.0)
    rec["scores_within_tol"] += int(np.all(np.abs(g_sc - ref["shot_scores"]) <= SCORE_RTOL * np.abs(ref["shot_scores"]) + SCORE_ATOL))
    g_keep = gpu["keep"][l, :S].numpy()
    n = int(gpu["kept_count"][l])
    same = bool(np.array_equal(g_keep, ref["keep"]))
    rec["units_checked"] += 1
    if same:
        rec["kept_sets_equal"] += 1
        ok = n == len(ref["kept_idx"]) and np.array_equal(gpu["kept_idx"][l, :n].numpy(), ref["kept_idx"])
        rec["kept_idx_equal"] += int(ok)
        if l < gpu["Kc"].shape[0]:
            rec["kv_rows_units"] += 1
            rec["kv_rows_bit_exact"] += int(np.array_equal(wl.bf16_bits(gpu["Kc"][l, :, :n]), ref["Kc_bits"]) and
                                            np.array_equal(wl.bf16_bits(gpu["Vc"][l, :, :n]), ref["Vc"]))
    else:
        # a tie: the kept sets differ; report how close the oracle's scores of the exchanged shots are
        changed = np.nonzero(g_keep != ref["keep"])[0]
        sc = ref["shot_scores"][changed]
        gap = float((sc.max() - sc.min()) / max(abs(sc).max(), 1e-300)) if len(sc) else 0.0
        rec["ties"] += 1
        rec["closest_tie_rel_gap"] = gap if rec["closest_tie_rel_gap"] is None else min(rec["closest_tie_rel_gap"], gap)
        rec["widest_tie_rel_gap"] = gap if rec["widest_tie_rel_gap"] is None else max(rec["widest_tie_rel_gap"], gap)
        rec["tie_units"].append(int(l))
        rec["ties_beyond_tolerance"] += int(gap > 2 * SCORE_RTOL)      # must stay 0: such a difference is an error, not a tie


def cpu_baseline(cfg, off, budget_s: float = 20.0, gpu: dict | None = None):
    """The fp64 oracle on the host cores, on as many (prompt 0, layer l) units of the same workload
    as fit in about `budget_s` seconds.  One unit = N tokens of one layer; a prompt is L units.
    With `gpu` (host copies of the timed steps' outputs for prompt 0) the oracle's results for those
    units are also compared with them: returns (baseline, parity record)."""
    rec = {"units_checked": 0, "sample": "", "score_tol": f"{SCORE_RTOL}*|ref| + {SCORE_ATOL}", "max_rel_score_err": 0.0,
           "scores_within_tol": 0, "kept_sets_equal": 0, "kept_idx_equal": 0, "kv_rows_units": 0, "kv_rows_bit_exact": 0,
           "ties": 0, "ties_beyond_tolerance": 0, "closest_tie_rel_gap": None, "widest_tie_rel_gap": None, "tie_units": []}
    t_total, n_units = 0.0, 0
    while t_total < budget_s and n_units < cfg.L:
        ins = (gpu["Q"][n_units], gpu["K"][n_units], gpu["V"][n_units]) if gpu is not None else None
        dt, ref = oracle_unit_seconds(cfg, 0, n_units, off[0], keep_result=True, inputs=ins)
        t_total += dt
        if gpu is not None:
            parity_of_unit(ref, gpu, n_units, rec)
        n_units += 1
    tokens_per_s = cfg.N / (t_total / n_units * cfg.L)
    base = {"value": round(tokens_per_s, 2), "unit": UNIT, "cores": oracle_threads(), "host_cpus": os.cpu_count(),
            "kind": "oracle", "sample": f"{n_units} of {cfg.B * cfg.L} (prompt, layer) units of {cfg.name} "
                                        f"({n_units * cfg.N} token-layers) in {t_total:.1f} s; scaled to whole prompts"}
    rec["sample"] = (f"prompt 0, layers 0..{n_units - 1} of the timed workload: the units the CPU baseline ran; a tie is a unit "
                     "whose kept set differs from the oracle's (gap = spread of the oracle's scores over the exchanged shots)")
    rec["max_rel_score_err"] = float(f"{rec['max_rel_score_err']:.3e}")
    return base, (rec if gpu is not None else None)


def run_reference(args):
    """The reference arm is the oracle itself (there is no reference implementation to install):
    each step compresses a bounded sample -- one (prompt, layer) unit -- of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = wl.CONFIGS[args.workload]
    off = wl.all_shot_offsets(cfg)
    steps, warm = min(args.steps, 8), min(max(args.warmup, 1), 2)
    for i in range(warm):
        oracle_unit_seconds(cfg, 0, i % cfg.L, off[0])
    t = [oracle_unit_seconds(cfg, 0, (warm + i) % cfg.L, off[0]) for i in range(steps)]
    sec = sum(t) / steps
    value = cfg.N / (sec * cfg.L)
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": round(sec * 1e3, 2), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, args.gpus),
            "cpu_baseline": {"value": round(value, 2), "unit": UNIT, "kind": "oracle", "cores": oracle_threads(),
                             "sample": f"each step = one (prompt, layer) unit of {cfg.name} ({cfg.N} token-layers); "
                                       f"tokens/s scaled by L = {cfg.L} layers per prompt"},
            "e2e": {"value": round(value, 2), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=[1, 2, 3], help="prefill config timed as the step")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--batch", type=int, default=0, help="override B (profiler captures of a smaller case)")
    ap.add_argument("--layers", type=int, default=0, help="override L (profiler captures of a smaller case)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the number of decode steps")
    ap.add_argument("--decode-batch", type=int, default=0, help="override the decode batch (profiler captures)")
    ap.add_argument("--units", default="shots", choices=["shots", "sentences", "chunks"],
                    help="semantic units of the timed workload: the config's few-shot examples (default), sentence-sized "
                         "units of 10-40 tokens (the document-QA adaptation), or fixed chunks of 16 tokens")
    ap.add_argument("--chunk-tokens", type=int, default=16, help="chunk length for --units chunks")
    ap.add_argument("--scoring", default="fast", choices=sorted(SCORING_MODES),
                    help="scoring kernel: the default pair (fast kernel + exact repair) or the exact kernel alone")
    ap.add_argument("--groups", type=int, default=0, choices=[0, 1, 2, 3, 4],
                    help="groups of units the fused call pipelines (0: the library's choice; 1: no overlap of steps)")
    ap.add_argument("--no-tokens", action="store_true", help="skip the per-token-importance form of the step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-units", action="store_true", help="skip the sentence-unit and chunk-unit forms of the step")
    ap.add_argument("--no-sustained", action="store_true", help="skip the seconds-long repeat of the step")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
