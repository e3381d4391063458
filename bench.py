#!/usr/bin/env python
"""Throughput of the cache-conditional MoE decode step on synthetic, model-shaped workloads.

One "step" is one token of every (stream, layer): fused routing (router GEMV, softmax, cache-aware
promotion, top-k, LRU update, miss counting), expert grouping, the grouped SwiGLU expert FFN and the
weighted combine.  The metric is stream*token*layer steps per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload qwen] [--impl mcce|reference]

Prints one JSON line (rank 0).  `--impl reference` times the plain CPU oracle on the host cores on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2412_00099_b200 import synth  # noqa: E402

METRIC = "cache-aware MoE decode steps/s (stream*token*layer)"
UNIT = "steps/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM counters of the dominant kernel from an ncu capture of a small case, kept as a tracked data file beside
# its summary; the sources of the kernel are hashed into it, so that a figure taken from an older kernel is
# not reported for the current one.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ffn_up_dram_traffic.json")
KERNEL_SOURCES = ("paper_2412_00099_b200/csrc/ffn_tc.cu", "paper_2412_00099_b200/csrc/tc_common.cuh")


def kernel_sources_sha():
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_traffic(workload_name, n_layers, default_config):
    """(bytes per launch, source) of ffn_up from the tracked capture: the capture's per-layer DRAM bytes (read +
    write) times the layers of this run -- the kernel streams every layer's experts once, so its traffic grows in
    proportion to the layer count.  (None, why) when there is no capture of this workload in its default
    configuration, or when the kernel's sources have changed since the capture."""
    try:
        rec = json.load(open(TRAFFIC_FILE))
    except (OSError, ValueError):
        return None, "no capture on file"
    cap = rec.get("captures", {}).get(workload_name)
    if cap is None or not default_config:
        return None, "no capture of this configuration"
    if rec.get("kernel_sources_sha16") != kernel_sources_sha():
        return None, "kernel sources changed since the capture in profiles/%s" % os.path.basename(TRAFFIC_FILE)
    per_layer = (cap["dram_bytes_read"] + cap["dram_bytes_write"]) / cap["layers"]
    return per_layer * n_layers, "profiles/%s: %s, %d-layer capture scaled by layers (%d / %d)" % (
        os.path.basename(TRAFFIC_FILE), cap["kernel"], cap["layers"], n_layers, cap["layers"])


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="qwen", choices=sorted(synth.ALIASES))
    ap.add_argument("--cache", type=int, default=None, help="cache capacity C per (stream, layer)")
    ap.add_argument("--lam", type=float, default=None, help="promotion strength lambda")
    ap.add_argument("--layers", type=int, default=None,
                    help="fewer layers than the workload has (small cases for profiler captures; not a bench line)")
    ap.add_argument("--rerank", default="prior", choices=["prior", "maxrank", "cumsum"],
                    help="Cache-Prior (Eq. 7, the headline), or the Max-Rank / Cumsum-Threshold baselines")
    ap.add_argument("--max-rank", type=int, default=None, help="M of Max-Rank (default 2K)")
    ap.add_argument("--cum-p", type=float, default=0.5, help="p of Cumsum-Threshold")
    ap.add_argument("--lifetimes", action="store_true", help="also track and report cache lifetimes")
    ap.add_argument("--chained", action="store_true",
                    help="sequential-layer mode: the layers of a token chained through a residual stream (L rounds "
                         "of single-layer launches per step) instead of independent layers")
    ap.add_argument("--route-only", action="store_true",
                    help="routing alone (router logits, promotion, top-K, miss counting, LRU): no expert weights, "
                         "--route-tokens tokens per launch; one step = one launch")
    ap.add_argument("--route-tokens", type=int, default=8, help="tokens per launch with --route-only")
    ap.add_argument("--route-impl", default="auto", choices=["auto", "two", "fused"])
    ap.add_argument("--impl", default="mcce", choices=["mcce", "reference"])
    ap.add_argument("--ffn", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--deterministic", action="store_true",
                    help="slot-order combine on the tensor-core path (bit-identical repeats) instead of atomic adds")
    ap.add_argument("--checked", action="store_true", help="checked mode of the context (consistency kernels after each pass)")
    ap.add_argument("--step-by-step", action="store_true",
                    help="one mcce_route_step + mcce_moe_forward per token on one stream instead of mcce_pipeline_submit")
    ap.add_argument("--no-steady-state", action="store_true",
                    help="skip the 200-step steady-state region that follows a shorter timed region")
    ap.add_argument("--no-kernel-timing", action="store_true",
                    help="do not bracket each kernel with CUDA events (no roofline block; shows their overhead)")
    return ap.parse_args()


def workload_of(args):
    wl = synth.ALIASES[args.workload]
    if args.cache is not None:
        wl = wl.with_(C=args.cache)
    if args.lam is not None:
        wl = wl.with_(lam=args.lam)
    if args.layers is not None:
        wl = wl.with_(L=args.layers, name=wl.name + "[%d layers]" % args.layers)
    return wl


def config_of(wl, extra=None):
    cfg = {"workload": wl.name, "streams": wl.S, "layers": wl.L, "experts": wl.E, "top_k": wl.K, "top_j": wl.J,
           "shared_experts": wl.n_shared, "d_model": wl.d, "d_ff": wl.I, "cache_capacity": wl.C, "lambda": wl.lam,
           "seed": wl.seed}
    cfg.update(extra or {})
    return cfg


# ---------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample (used by --impl reference and by the cpu_baseline key)
def oracle_sample(wl, steps: int, warmup: int, core_seconds: float = 20.0):
    """Times the oracle (routing + FFN, layer 0, the first S_s streams) on the host cores.
    Returns (steps/s, threads, description, seconds per step)."""
    from oracle import oracle as orc
    threads = os.cpu_count() or 1
    S_s = min(wl.S, max(4, threads))
    sub = wl.with_(L=1, S=S_s)
    # inputs of layer 0 from the seeded generator (identical to the full workload's)
    Wr = sub.router()
    W = {"Wg": sub.expert_tensor(synth.T_WG), "Wu": sub.expert_tensor(synth.T_WU), "Wd": sub.expert_tensor(synth.T_WD)}
    sh = {}
    for k, tid in (("shWg", synth.T_SH_WG), ("shWu", synth.T_SH_WU), ("shWd", synth.T_SH_WD)):
        sh[k] = sub.expert_tensor(tid) if wl.n_shared else None
    rows = [(0, s) for s in range(S_s)]
    xs = [x.reshape(1, S_s, wl.d) for x in wl.hidden_trace(warmup + steps, rows=rows)]
    o = orc.Oracle(orc.OracleConfig(1, wl.E, wl.K, wl.J, wl.n_shared, wl.d, wl.I, wl.C, S_s, wl.lam, 0, 1,
                                    1 if wl.bf16 else 0), threads=threads)

    def one(x):
        z = o.logits(Wr, x)
        sel, w = o.route(z)
        return o.ffn(x, sel, w, W["Wg"], W["Wu"], W["Wd"], sh["shWg"], sh["shWu"], sh["shWd"])

    for x in xs[:warmup]:
        one(x)
    t0 = time.perf_counter()
    for x in xs[warmup:]:
        one(x)
    dt = time.perf_counter() - t0
    desc = "layer 0, first %d of %d streams, %d tokens, routing + expert FFN, %d host threads" % (
        S_s, wl.S, steps, threads)
    # the same code on one core (a fresh oracle on the first two streams, one token)
    n1 = min(2, S_s)
    o1 = orc.Oracle(orc.OracleConfig(1, wl.E, wl.K, wl.J, wl.n_shared, wl.d, wl.I, wl.C, n1, wl.lam, 0, 1,
                                     1 if wl.bf16 else 0), threads=1)
    x1 = np.ascontiguousarray(xs[-1][:, :n1])
    t1 = time.perf_counter()
    z1 = o1.logits(Wr, x1)
    sel1, w1 = o1.route(z1)
    o1.ffn(x1, sel1, w1, W["Wg"], W["Wu"], W["Wd"], sh["shWg"], sh["shWu"], sh["shWd"])
    oracle_sample.single_core = n1 / (time.perf_counter() - t1)
    return S_s * steps / dt, threads, desc, dt / steps


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload_of(args)
    # each step is one token of the bounded sample (about 0.1 s of wall time): K steps as asked, which keeps
    # the whole run within a few minutes for any K the GPU arm is run with
    steps, warmup = max(1, min(args.steps, 2000)), max(0, min(args.warmup, 50))
    value, threads, desc, sec = oracle_sample(wl, steps, warmup)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, {"sample": desc}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                             "value_one_core": oracle_sample.single_core},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi samples of the SM clock and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", gpu_id, "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 6]
        os.unlink(self.f.name)
        try:
            sm = [float(r[0]) for r in rows]
            out["sm_mhz"] = float(np.median(sm)) if sm else None
            out["sm_max_mhz"] = float(rows[0][1]) if rows else None
            out["power_w_max"] = max(float(r[2]) for r in rows) if rows else None
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [n for i, n in enumerate(names) if any("Active" == r[3 + i].strip() for r in rows)]
            out["samples"] = len(rows)
        except (ValueError, IndexError):
            pass
        return out


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except (KeyError, ValueError):
            pass
    return FALLBACK_HBM_GBS, "fallback (earlier pool measurement)"


def route_only_arm(args):
    """Routing alone on one GPU: hidden states resident in HBM, --route-tokens tokens per launch."""
    import torch

    from paper_2412_00099_b200 import binding as mb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    dev = torch.device("cuda", 0)
    wl = workload_of(args)
    n, W, K = args.route_tokens, args.warmup, args.steps
    impl = {"auto": mb.ROUTE_AUTO, "two": mb.ROUTE_TWO_KERNELS, "fused": mb.ROUTE_FUSED}[args.route_impl]
    # the expert buffers of the context are not used: smallest intermediate size, no shared experts
    eng = mb.engine_for(wl, n_shared=0, I=8, ffn_impl=mb.FFN_SIMT, route_impl=impl)
    wdt = torch.bfloat16 if wl.bf16 else torch.float32
    Wr = mb.gen_normal(torch.empty((wl.L, wl.E, wl.d), dtype=torch.float32, device=dev), wl.seed, synth.T_ROUTER,
                       std=wl.weight_std)
    eng.set_router(Wr)
    slots = 6                                                   # launches cycle over 6 * n tokens of hidden states
    hidden = torch.empty((slots * n, wl.L, wl.S, wl.d), dtype=wdt, device=dev)
    state = torch.empty(wl.L * wl.S * wl.d, dtype=torch.float32, device=dev)
    for t in range(slots * n):
        mb.gen_hidden_step(state, hidden[t], wl.seed, t, wl.rho, wl.topic_offset)
    sel = torch.empty((n, wl.L, wl.S, wl.K), dtype=torch.int32, device=dev)
    sw = torch.empty((n, wl.L, wl.S, wl.K), dtype=torch.float32, device=dev)

    def step(i):
        o = (i % slots) * n
        eng.route_step(hidden=hidden[o:o + n], n_steps=n, out=(sel, sw))

    for i in range(W):
        step(i)
    eng.profile(True)
    eng.profile_read(reset=True)
    torch.cuda.synchronize(dev)
    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler("GPU-" + str(props.uuid)) if hasattr(props, "uuid") else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(W, W + K):
        step(i)
    e1.record()
    torch.cuda.synchronize(dev)
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
    prof = eng.profile_read(reset=True)
    eng.profile(False)
    total, _ = eng.cache_stats()
    esz = 2 if wl.bf16 else 4
    EW = (wl.E + 31) // 32
    # per launch: hidden rows and results of n tokens, the router once per token, cache state in and out once
    alg = n * (wl.L * wl.S * (wl.d * esz + wl.K * 8) + wl.L * wl.E * wl.d * 4) + wl.L * wl.S * 2 * (wl.E * 4 + EW * 4 + 12)
    launches = prof["route"][1] + prof["route_gemm"][1]
    kern_ms = (prof["route"][0] + prof["route_gemm"][0]) / K
    peak, peak_src = measured_hbm_peak()
    achieved = alg / (kern_ms * 1e-3) / 1e9
    kind = {mb.ROUTER_FP32_PIPE: "fp32-pipe logits inside the route kernel", mb.ROUTER_GEMM_TAIL: "tcgen05 GEMM, then tail",
            mb.ROUTER_RESIDENT_TAIL: "router-resident tcgen05 GEMM, then tail",
            mb.ROUTER_FUSED: "router-resident tcgen05 GEMM and tail in one cooperative kernel"}[eng.router_kernel_kind(n)]
    line = {"metric": METRIC + ", routing only", "value": wl.S * wl.L * n * K / (ms_total * 1e-3), "unit": UNIT, "n_gpus": 1,
            "steps": K, "warmup": W, "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if wl.bf16 else "f32", "data": "synthetic",
            "config": config_of(wl, {"route_only": True, "tokens_per_launch": n, "kernels": kind,
                                     "l2": "hidden states of %d launches cycled (%.0f MB, larger than L2)"
                                           % (slots, slots * n * wl.L * wl.S * wl.d * esz / 1e6)}),
            "miss_rate": total[2] / max(1, total[1]),
            "roofline": {"kernel": "routing step (logits + tail)", "bound": "hbm", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src, "traffic": None,
                         "algorithmic_bytes_per_launch": alg, "avg_launch_ms": kern_ms},
            "kernels": {k: {"ms_per_step": v[0] / K, "launches": v[1]} for k, v in prof.items() if v[1]},
            "gpu_launches": launches, "clocks": clocks}
    print(json.dumps(line), flush=True)
    eng.close()


def main_arm(args):
    import torch
    import torch.distributed as dist

    from paper_2412_00099_b200 import binding as mb
    from paper_2412_00099_b200.shard import replica_seed, reduce_max, reduce_sum

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    wl = workload_of(args)
    # streams are independent: rank r owns its own S streams (weak scaling), distinguished by the seed
    seed = replica_seed(wl.seed, rank)
    ffn_impl = {"auto": mb.FFN_AUTO, "simt": mb.FFN_SIMT, "tensor": mb.FFN_TENSOR}[args.ffn]
    rerank = {"prior": mb.RERANK_CACHE_PRIOR, "maxrank": mb.RERANK_MAX_RANK, "cumsum": mb.RERANK_CUMSUM}[args.rerank]
    max_rank = min(wl.E, args.max_rank if args.max_rank is not None else 2 * wl.K)
    eng = mb.engine_for(wl, ffn_impl=ffn_impl, device=local, rerank_mode=rerank, max_rank=max_rank,
                        cum_threshold=args.cum_p, track_lifetime=args.lifetimes, deterministic=args.deterministic,
                        checked=args.checked)
    wdt = torch.bfloat16 if wl.bf16 else torch.float32

    # ---- weights, generated on the device ------------------------------------------------------------
    Wr = mb.gen_normal(torch.empty((wl.L, wl.E, wl.d), dtype=torch.float32, device=dev), seed, synth.T_ROUTER,
                       std=wl.weight_std)
    shp_up, shp_dn = (wl.L, wl.E, wl.I, wl.d), (wl.L, wl.E, wl.d, wl.I)
    Wg = mb.gen_normal(torch.empty(shp_up, dtype=wdt, device=dev), seed, synth.T_WG, std=wl.weight_std)
    Wu = mb.gen_normal(torch.empty(shp_up, dtype=wdt, device=dev), seed, synth.T_WU, std=wl.weight_std)
    Wd = mb.gen_normal(torch.empty(shp_dn, dtype=wdt, device=dev), seed, synth.T_WD, std=wl.weight_std)
    sh = [None, None, None]
    if wl.n_shared:
        for i, (tid, shp) in enumerate(((synth.T_SH_WG, (wl.L, wl.n_shared, wl.I, wl.d)),
                                        (synth.T_SH_WU, (wl.L, wl.n_shared, wl.I, wl.d)),
                                        (synth.T_SH_WD, (wl.L, wl.n_shared, wl.d, wl.I)))):
            sh[i] = mb.gen_normal(torch.empty(shp, dtype=wdt, device=dev), seed, tid, std=wl.weight_std)
    eng.set_router(Wr)
    eng.set_experts(Wg, Wu, Wd, *sh)

    # ---- hidden-state trace for warm-up + timed steps, resident in HBM ---------------------------------
    W, K = args.warmup, args.steps
    # a steady-state region of STEADY steps follows the timed one when that is shorter (a short region runs
    # before the GPU has settled at its power cap and reads a few per cent faster)
    STEADY = 200
    steady = (not args.no_steady_state) and not args.chained and K < STEADY
    n_tok = W + K + (STEADY if steady else 0)
    per_tok = wl.L * wl.S * wl.d * (2 if wl.bf16 else 4)
    if steady and n_tok * per_tok > 12e9:
        steady, n_tok = False, W + K
    if n_tok * per_tok > 24e9:
        raise SystemExit("hidden trace of %d tokens does not fit the budget; use fewer steps" % n_tok)
    hidden = torch.empty((n_tok, wl.L, wl.S, wl.d), dtype=wdt, device=dev)
    state = torch.empty(wl.L * wl.S * wl.d, dtype=torch.float32, device=dev)
    for t in range(n_tok):
        mb.gen_hidden_step(state, hidden[t], seed, t, wl.rho, wl.topic_offset)
    sel = torch.empty((1, wl.L, wl.S, wl.K), dtype=torch.int32, device=dev)
    sw = torch.empty((1, wl.L, wl.S, wl.K), dtype=torch.float32, device=dev)
    y = torch.empty((2, wl.L, wl.S, wl.d), dtype=torch.float32, device=dev)
    torch.cuda.synchronize(dev)          # the pipelined entry point reads hidden on a stream of its own

    def step(t):
        if args.chained:
            eng.decode_step_chained(hidden[t, 0])
        elif args.step_by_step:
            eng.route_step(hidden=hidden[t], out=(sel, sw))
            eng.moe_forward(hidden[t], sel[0], sw[0], out=y[0])
        else:
            # routing + grouping of this token on the library's internal stream, overlapping the previous token's experts
            eng.pipeline_submit(hidden[t], y[t & 1])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for t in range(W):
        step(t)
    eng.profile(not args.no_kernel_timing)
    eng.profile_read(reset=True)
    barrier()
    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler("GPU-" + str(props.uuid)) if hasattr(props, "uuid") else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(W, W + K):
        step(t)
    e1.record()
    barrier()
    eng.pipeline_wait()
    ms_total = reduce_max(e0.elapsed_time(e1), dev if world > 1 else None)
    clocks = sampler.stop() if sampler else {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
    prof = eng.profile_read(reset=True)
    eng.profile(False)

    units_per_step = wl.S * wl.L                      # per rank
    value = world * units_per_step * K / (ms_total * 1e-3)
    steady_rec = None
    if steady:
        barrier()
        sampler = ClockSampler("GPU-" + str(props.uuid)) if hasattr(props, "uuid") else None
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for t in range(W + K, W + K + STEADY):
            step(t)
        s1.record()
        barrier()
        eng.pipeline_wait()
        ms_steady = reduce_max(s0.elapsed_time(s1), dev if world > 1 else None)
        steady_rec = {"steps": STEADY, "value": world * units_per_step * STEADY / (ms_steady * 1e-3), "unit": UNIT,
                      "ms_per_step": ms_steady / STEADY,
                      "clocks": sampler.stop() if sampler else {"sm_mhz": None, "sm_max_mhz": None, "reasons": []},
                      "note": "the same step for %d more tokens right after the timed region" % STEADY}
    total, _ = eng.cache_stats()
    miss_rate = total[2] / max(1, total[1])
    misses = reduce_sum(total[2], dev if world > 1 else None)
    selections = reduce_sum(total[1], dev if world > 1 else None)

    # ---- roofline of the dominant kernel (gate/up projection of the grouped expert FFN) ---------------
    offsets, _ = eng.grouping()
    touched = int((np.diff(offsets, axis=1) > 0).sum()) + wl.L * wl.n_shared
    rows = wl.L * wl.S * (wl.K + wl.n_shared)
    esz = 2 if wl.bf16 else 4
    bytes_up_weights = touched * 2 * wl.d * wl.I * esz
    bytes_up = bytes_up_weights + rows * wl.d * esz + rows * wl.I * esz
    # down projection: weights + H rows; the tensor path adds into y (L*S*d fp32) in its epilogue, the
    # fp32-pipe path writes one fp32 row per (pair) for a separate combine pass
    bytes_down = touched * wl.d * wl.I * esz + rows * wl.I * esz + (
        wl.L * wl.S * wl.d * 4 if _uses_tensor(eng) else rows * wl.d * 4)
    roofline, roofline_route, kernels = None, None, {}
    if not args.no_kernel_timing:
        up_ms, up_n = prof["ffn_up"]
        peak, peak_src = measured_hbm_peak()
        up_launch_s = up_ms / max(1, up_n) * 1e-3
        # algorithmic bytes of the gate/up kernel: the gate and up matrices of every touched expert, once
        achieved = bytes_up_weights / up_launch_s / 1e9
        default_cfg = args.cache is None and args.layers is None
        traffic, traffic_src = (measured_traffic(synth.ALIASES[args.workload].name, wl.L, default_cfg)
                                if _uses_tensor(eng) else (None, "no capture of the fp32-pipe kernels"))
        roofline = {"kernel": "ffn_up (H = silu(X Wg^T) * (X Wu^T), all expert groups)", "bound": "hbm",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_source": peak_src,
                    "traffic": traffic, "traffic_source": traffic_src,
                    "algorithmic_bytes_per_launch": bytes_up_weights,
                    "algorithmic_bytes_definition": "2 * d * I * 2 B per touched expert (gate and up weights, read once)",
                    "achieved_with_activation_rows": bytes_up / up_launch_s / 1e9,
                    "avg_launch_ms": up_ms / max(1, up_n)}
        if achieved > peak:
            roofline["note"] = ("above 1: the peak is a copy (half reads, half writes); a kernel that almost only "
                                "reads can exceed it")
        kernels = {k: {"ms_per_step": v[0] / K, "launches": v[1]} for k, v in prof.items()}
        dn_ms, dn_n = prof["ffn_down"]
        kernels["ffn_down"]["achieved_gbs"] = bytes_down / (dn_ms / max(1, dn_n) * 1e-3) / 1e9
        # routing (logits + fused tail): hidden rows, the router once per layer, cache state in and out, results
        EW = (wl.E + 31) // 32
        bytes_route = wl.L * wl.S * (wl.d * esz + 2 * (wl.E * 4 + EW * 4 + 12) + wl.K * 8) + wl.L * wl.E * wl.d * 4
        route_ms = (prof["route"][0] + prof["route_gemm"][0]) / K
        kernels["route"]["achieved_gbs_with_gemm"] = bytes_route / (route_ms * 1e-3) / 1e9
        kernels["route"]["algorithmic_bytes"] = bytes_route
        kernels["route"]["frac_of_hbm_peak"] = kernels["route"]["achieved_gbs_with_gemm"] / peak
        roofline_route = {"kernel": "routing step inside the decode step (logits + tail, one token per launch)",
                          "bound": "hbm", "achieved": kernels["route"]["achieved_gbs_with_gemm"], "peak": peak,
                          "unit": "GB/s", "frac": kernels["route"]["frac_of_hbm_peak"], "traffic": None,
                          "algorithmic_bytes_per_launch": bytes_route, "avg_launch_ms": route_ms,
                          "note": "one token per launch is bound by launch and fill latency, not by HBM"}
        # grouping + gather: selections in, offsets / permutation out, hidden rows copied into expert order
        bytes_group = wl.L * wl.S * wl.K * (4 + 8) + 2 * wl.L * wl.S * wl.K * wl.d * esz
        kernels["gather"]["achieved_gbs_with_group"] = bytes_group / (
            (prof["group"][0] + prof["gather"][0]) / K * 1e-3) / 1e9

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if wl.bf16 else "f32", "data": "synthetic",
            "config": config_of(wl, {"l2": "inputs larger than L2: %.1f GB of expert weights streamed per step"
                                           % ((bytes_up + bytes_down) / 1e9),
                                     "ffn_path": "tensor" if _uses_tensor(eng) else "simt",
                                     "combine": "slot order (deterministic)" if args.deterministic else "default",
                                     "layer_mode": "chained through a residual stream" if args.chained else "independent",
                                     "call": ("mcce_decode_step_chained" if args.chained else
                                              "mcce_route_step + mcce_moe_forward per token" if args.step_by_step else
                                              "mcce_pipeline_submit (device buffers)"),
                                     "rerank": args.rerank if args.rerank == "prior" else (
                                         "maxrank M=%d" % max_rank if args.rerank == "maxrank"
                                         else "cumsum p=%g" % args.cum_p),
                                     "experts_touched_per_step": touched}),
            "miss_rate": misses / max(1, selections), "roofline": roofline, "roofline_route": roofline_route,
            "kernels": kernels,
            # kernels of this library launched in the timed region: counted by the library itself (one count per
            # bracketed launch) when kernel timing is on
            "gpu_launches": (sum(v[1] for v in prof.values()) if not args.no_kernel_timing else None),
            "clocks": clocks}
    if steady_rec:
        line["steady_state"] = steady_rec

    # ---- routing alone, several tokens per launch (state stays in registers, the GEMM sees more tiles) -----
    if not args.no_kernel_timing and wl.bf16 and n_tok >= 8 and not args.chained:
        eng.profile(True)
        eng.profile_read(reset=True)
        sel8 = torch.empty((8, wl.L, wl.S, wl.K), dtype=torch.int32, device=dev)
        sw8 = torch.empty((8, wl.L, wl.S, wl.K), dtype=torch.float32, device=dev)
        for it in range(13):
            if it == 3:
                eng.profile_read(reset=True)
            eng.route_step(hidden=hidden[:8], n_steps=8, out=(sel8, sw8))
        pr = eng.profile_read(reset=True)
        eng.profile(False)
        # with several tokens per launch the GEMM and the tail run as one kernel (no separate GEMM launches)
        us = 1e3 * (pr["route"][0] + pr["route_gemm"][0]) / max(1, pr["route"][1])
        state_bytes = 2 * (wl.E * 4 + EW * 4 + 12)
        b8 = 8 * (wl.L * wl.S * (wl.d * esz + wl.K * 8) + wl.L * wl.E * wl.d * 4) + wl.L * wl.S * state_bytes
        line["kernels"]["route"]["batched_8_tokens"] = {"us_per_launch": us, "achieved_gbs": b8 / (us * 1e-6) / 1e9,
                                                        "frac_of_hbm_peak": b8 / (us * 1e-6) / 1e9 / measured_hbm_peak()[0],
                                                        "algorithmic_bytes": b8}
        if line["roofline_route"] is not None:
            line["roofline_route"]["eight_tokens_per_launch"] = line["kernels"]["route"]["batched_8_tokens"]
        if line["roofline_route"] is not None and not args.step_by_step:
            # In the pipelined step the routing kernels run under the previous step's expert kernels, and their
            # event brackets include the time they wait for free SMs: the roofline entry is taken from launches
            # of one token that run alone, right here (ten timed launches over different tokens' hidden states).
            eng.profile(True)
            eng.profile_read(reset=True)
            for it in range(13):
                if it == 3:
                    eng.profile_read(reset=True)
                eng.route_step(hidden=hidden[it % n_tok:it % n_tok + 1], n_steps=1, out=(sel8[:1], sw8[:1]))
            pr = eng.profile_read(reset=True)
            eng.profile(False)
            ms1 = (pr["route"][0] + pr["route_gemm"][0]) / max(1, pr["route"][1])
            rr = line["roofline_route"]
            rr["avg_launch_ms"] = ms1
            rr["achieved"] = rr["algorithmic_bytes_per_launch"] / (ms1 * 1e-3) / 1e9
            rr["frac"] = rr["achieved"] / rr["peak"]
            rr["measured"] = "10 launches of one token after the timed region, not overlapped with the expert kernels"
            line["kernels"]["route"]["achieved_gbs_with_gemm"] = rr["achieved"]
            line["kernels"]["route"]["frac_of_hbm_peak"] = rr["frac"]

    if args.lifetimes:
        (n_ev, mean, sd), _ = eng.lifetimes()
        line["cache_lifetime"] = {"evictions": n_ev, "mean_tokens": mean, "sd_tokens": sd,
                                  "tokens_per_stream": n_tok}

    # ---- end to end through the host-buffer entry points ----------------------------------------------------
    if not args.no_e2e and not args.chained:
        n_e2e = max(4, min(K, 20))
        hh = torch.empty((n_e2e + 1, wl.L, wl.S, wl.d), dtype=wdt).pin_memory()
        hh.copy_(hidden[:n_e2e + 1])
        yh = torch.empty((2, wl.L, wl.S, wl.d), dtype=torch.float32).pin_memory()   # one per step in flight
        # (a) pipelined: the upload of step t+1 and the download of step t-1 overlap the compute of step t
        eng.pipeline_submit_host(hh[0], yh[0])
        eng.pipeline_wait()
        barrier()
        t0 = time.perf_counter()
        for t in range(1, n_e2e + 1):
            eng.pipeline_submit_host(hh[t], yh[t & 1])
        eng.pipeline_wait()
        dt = reduce_max(time.perf_counter() - t0, dev if world > 1 else None)
        # (b) one synchronous call per step: copy in, compute, copy out, wait
        barrier()
        t0 = time.perf_counter()
        for t in range(1, n_e2e + 1):
            eng.decode_step_host(hh[t], yh[0])
        dt_sync = reduce_max(time.perf_counter() - t0, dev if world > 1 else None)
        line["e2e"] = {"value": world * units_per_step * n_e2e / dt, "unit": UNIT,
                       "h2d_bytes_per_step": hh[0].numel() * hh.element_size(),
                       "d2h_bytes_per_step": yh[0].numel() * 4, "steps": n_e2e,
                       "call": "mcce_pipeline_submit_host / mcce_pipeline_wait (pinned host buffers; every step's "
                               "upload and download inside the timed region, overlapped with neighbouring steps)",
                       "synchronous_value": world * units_per_step * n_e2e / dt_sync,
                       "synchronous_call": "mcce_decode_step_host (copy in, compute, copy out, wait, per step)"}

    # ---- the oracle on the host cores, beside it ------------------------------------------------------------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, threads, desc, _ = oracle_sample(wl, steps=4, warmup=1)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                                "value_one_core": oracle_sample.single_core}

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def _uses_tensor(eng):
    return bool(eng.uses_tensor_path())


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        reference_arm(a)
    elif a.route_only:
        route_only_arm(a)
    else:
        main_arm(a)
