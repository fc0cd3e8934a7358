#!/usr/bin/env python
"""Benchmark: token-reduced prefill of the 12-layer hybrid Mamba-2/attention stack on B200.

One "step" = one whole prefill of the stack (all layers: projections, conv, scan, importance score,
top-K select, compaction, attention) over one synthetic batch.  Metric: tokens/s = Bz*(N+M)/time.
Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a bounded sample.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "token-reduced prefill tokens/s per layer stack"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# Measured DRAM traffic / algorithmic bytes of one launch, from the ncu captures summarised under profiles/
# (smaller cases of the same kernels; traffic grows in proportion to the algorithmic bytes).  A kernel that
# has changed since its capture is left out (traffic is then reported as null).
NCU_TRAFFIC_RATIO = {"gemm": 514.1 / 343.2, "ssd_scan": 115.1 / 157.9, "mamba_score": 86.7 / 84.0, "compact": 226.6 / 270.7}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def workload(args):
    from paper_2603_00198_b200 import inputs
    cfg = dict(inputs.CONFIGS["C3"])
    cfg["ffn_dim"] = 0
    if args.pattern:
        # secondary workloads: any sequence of Mamba-2 / attention / FFN layers (e.g. the hybrid's M F ... A F
        # interleaving or an attention + FFN Transformer), three equal retention stages unless told otherwise
        cfg["pattern"] = args.pattern
        cfg["ffn_dim"] = args.ffn_dim or 4 * cfg["mamba"]["D"]
        cfg["alpha_bp"] = inputs.sweep_alpha_bp(args.final_bp or 2500, len(args.pattern))
    if args.n_vis:
        cfg["n_vis"] = args.n_vis
    if args.final_bp:
        cfg["alpha_bp"] = inputs.sweep_alpha_bp(args.final_bp, len(cfg["pattern"]))
    if args.schedule == "sigmoid":
        # all-layer sigmoid retention (the paper's appendix: k = 20, start 1.0, end 0.125, midpoint x0): every
        # layer cuts a little, so the attention layers select inside the stack as well
        from paper_2603_00198_b200 import binding
        cfg["alpha_bp"] = binding.str_sigmoid_schedule_bp(len(cfg["pattern"]), 20.0, args.x0, 1.0, 0.125)
    cfg["batch"] = args.batch
    return cfg


# ------------------------------------------------------------------ algorithmic work per category
def work_model(cfg, keep_counts):
    """Algorithmic flops / bytes of one step, per kernel category: 2 M N K per product and one read + one write of
    every operand for the GEMMs, the causal chunked count for the scan, the score / select / gather byte counts."""
    ms, at = cfg["mamba"], cfg["attn"]
    D, M, Bz = ms["D"], cfg["n_text"], cfg["batch"]
    H, p, n, G, Q = ms["H"], ms["p"], ms["n"], ms["G"], ms["Q"]
    Hq, Hkv, d = at["Hq"], at["Hkv"], at["d"]
    d_inner, gn = H * p, G * n
    dip, dqkv = 2 * d_inner + 2 * gn + H, (Hq + 2 * Hkv) * d
    w = {k: dict(flops=0.0, bytes=0.0) for k in
         ("gemm", "ssd_scan", "mamba_score", "attn_score", "topk", "compact", "attn_fwd")}
    n_cur = cfg["n_vis"]
    for kind, K in zip(cfg["pattern"], keep_counts):
        T = n_cur + M
        To = min(K, n_cur) + M          # a reducing layer projects only the rows it keeps
        if kind == "F":
            F = cfg["ffn_dim"]
            w["gemm"]["flops"] += 4.0 * Bz * T * D * F
            w["gemm"]["bytes"] += 2.0 * (2 * Bz * T * (D + F) + 2 * D * F + Bz * T * D)
        elif kind == "M":
            # a reducing layer projects the gate z (d_inner of the dip columns) for the rows it keeps only
            w["gemm"]["flops"] += 2.0 * Bz * D * (T * (dip - d_inner) + To * d_inner) + 2.0 * Bz * To * d_inner * D
            w["gemm"]["bytes"] += 2.0 * (Bz * T * (D + dip - d_inner) + Bz * To * (D + d_inner) + D * dip) \
                + 2.0 * (Bz * To * (d_inner + 2 * D) + d_inner * D)
            w["ssd_scan"]["flops"] += Bz * T * (G * 2 * n * (Q + 1) / 2 + H * (2 * p * (Q + 1) / 2 + 4 * n * p))
            w["ssd_scan"]["bytes"] += Bz * T * (2 * (2 * H * p + 2 * G * n) + 4 * H)
            if K < n_cur:
                w["mamba_score"]["flops"] += Bz * n_cur * 2.0 * M * n * G
                w["mamba_score"]["bytes"] += Bz * n_cur * (2 * G * n + 4 * H + 4)
        else:
            w["gemm"]["flops"] += 2.0 * Bz * T * D * dqkv + 2.0 * Bz * To * Hq * d * D
            w["gemm"]["bytes"] += 2.0 * (Bz * T * (D + dqkv) + D * dqkv) + 2.0 * (Bz * To * (Hq * d + 2 * D) + Hq * d * D)
            w["attn_fwd"]["flops"] += Bz * Hq * 4.0 * d * T * (T + 1) / 2
            w["attn_fwd"]["bytes"] += Bz * T * 2.0 * (2 * Hq * d + 2 * Hkv * d)
            if K < n_cur:
                w["attn_score"]["flops"] += 2 * Bz * n_cur * 2.0 * M * d * Hq
                w["attn_score"]["bytes"] += 2 * Bz * n_cur * 2.0 * Hkv * d
        if K < n_cur:
            w["topk"]["bytes"] += Bz * (4.0 * n_cur + 4.0 * K)
            w["compact"]["bytes"] += Bz * 2.0 * (K + M) * (2 * D + 8)       # residual rows, positions, index map
            if kind == "A":
                w["compact"]["bytes"] += Bz * 2.0 * (K + M) * 2 * Hq * d     # the survivors' query rows
            n_cur = K
    return w


BOUND = {"gemm": "tensor", "attn_fwd": "tensor", "ssd_scan": "tensor", "mamba_score": "hbm", "attn_score": "tensor",
         "topk": "hbm", "compact": "hbm"}


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index, interval_ms=100):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", str(int(interval_ms))], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["sm_max_mhz"] = float(max(mx))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------ CPU oracle leg
def oracle_sample_tokens_per_s(cfg, n_vis_s, n_text_s, seed):
    """Times the fp64 oracle, as it stands, on a short sequence with the full layer shapes and the
    same schedule.  Returns (tokens/s, seconds, threads)."""
    import oracle
    from paper_2603_00198_b200 import inputs
    layers = inputs.stack_params(seed, cfg["pattern"], cfg["mamba"], cfg["attn"], cfg["dtype"], ffn_dim=cfg.get("ffn_dim", 0))
    h0 = inputs.hidden_inputs(seed, n_vis_s + n_text_s, cfg["mamba"]["D"], cfg["dtype"])[0]
    K = oracle.schedule_keep_counts(cfg["alpha_bp"], n_vis_s, 0, cfg["pattern"])
    t0 = time.perf_counter()
    oracle.stack_prefill(h0, n_text_s, layers, K, oracle.round_to_bf16)
    sec = time.perf_counter() - t0
    return (n_vis_s + n_text_s) / sec, sec, layers


def oracle_whole_config(name):
    """The oracle on one whole single-layer configuration (C0: tiny fp32 Mamba-2 layer, C1: 8B-class Mamba-2 layer),
    inputs and weights as the configuration states them.  Returns seconds and tokens/s."""
    import oracle
    from paper_2603_00198_b200 import inputs
    cfg = inputs.CONFIGS[name]
    layers = inputs.stack_params(cfg["seed"], "M", cfg["shape"], cfg["shape"], cfg["dtype"])
    T = cfg["n_vis"] + cfg["n_text"]
    h0 = inputs.hidden_inputs(cfg["seed"], T, cfg["shape"]["D"], cfg["dtype"])[0]
    K = oracle.schedule_keep_counts([cfg["keep_bp"]], cfg["n_vis"], 0)
    rnd = oracle.round_to_bf16 if cfg["dtype"] == "bf16" else oracle._identity
    t0 = time.perf_counter()
    oracle.stack_prefill(h0, cfg["n_text"], layers, K, rnd)
    sec = time.perf_counter() - t0
    return {"seconds": sec, "tokens_per_s": T / sec, "tokens": T}


def run_reference(args):
    """--impl reference: the oracle on host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2603_00198_b200 import inputs
    cfg = workload(args)
    cores = os.cpu_count() or 1
    n_text_s = 16
    n_vis_s = args.ref_tokens - n_text_s
    layers = inputs.stack_params(cfg["seed"], cfg["pattern"], cfg["mamba"], cfg["attn"], cfg["dtype"], ffn_dim=cfg.get("ffn_dim", 0))
    h0 = inputs.hidden_inputs(cfg["seed"], n_vis_s + n_text_s, cfg["mamba"]["D"], cfg["dtype"])[0]
    K = oracle.schedule_keep_counts(cfg["alpha_bp"], n_vis_s, 0, cfg["pattern"])

    def step():
        oracle.stack_prefill(h0, n_text_s, layers, K, oracle.round_to_bf16)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    sec = (time.perf_counter() - t0) / max(1, args.steps)
    val = (n_vis_s + n_text_s) / sec
    sample = ("fp64 oracle stack_prefill, full layer shapes, %d visual + %d text tokens per step, same schedule"
              % (n_vis_s, n_text_s))
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "C3 12-layer hybrid stack [M,M,M,M,M,A]x2 (sampled: %d tokens)" % (n_vis_s + n_text_s),
                   "schedule_bp": cfg["alpha_bp"]},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def max_over_ranks(values, world, device):
    """Element-wise maximum of per-rank timings over all ranks (every rank gets the result).  The path does
    not shard, so this reduction of the measured times is the only collective the benchmark makes."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_tokens_per_s(tokens_per_rank, world, ms_step_max):
    """Whole-job throughput of `world` independent replicas: all ranks' tokens over the slowest rank's time."""
    return tokens_per_rank * world / (ms_step_max * 1e-3)


# ------------------------------------------------------------------ GPU arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2603_00198_b200 import binding, inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    cfg = workload(args)
    Bz, n_vis, M, D = cfg["batch"], cfg["n_vis"], cfg["n_text"], cfg["mamba"]["D"]
    T0 = n_vis + M
    K = binding.str_schedule_keep_counts_layers(cfg["alpha_bp"], cfg["pattern"], n_vis, cfg["min_keep"])

    ctx = binding.Context(local)
    # weights: seeded on the host, one replica per rank (the path does not shard: replicas only)
    layers = inputs.stack_params(cfg["seed"], cfg["pattern"], cfg["mamba"], cfg["attn"], "f32", ffn_dim=cfg["ffn_dim"])
    stack = binding.Stack(ctx, layers, cfg["dtype"], Bz, n_vis, M, K, Q=cfg["mamba"]["Q"], mamba_score=args.mamba_score,
                          attn_denominator=args.attn_denominator)
    del layers
    h_host = torch.from_numpy(inputs.hidden_inputs(cfg["seed"] + 1000 * rank, T0, D, "bf16", batch=Bz)).to(torch.bfloat16)
    h_pin = h_host.pin_memory()
    h_dev = h_pin.cuda()
    out_pin = torch.empty((Bz, K[-1] + M, D), dtype=torch.bfloat16).pin_memory()
    idx_pin = torch.empty((Bz, K[-1] + M), dtype=torch.int32).pin_memory()
    ctx.workspace(max(stack.ws_bytes, stack.host_ws_bytes))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    for _ in range(args.warmup):
        binding.str_stack_prefill(stack, h_dev)
    ctx.check_status()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    l0 = ctx.launch_count()
    tc0, fb0 = ctx.path_counts()
    ctx.profile_enable(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        out, pos, idx = binding.str_stack_prefill(stack, h_dev)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    ctx.profile_enable(False)
    prof = ctx.profile_collect()
    ms_graph = None
    if args.graph:
        # the same step captured once into a CUDA graph and replayed: the stack call only enqueues kernels and
        # device-to-device copies on the caller's stream, so it can be captured after a warm-up call
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            g_out, g_pos, g_idx = binding.str_stack_prefill(stack, h_dev)
        gr.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(args.steps):
            gr.replay()
        g1.record()
        torch.cuda.synchronize()
        ms_graph = g0.elapsed_time(g1) / args.steps
        assert bool((g_out == out).all()) and bool((g_idx == idx).all())
    launches = ctx.launch_count() - l0
    tc1, fb1 = ctx.path_counts()
    clocks = sampler.stop() if sampler else None
    ctx.check_status()
    # the headline number is a tensor-core number: no call of the timed region may have taken an fp32-FMA fallback
    if fb1 != fb0:
        raise SystemExit("bench: %d calls of the timed region fell back to the fp32-FMA kernels" % (fb1 - fb0))

    # ---- end to end through the host-buffer entry point (H2D + stack + D2H inside the timed region)
    for _ in range(max(1, min(args.warmup, 2))):
        binding.str_stack_prefill_host(stack, h_pin, out_pin, idx_pin)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(1, min(args.steps, 5))
    e0.record()
    for _ in range(e2e_steps):
        binding.str_stack_prefill_host(stack, h_pin, out_pin, idx_pin)
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    same = bool((out_pin.cuda() == out).all()) and bool((idx_pin.cuda() == idx).all())

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], world, "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_step = ms_total / args.steps
    value = aggregate_tokens_per_s(Bz * T0, world, ms_step)
    e2e_value = aggregate_tokens_per_s(Bz * T0, world, ms_e2e / e2e_steps)
    pk = peaks()
    work = work_model(cfg, K)
    kernels = {}
    for cat, (ms, calls) in prof.items():
        if calls == 0:
            continue
        per_step_ms = ms / args.steps
        ent = {"ms_per_step": per_step_ms, "calls_per_step": calls / args.steps, "share": ms / ms_total}
        if cat in work:
            wk = work[cat]
            ent["tflops"] = wk["flops"] / (per_step_ms * 1e-3) / 1e12 if wk["flops"] else None
            ent["gbs"] = wk["bytes"] / (per_step_ms * 1e-3) / 1e9
            if BOUND[cat] == "tensor":
                ent["frac_of_tensor_peak"] = ent["tflops"] / pk["bf16_tflops_sustained"]
            else:
                ent["frac_of_hbm_peak"] = ent["gbs"] / pk["hbm_gbs"]
        kernels[cat] = ent
    dom = max((c for c in kernels if c in work), key=lambda c: kernels[c]["ms_per_step"])
    if BOUND[dom] == "tensor":
        roof = {"bound": "tensor", "achieved": kernels[dom]["tflops"], "peak": pk["bf16_tflops_sustained"],
                "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": kernels[dom]["gbs"], "peak": pk["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    per_launch_bytes = work[dom]["bytes"] / kernels[dom]["calls_per_step"]
    roof["traffic"] = NCU_TRAFFIC_RATIO[dom] * per_launch_bytes if dom in NCU_TRAFFIC_RATIO else None
    roof["algorithmic_bytes_per_launch"] = per_launch_bytes
    roof["kernel"] = dom
    roof["peak_source"] = "%s (sustained figure: kernel timed inside a long step)" % pk["source"]
    roof["launch_ms"] = kernels[dom]["ms_per_step"] / kernels[dom]["calls_per_step"]

    # ---- CPU oracle on a bounded sample of the same workload (rank 0, N=1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        n_text_s = 16
        val, sec, _ = oracle_sample_tokens_per_s(cfg, args.ref_tokens - n_text_s, n_text_s, cfg["seed"])
        cpu = {"value": val, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
               "sample": "fp64 oracle stack_prefill, full layer shapes and schedule, %d visual + %d text tokens, %.1f s"
                         % (args.ref_tokens - n_text_s, n_text_s, sec),
               "whole_configs": {name: oracle_whole_config(name) for name in ("C0", "C1")}}

    # ---- the exported hot-path calls alone, at the configurations' shapes (outside the timed region; rank 0, N=1)
    alone = None
    if world == 1 and not args.no_kernels_alone:
        del out, pos, idx
        alone = []
        for name, nv, bp in KERNELS_ALONE:
            r = micro_case(ctx, pk, name, Bz=1, n_vis=nv, final_bp=bp, steps=5, warmup=3, min_seconds=0.5, gpu_index=local)
            alone.append({"kernel": name, "n_vis": nv, "ms": r["ms"], "bound": r["roofline"]["bound"],
                          "achieved": r["roofline"]["achieved"], "unit": r["roofline"]["unit"], "frac": r["roofline"]["frac"],
                          "gbs": r["gbs"], "tflops": r["tflops"], "launches_timed": r["launches_timed"], "clocks": r["clocks"]})
            torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "%s, %d visual + %d text tokens, batch %d, "
                               "schedule %s" % ("C3 12-layer hybrid stack [M,M,M,M,M,A]x2" if not args.pattern else
                                                "%d-layer stack %s (M Mamba-2, A attention, F FFN %d)" % (len(cfg["pattern"]), cfg["pattern"], cfg["ffn_dim"]),
                                                n_vis, M, Bz, "/".join(str(a // 100) for a in (cfg["alpha_bp"][::4] if args.schedule == "step"
                                                                                  else cfg["alpha_bp"]))),
                   "mamba_score": args.mamba_score, "attn_denominator": args.attn_denominator, "keep_counts": K, "l2": "inputs larger than L2 (hidden %d MB, workspace %d MB)"
                                           % (h_dev.numel() * 2 >> 20, stack.ws_bytes >> 20),
                   "multi_gpu": "replicas only (the path does not shard)"},
        "roofline": roof, "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h_pin.numel() * 2),
                "d2h_bytes_per_step": int(out_pin.numel() * 2 + idx_pin.numel() * 4), "matches_device_run": same},
        "gpu_launches": int(launches), "clocks": clocks, "kernels": kernels,
        "paths": {"tensor_core_calls": int(tc1 - tc0), "fallback_calls": int(fb1 - fb0)},
        "ms_per_step_cuda_graph": ms_graph,
        "kernels_alone": alone,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()



# ------------------------------------------------------------------ single-kernel microbenchmarks
def micro_case(ctx, pk, name, Bz=1, n_vis=32768, final_bp=5000, attn_denominator="visual", steps=5, warmup=3,
               min_seconds=0.0, gpu_index=0):
    """Times one entry point of the hot path alone (CUDA events on the launching stream, L2 flushed between launches)
    on seeded device-side inputs of the C1 / C2 layer shapes.  Returns a dict with its roofline and the SM clocks
    sampled while it ran (launches are repeated for at least `min_seconds` so that the sampler sees the GPU under
    load)."""
    import torch
    from paper_2603_00198_b200 import binding, inputs
    torch.manual_seed(1234)
    ms_, at_ = inputs.MAMBA_8B, inputs.ATTN_8B
    M = 128
    T = n_vis + M
    dev = "cuda:%d" % gpu_index
    bf = torch.bfloat16
    flops = nbytes = 0.0
    bound = "hbm"
    if name == "ssd":
        H, p, n, G, Q = ms_["H"], ms_["p"], ms_["n"], ms_["G"], ms_["Q"]
        x = torch.randn(Bz, T, H, p, device=dev).to(bf)
        Bm = torch.randn(Bz, T, G, n, device=dev).to(bf)
        Cm = torch.randn(Bz, T, G, n, device=dev).to(bf)
        dt = torch.empty(Bz, T, H, device=dev).uniform_(1e-3, 1e-1)
        A = -torch.exp(torch.empty(H, device=dev).uniform_(0.0, float(np.log(16.0))))
        fn = lambda: binding.str_mamba2_prefill(ctx, x, dt, A, Bm, Cm, Q=Q)
        flops = Bz * T * (G * 2 * n * (Q + 1) / 2 + H * (2 * p * (Q + 1) / 2 + 4 * n * p))
        nbytes = Bz * T * (2 * (2 * H * p + 2 * G * n) + 4 * H)
        bound = "tensor"
    elif name == "mamba_score":
        H, n, G = ms_["H"], ms_["n"], ms_["G"]
        Bm = torch.randn(Bz, T, G, n, device=dev).to(bf)
        Cm = torch.randn(Bz, T, G, n, device=dev).to(bf)
        dt = torch.empty(Bz, T, H, device=dev).uniform_(1e-3, 1e-1)
        fn = lambda: binding.str_mamba_importance(ctx, Bm, Cm, dt, n_vis, M)
        flops = Bz * n_vis * 2.0 * M * n * G
        nbytes = Bz * n_vis * (2 * G * n + 4 * H + 4)
    elif name == "mamba_dyn_score":
        # Full Mamba Dynamic (Eq. 1 weights): reads B of the visual rows and dt of every row, writes and re-reads
        # the bf16 high/low decay weights (64 columns per group), two products per tile
        H, n, G = ms_["H"], ms_["n"], ms_["G"]
        Bm = torch.randn(Bz, T, G, n, device=dev).to(bf)
        Cm = torch.randn(Bz, T, G, n, device=dev).to(bf)
        dt = torch.empty(Bz, T, H, device=dev).uniform_(1e-3, 1e-1)
        A = -torch.exp(torch.empty(H, device=dev).uniform_(0.0, float(np.log(16.0))))
        fn = lambda: binding.str_mamba_importance_dynamic(ctx, Bm, Cm, dt, A, n_vis, M)
        flops = Bz * n_vis * 2.0 * M * (n + 3 * H // G) * G
        nbytes = Bz * n_vis * (2 * G * n + 2 * 4 * H + 2 * 2 * G * 64 + 4)
    elif name == "attn_score":
        Hq, Hkv, d = at_["Hq"], at_["Hkv"], at_["d"]
        q = torch.randn(Bz, T, Hq, d, device=dev).to(bf)
        k = torch.randn(Bz, T, Hkv, d, device=dev).to(bf)
        fn = lambda: binding.str_attn_importance(ctx, q, k, n_vis, M, 1.0 / np.sqrt(d), denominator=attn_denominator)
        flops = 2 * Bz * n_vis * 2.0 * M * d * Hq
        nbytes = 2 * Bz * n_vis * 2.0 * Hkv * d
        bound = "tensor"
    elif name == "attn_fwd":
        Hq, Hkv, d = at_["Hq"], at_["Hkv"], at_["d"]
        q = torch.randn(Bz, T, Hq, d, device=dev).to(bf)
        k = torch.randn(Bz, T, Hkv, d, device=dev).to(bf)
        v = torch.randn(Bz, T, Hkv, d, device=dev).to(bf)
        fn = lambda: binding.str_attn_prefill(ctx, q, k, v, 1.0 / np.sqrt(d))
        flops = Bz * Hq * 4.0 * d * T * (T + 1) / 2
        nbytes = Bz * T * 2.0 * (2 * Hq * d + 2 * Hkv * d)
        bound = "tensor"
    elif name == "topk":
        K = max(1, n_vis * (final_bp or 5000) // 10000)
        sc = torch.rand(Bz, n_vis, device=dev)
        fn = lambda: binding.str_topk_select(ctx, sc, K)
        nbytes = Bz * (4.0 * n_vis + 4.0 * K)
    elif name == "compact":
        D = ms_["D"]
        K = max(1, n_vis * (final_bp or 5000) // 10000)
        hid = torch.randn(Bz, T, D, device=dev).to(bf)
        pos = torch.arange(T, device=dev, dtype=torch.int32).repeat(Bz, 1).contiguous()
        kept = torch.sort(torch.rand(Bz, n_vis, device=dev).argsort(dim=1)[:, :K], dim=1).values.to(torch.int32).contiguous()
        fn = lambda: binding.str_compact(ctx, hid, pos, pos, kept, M)
        nbytes = Bz * 2.0 * (K + M) * (2 * D + 8)
    elif name == "gemm":
        D = ms_["D"]
        N = 2 * ms_["H"] * ms_["p"] + 2 * ms_["G"] * ms_["n"] + ms_["H"]
        a = torch.randn(Bz * T, D, device=dev).to(bf)
        w = (torch.randn(N, D, device=dev) / 64.0).to(bf)
        fn = lambda: binding.str_gemm(ctx, a, w)
        flops = 2.0 * Bz * T * N * D
        nbytes = 2.0 * (Bz * T * (D + N) + N * D)
        bound = "tensor"
    else:
        raise SystemExit("unknown --micro " + name)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for _ in range(max(3, warmup)):
        fn()
    ctx.check_status()
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_index, interval_ms=50)
    times = []
    t_begin = time.perf_counter()
    while len(times) < steps or time.perf_counter() - t_begin < min_seconds:
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    ctx.check_status()
    ms = float(np.median(times))
    if bound == "tensor":
        ach, peak, unit = flops / (ms * 1e-3) / 1e12, pk["bf16_tflops"], "TFLOP/s"
    else:
        ach, peak, unit = nbytes / (ms * 1e-3) / 1e9, pk["hbm_gbs"], "GB/s"
    return {"micro": name, "batch": Bz, "n_vis": n_vis, "n_text": M, "ms": ms, "ms_min": float(min(times)),
            "launches_timed": len(times), "l2": "256 MB buffer written between launches",
            "roofline": {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                         "peak_source": pk["source"] + " (burst figure: kernel timed alone)"},
            "gbs": nbytes / (ms * 1e-3) / 1e9, "tflops": flops / (ms * 1e-3) / 1e12 if flops else None, "clocks": clocks}


# The exported hot-path calls at the shapes the benchmark configurations give them, timed alone after the headline run.
KERNELS_ALONE = [("ssd", 4096, 0), ("ssd", 32768, 0), ("mamba_score", 32768, 0), ("attn_score", 16384, 0),
                 ("topk", 32768, 5000), ("compact", 32768, 5000)]


def run_micro(args):
    """--micro NAME: one entry point alone; prints one JSON line with its roofline and clock record."""
    import torch
    from paper_2603_00198_b200 import binding
    torch.cuda.set_device(0)
    ctx = binding.Context(0)
    res = micro_case(ctx, peaks(), args.micro, Bz=args.batch, n_vis=args.n_vis or 32768, final_bp=args.final_bp,
                     attn_denominator=args.attn_denominator, steps=args.steps, warmup=args.warmup, min_seconds=args.micro_seconds)
    print(json.dumps(res))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--n-vis", type=int, default=0, help="override the visual token count (default: 32768)")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--final-bp", type=int, default=0, help="final keep budget in basis points (sweep)")
    ap.add_argument("--ref-tokens", type=int, default=256, help="tokens per step of the CPU oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--schedule", default="step", choices=["step", "sigmoid"], help="retention schedule of the stack")
    ap.add_argument("--pattern", default="", help="layer pattern of a secondary workload, e.g. MFMFAFMFMFAF or AFAFAFAF")
    ap.add_argument("--ffn-dim", type=int, default=0, help="FFN width of --pattern workloads (default 4 D)")
    ap.add_argument("--mamba-score", default="decoupled", choices=["decoupled", "full_dynamic"],
                    help="Mamba-layer importance: Eq. 2 (the method) or |w| of Eq. 1 (the paper's scoring ablation)")
    ap.add_argument("--attn-denominator", default="visual", choices=["visual", "causal_row"],
                    help="normaliser of the attention-layer importance: visual keys only (the paper's formula) or the causal row")
    ap.add_argument("--x0", type=float, default=0.11, help="midpoint of the sigmoid schedule (0.11 / 0.24 / 0.41)")
    ap.add_argument("--micro-seconds", type=float, default=0.0, help="repeat a --micro launch for at least this long, so that the clock sampler sees the GPU under load")
    ap.add_argument("--graph", action="store_true", help="also time the step replayed from a CUDA graph")
    ap.add_argument("--no-kernels-alone", action="store_true", help="skip the per-kernel timings after the headline run")
    ap.add_argument("--micro", default="", help="time one kernel alone: ssd | mamba_score | mamba_dyn_score | attn_score | attn_fwd | "
                                                "topk | compact | gemm")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.micro:
        run_micro(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
