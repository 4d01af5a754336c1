#!/usr/bin/env python
"""Benchmark of the BASP attention-layer hot path on B200.

One step = one pass of the layer over one synthetic micro-batch held as N virtual ranks on one
GPU: all-to-all reshard of Q, K, V (sequence- to head-sharded), causal attention over every rank's
head slice, reverse reshard of O.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With --gpus N > 1 (launched by torchrun, one process per GPU) every GPU runs its own micro-batch
of the same shape (weak scaling; BASP groups and micro-batches are independent, so the data path
has no collective); times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2609_03151_b200 import dist as pdist  # noqa: E402
from paper_2609_03151_b200 import synth  # noqa: E402

METRIC = "attention-layer tokens/sec"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "llama3_8b_32k"          # BASELINE config 2: N=8, b=2, S=32768, 32/8 heads, D=128

# DRAM bytes (read + write) of one attention launch from an ncu capture, per workload; None = not captured.
NCU_TRAFFIC_BYTES = {
    # profiles/attn_fwd_ws_traffic_llama3_8b_32k.md: dram__bytes_read.sum + dram__bytes_write.sum of one launch
    "llama3_8b_32k": 3033940992 + 539852800,
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"],
                    bf16_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = f"/tmp/basp_clocks_{os.getpid()}.csv"
        self.proc = None
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(gpu_index)], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.out.close()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------
def oracle_sample(w: synth.Workload, budget_rows: int = 8192, seed: int = 0):
    """Time the fp64 oracle (as it stands) on a bounded sample of workload w and extrapolate to the
    full layer by exact counts.  Returns (tokens_per_s, cores, description, seconds_spent)."""
    import numpy as np
    import oracle

    t_start = time.time()
    cores = oracle.num_threads()
    # attention: every (S // budget_rows)-th row of ONE (sequence, head); independent rows, exact pair count
    S = w.S
    stride = max(1, S // budget_rows)
    gen = torch.Generator().manual_seed(seed)
    q = synth.bits(synth.randn_bf16(gen, (1, S, 1, w.D)))
    k = synth.bits(synth.randn_bf16(gen, (1, S, 1, w.D)))
    v = synth.bits(synth.randn_bf16(gen, (1, S, 1, w.D)))
    rows = np.array([(0, 0, i) for i in range(stride - 1, S, stride)], dtype=np.int32)
    t0 = time.time()
    oracle.attn_fwd_rows(q, k, v, rows)
    t_attn = time.time() - t0
    sample_pairs = float(np.sum(rows[:, 2].astype(np.float64) + 1))
    total_pairs = float(S) * (S + 1) / 2 * w.B * w.Hq
    attn_full = t_attn * total_pairs / sample_pairs
    # reshards: the oracle's element loops on the same rank/head structure with 256 tokens per rank
    ws = synth.shrink(w, 256)
    pl = oracle.plan(ws.N, ws.B, ws.S, ws.G)
    t0 = time.time()
    for H in (w.Hq, w.Hkv, w.Hkv):
        oracle.s2h(synth.random_bits((ws.N, pl.Bl, pl.T, H, w.D), seed=1), pl)
    oracle.h2s(synth.random_bits((ws.N, pl.Bl, ws.S, w.Hq // pl.K, w.D), seed=2), pl)
    t_resh = time.time() - t0
    resh_full = t_resh * (w.tokens / ws.tokens)
    desc = (f"attention: every {stride}th row of one (sequence, head) = {100 * sample_pairs / total_pairs:.4f}% "
            f"of the causal pairs, {t_attn:.1f}s; reshards: same ranks/heads at {ws.S} tokens per sequence "
            f"({100 * ws.tokens / w.tokens:.2f}% of the tokens), {t_resh:.1f}s; extrapolated by exact pair/token counts")
    return w.tokens / (attn_full + resh_full), cores, desc, time.time() - t_start


def run_reference(args, w: synth.Workload):
    """The oracle as the reference arm: rank 0 only, each step a bounded sample."""
    rank, _, world = pdist.env_world()
    if rank != 0:
        return
    vals, cores, desc = [], 0, ""
    for i in range(args.warmup + args.steps):
        v, cores, desc, _ = oracle_sample(w, budget_rows=512)
        if i >= args.warmup:
            vals.append(v)
    value = statistics.mean(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.tokens / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "N": w.N, "b": w.B, "S": w.S, "Hq": w.Hq, "Hkv": w.Hkv, "D": w.D,
                       "note": "fp64 CPU oracle on a bounded sample per step, extrapolated"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
def run_gpu(args, w: synth.Workload):
    from paper_2609_03151_b200 import binding as basp

    rank, local_rank, world = pdist.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback of the product path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = measured_peaks()

    plan = basp.basp_plan_create(w.N, w.B, w.S, w.Hq, w.Hkv, w.D, num_groups=w.G)
    N, K, T, Bl = w.N, plan.K, plan.T, plan.Bl
    gen = torch.Generator(device=dev).manual_seed(1000 + rank)

    def randn(shape):
        return torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)

    # sequence-sharded inputs, one allocation per virtual rank (N(0,1) -> bf16, seeded per GPU)
    q_seq = [randn((Bl, T, w.Hq, w.D)) for _ in range(N)]
    k_seq = [randn((Bl, T, w.Hkv, w.D)) for _ in range(N)]
    v_seq = [randn((Bl, T, w.Hkv, w.D)) for _ in range(N)]
    o_seq = [torch.empty_like(t) for t in q_seq]
    q_head = [torch.empty((Bl, w.S, plan.Hq_l, w.D), dtype=torch.bfloat16, device=dev) for _ in range(N)]
    k_head = [torch.empty((Bl, w.S, plan.Hkv_l, w.D), dtype=torch.bfloat16, device=dev) for _ in range(N)]
    v_head = [torch.empty((Bl, w.S, plan.Hkv_l, w.D), dtype=torch.bfloat16, device=dev) for _ in range(N)]
    o_head = [torch.empty_like(t) for t in q_head]

    train = w.train
    if train:
        do_seq = [randn((Bl, T, w.Hq, w.D)) for _ in range(N)]
        do_head = [torch.empty_like(t) for t in q_head]
        dq_head = [torch.empty_like(t) for t in q_head]
        dk_head = [torch.empty_like(t) for t in k_head]
        dv_head = [torch.empty_like(t) for t in k_head]
        dq_seq = [torch.empty_like(t) for t in q_seq]
        dk_seq = [torch.empty_like(t) for t in k_seq]
        dv_seq = [torch.empty_like(t) for t in k_seq]
        lse = [torch.empty((Bl, plan.Hq_l, w.S), dtype=torch.float32, device=dev) for _ in range(N)]
        bwd_ws = torch.empty(basp.basp_attn_bwd_workspace_bytes(plan), dtype=torch.uint8, device=dev)
    n_ev = 7 if train else 4

    def step(events=None):
        """a2 -> a3 -> a4 (what basp_layer_fwd launches) and, for a training workload, a7 -> a6 -> a7
        (what basp_layer_bwd launches), with optional events between the launches."""
        def mark(i):
            if events:
                events[i].record()
        mark(0)
        basp.basp_reshard_qkv_s2h(plan, q_seq, k_seq, v_seq, q_head, k_head, v_head)
        mark(1)
        basp.basp_attn_fwd(plan, q_head, k_head, v_head, o_head, lse if train else None)
        mark(2)
        basp.basp_reshard_h2s(plan, w.Hq, o_head, o_seq)
        mark(3)
        if train:
            basp.basp_reshard_s2h(plan, w.Hq, do_seq, do_head)
            mark(4)
            basp.basp_attn_bwd(plan, q_head, k_head, v_head, o_head, do_head, lse, dq_head, dk_head, dv_head, bwd_ws)
            mark(5)
            basp.basp_reshard_grads_h2s(plan, dq_head, dk_head, dv_head, dq_seq, dk_seq, dv_seq)
            mark(6)

    basp.basp_clear_status()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    basp.basp_get_status()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank) if rank == 0 else None
    launches0 = basp.basp_launch_count()
    pdist.barrier()
    torch.cuda.synchronize()
    for i in range(args.steps):
        step(ev[i])
    torch.cuda.synchronize()
    pdist.barrier()
    launches = basp.basp_launch_count() - launches0
    total_ms = ev[0][0].elapsed_time(ev[-1][n_ev - 1])
    per_step = [e[0].elapsed_time(e[n_ev - 1]) for e in ev]          # each step on its own (the headline is total / steps)
    ms_s2h = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    ms_attn = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    ms_h2s = statistics.mean(e[2].elapsed_time(e[3]) for e in ev)
    ms_bwd = [statistics.mean(e[i].elapsed_time(e[i + 1]) for e in ev) for i in (3, 4, 5)] if train else None
    basp.basp_get_status()

    proj = None
    if args.proj:      # the projections on either side of the core (not part of the step): X W_qkv^T and O W_o^T
        hidden = w.Hq * w.D
        xs = [randn((Bl * T, hidden)) for _ in range(N)]
        w_qkv = (torch.randn(((w.Hq + 2 * w.Hkv) * w.D, hidden), generator=gen, device=dev) / hidden ** 0.5).to(torch.bfloat16)
        w_o = (torch.randn((hidden, w.Hq * w.D), generator=gen, device=dev) / hidden ** 0.5).to(torch.bfloat16)
        ys = [torch.empty((Bl * T, hidden), dtype=torch.bfloat16, device=dev) for _ in range(N)]
        pe = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        for it in range(args.warmup + args.steps):
            if it == args.warmup:
                pe[0].record()
            basp.basp_qkv_proj(plan, hidden, xs, w_qkv, q_seq, k_seq, v_seq)
        pe[1].record()
        for it in range(args.steps):
            basp.basp_out_proj(plan, hidden, o_seq, w_o, ys)
        pe[2].record()
        ms_rope = None
        if w.D in (64, 128):      # the same projection with rotary position embedding in its epilogue
            cos, sin = (t.t().contiguous().to(dev) for t in synth.rope_tables(w.S, w.D))      # feature-major
            re = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            for it in range(args.warmup + args.steps):
                if it == args.warmup:
                    re[0].record()
                basp.basp_qkv_proj_rope(plan, hidden, xs, w_qkv, cos, sin, q_seq, k_seq, v_seq)
            re[1].record()
            torch.cuda.synchronize()
            ms_rope = re[0].elapsed_time(re[1]) / args.steps
        torch.cuda.synchronize()
        basp.basp_get_status()
        ms_qkv, ms_out = pe[0].elapsed_time(pe[1]) / args.steps, pe[1].elapsed_time(pe[2]) / args.steps
        f_qkv = 2.0 * N * Bl * T * hidden * (w.Hq + 2 * w.Hkv) * w.D
        f_out = 2.0 * N * Bl * T * hidden * w.Hq * w.D
        proj = {"hidden": hidden, "qkv_ms": ms_qkv, "qkv_tflops": f_qkv / ms_qkv / 1e9, "out_ms": ms_out,
                "out_tflops": f_out / ms_out / 1e9, "qkv_rope_ms": ms_rope,
                "qkv_rope_tflops": f_qkv / ms_rope / 1e9 if ms_rope else None, "peak_sustained": peaks["bf16_sustained"]}
        del xs, ys, w_qkv, w_o

    if args.quick:     # kernel timings only (what the ncu recipes in profiles/ run)
        clocks = sampler.stop() if sampler else None
        if rank == 0:
            print(json.dumps({"workload": w.name, "ms_per_step": total_ms / args.steps, "ms_s2h": ms_s2h,
                              "ms_attn": ms_attn, "ms_h2s": ms_h2s, "gpu_launches": launches,
                              "attn_tflops": w.attn_flops_fwd() / ms_attn / 1e9, "clocks": clocks,
                              "bwd_ms_s2h_attn_h2s": ms_bwd, "projections": proj,
                              "attn_bwd_tflops": (w.attn_flops_bwd() / ms_bwd[1] / 1e9) if train else None}), flush=True)
        pdist.finalize()
        return

    if train:
        return finish_train(args, w, basp, peaks, rank, world, sampler, launches, total_ms, ms_s2h, ms_attn, ms_h2s, ms_bwd, K)

    # fused layer (a5): one kernel straight from / to the sequence-sharded shards
    for _ in range(max(1, args.warmup // 2)):
        basp.basp_layer_fwd_fused(plan, q_seq, k_seq, v_seq, o_seq)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    f0.record()
    for _ in range(args.steps):
        basp.basp_layer_fwd_fused(plan, q_seq, k_seq, v_seq, o_seq)
    f1.record()
    torch.cuda.synchronize()
    ms_fused = f0.elapsed_time(f1) / args.steps
    basp.basp_get_status()

    # the same three launches replayed from a CUDA graph (the calls are capturable: asynchronous, no allocation, no
    # synchronisation): what the step costs without the host's launch path, which is what config 1 is bound by
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step()
    graph.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(args.steps):
        graph.replay()
    g1.record()
    torch.cuda.synchronize()
    ms_graph = g0.elapsed_time(g1) / args.steps
    basp.basp_get_status()
    del graph
    clocks = sampler.stop() if sampler else None

    # end to end through the C ABI with HOST buffers: H2D of Q, K, V and D2H of O inside the timed region
    e2e_steps = max(1, min(args.steps, 5))
    del q_head, k_head, v_head, o_head
    hq = [t.cpu().pin_memory() for t in q_seq]
    hk = [t.cpu().pin_memory() for t in k_seq]
    hv = [t.cpu().pin_memory() for t in v_seq]
    ho = [torch.empty_like(t).pin_memory() for t in hq]
    arena = torch.empty(basp.basp_host_arena_bytes(plan), dtype=torch.uint8, device=dev)
    basp.basp_layer_fwd_host(plan, hq, hk, hv, ho, arena)
    pdist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        basp.basp_layer_fwd_host(plan, hq, hk, hv, ho, arena)       # synchronises the stream itself
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    h2d = sum(t.numel() * 2 for t in hq + hk + hv)
    d2h = sum(t.numel() * 2 for t in ho)

    ms_per_step = pdist.max_over_ranks(total_ms / args.steps)
    e2e_ms = pdist.max_over_ranks(e2e_ms)
    ms_fused_max = pdist.max_over_ranks(ms_fused)
    tokens_all = w.tokens * world

    if rank == 0:
        flops = w.attn_flops_fwd()
        attn_tflops = flops / (ms_attn * 1e-3) / 1e12
        s2h_gbs = w.reshard_bytes_s2h() / (ms_s2h * 1e-3) / 1e9
        h2s_gbs = w.reshard_bytes_h2s() / (ms_h2s * 1e-3) / 1e9
        cpu = None
        if world == 1:
            v, cores, desc, _ = oracle_sample(w)
            cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        line = {
            "metric": METRIC, "value": tokens_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "N": w.N, "b": w.B, "group_size": K, "S": w.S, "Hq": w.Hq, "Hkv": w.Hkv,
                       "D": w.D, "causal": True, "path": "reshard_qkv_s2h -> attn_fwd -> reshard_h2s (3 launches/step)",
                       "l2": "inputs larger than L2 (Q+K+V 768 MiB per step for the default workload)",
                       "per_gpu_tokens": w.tokens},
            "clocks": clocks,
            "e2e": {"value": tokens_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "call": "basp_layer_fwd_host (fused kernel per arrived piece of query rows, copies and kernels pipelined, pinned host shards)"},
            "gpu_launches": launches,
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_best": min(per_step),
            "roofline": {"kernel": "attn_fwd", "bound": "tensor", "achieved": attn_tflops,
                         "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                         "frac": attn_tflops / peaks["bf16_sustained"], "traffic": NCU_TRAFFIC_BYTES.get(w.name),
                         "peak_source": f"bf16 sustained, of {peaks['source']}", "ms": ms_attn,
                         "frac_of_burst": attn_tflops / peaks["bf16_burst"], "frac_of_nominal_2250": attn_tflops / 2250.0,
                         "flops_per_launch": flops},
            "kernels": {
                "reshard_qkv_s2h": {"ms": ms_s2h, "bound": "hbm", "achieved": s2h_gbs, "unit": "GB/s",
                                    "frac": s2h_gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": s2h_gbs / 8000.0,
                                    "bytes": w.reshard_bytes_s2h()},
                "reshard_h2s": {"ms": ms_h2s, "bound": "hbm", "achieved": h2s_gbs, "unit": "GB/s",
                                "frac": h2s_gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": h2s_gbs / 8000.0,
                                "bytes": w.reshard_bytes_h2s()},
            },
            "fused": {"ms_per_step": ms_fused_max, "value": tokens_all / (ms_fused_max * 1e-3), "unit": UNIT,
                      "tflops": flops / (ms_fused * 1e-3) / 1e12, "launches_per_step": 1},
            "graph_replay": {"ms_per_step": ms_graph, "value": w.tokens / (ms_graph * 1e-3), "unit": UNIT,
                             "what": "the step's three launches captured once into a CUDA graph and replayed"},
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    pdist.finalize()


def finish_train(args, w, basp, peaks, rank, world, sampler, launches, total_ms, ms_s2h, ms_attn, ms_h2s, ms_bwd, K):
    """JSON line of a forward + backward workload (BASELINE config 5)."""
    clocks = sampler.stop() if sampler else None
    ms_per_step = pdist.max_over_ranks(total_ms / args.steps)
    tokens_all = w.tokens * world
    if rank == 0:
        fwd_tf = w.attn_flops_fwd() / (ms_attn * 1e-3) / 1e12
        bwd_tf = w.attn_flops_bwd() / (ms_bwd[1] * 1e-3) / 1e12
        gbs = lambda b, ms: b / (ms * 1e-3) / 1e9
        cpu = None
        if world == 1:
            v, cores, desc, _ = oracle_sample(w, budget_rows=2048)
            cpu = {"value": v / 3.5, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": desc + "; forward sample scaled by 3.5 for forward + backward (4*D + 10*D flop per pair)"}
        line = {
            "metric": METRIC, "value": tokens_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "N": w.N, "b": w.B, "group_size": K, "S": w.S, "Hq": w.Hq, "Hkv": w.Hkv,
                       "D": w.D, "causal": True,
                       "path": "forward (s2h, attn_fwd, h2s) + backward (s2h dO, attn_bwd, h2s dQ/dK/dV)",
                       "l2": "inputs larger than L2", "per_gpu_tokens": w.tokens},
            "clocks": clocks, "e2e": None, "gpu_launches": launches,
            "roofline": {"kernel": "attn_bwd (memset + Delta + main + dQ conversion)", "bound": "tensor",
                         "achieved": bwd_tf, "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                         "frac": bwd_tf / peaks["bf16_sustained"], "traffic": None,
                         "peak_source": f"bf16 sustained, of {peaks['source']}", "ms": ms_bwd[1],
                         "frac_of_burst": bwd_tf / peaks["bf16_burst"], "frac_of_nominal_2250": bwd_tf / 2250.0,
                         "flops_per_launch": w.attn_flops_bwd()},
            "kernels": {
                "attn_fwd": {"ms": ms_attn, "bound": "tensor", "achieved": fwd_tf, "unit": "TFLOP/s",
                             "frac": fwd_tf / peaks["bf16_sustained"]},
                "reshard_qkv_s2h": {"ms": ms_s2h, "achieved": gbs(w.reshard_bytes_s2h(), ms_s2h), "unit": "GB/s",
                                    "frac": gbs(w.reshard_bytes_s2h(), ms_s2h) / peaks["hbm_gbs"]},
                "reshard_h2s_o": {"ms": ms_h2s, "achieved": gbs(w.reshard_bytes_h2s(), ms_h2s), "unit": "GB/s",
                                  "frac": gbs(w.reshard_bytes_h2s(), ms_h2s) / peaks["hbm_gbs"]},
                "reshard_s2h_do": {"ms": ms_bwd[0], "achieved": gbs(w.reshard_bytes_h2s(), ms_bwd[0]), "unit": "GB/s",
                                   "frac": gbs(w.reshard_bytes_h2s(), ms_bwd[0]) / peaks["hbm_gbs"]},
                "reshard_grads_h2s": {"ms": ms_bwd[2], "achieved": gbs(w.reshard_bytes_s2h(), ms_bwd[2]), "unit": "GB/s",
                                      "frac": gbs(w.reshard_bytes_s2h(), ms_bwd[2]) / peaks["hbm_gbs"]},
            },
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    pdist.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="basp", choices=["basp", "reference"])
    ap.add_argument("--proj", action="store_true", help="also time the QKV and output projection GEMMs (with --quick)")
    ap.add_argument("--quick", action="store_true", help="time the three kernels only (for profiler runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_gpu(args, w)


if __name__ == "__main__":
    main()
