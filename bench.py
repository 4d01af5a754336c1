#!/usr/bin/env python
"""Benchmark of the BASP attention-layer hot path on B200.

One step = one pass of the layer over one synthetic micro-batch held as N virtual ranks on one
GPU: all-to-all reshard of Q, K, V (sequence- to head-sharded), causal attention over every rank's
head slice, reverse reshard of O (and, for a training workload, the backward: exchange of dO, attention
backward, reverse exchanges of dQ, dK, dV).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

The headline is the largest forward-only shape (Qwen2.5-7B heads, 64K tokens, two groups of four).  With one GPU
the line also carries `configs`: every benchmark shape (tiny; Llama-3-8B at 32K; the 65536-token sweep over
b = 1, 2, 4, 8; Qwen2.5-7B at 64K; the 128K-token training step) timed in the same run, each with its kernel rates,
its fused form, its end-to-end number and the clocks sampled during that leg; and `span`: the layer of one group of
eight ranks through the entry points that serve a group spread over GPUs (on one GPU: every rank local).

With --gpus N > 1 (launched by torchrun, one process per GPU) every GPU runs its own micro-batch
of the same shape (weak scaling; BASP groups and micro-batches are independent, so the data path
has no collective); times are the maximum over ranks.  The `span` leg then spreads ONE micro-batch's group of eight
ranks over the N GPUs (peer loads and stores over NVLink, no collective library on the data path).
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
DEFAULT_WORKLOAD = "qwen25_7b_64k"          # N=8, b=2 (groups of 4), S=65536, 28/4 heads, D=128: the largest forward shape
ALL_SHAPES = ["tiny", "llama3_8b_32k", "sweep_b1", "sweep_b2", "sweep_b4", "sweep_b8", "qwen25_7b_64k",
              "llama3_8b_128k_train"]
SPAN_WORKLOAD = "sweep_b1"                  # one group of eight ranks: the shape whose exchange crosses GPUs


def ncu_traffic(workload: str, kernel: str):
    """DRAM bytes (read + write) of one launch of `kernel` on `workload` from the profiler capture that the tracked
    table names, or None where no capture exists."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        entry = json.load(open(path))[workload][kernel]
        return int(entry["dram_bytes_read"]) + int(entry["dram_bytes_write"])
    except (OSError, KeyError, ValueError):
        return None


def config_dict(w: synth.Workload) -> dict:
    """The workload description both arms print."""
    path = ("forward (s2h, attn_fwd, h2s) + backward (s2h dO, attn_bwd, h2s dQ/dK/dV)" if w.train
            else "reshard_qkv_s2h -> attn_fwd -> reshard_h2s (3 launches/step)")
    return {"workload": w.name, "N": w.N, "b": w.B, "group_size": w.K, "S": w.S, "Hq": w.Hq, "Hkv": w.Hkv, "D": w.D,
            "causal": True, "path": path, "l2": "inputs larger than L2 (no flush needed)" if w.name != "tiny" else
            "tiny shape: L2-resident, launch-bound (no roofline claimed)", "per_gpu_tokens": w.tokens}


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
            "config": config_dict(w), "note": "fp64 CPU oracle on a bounded sample per step, extrapolated",
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)




# ------------------------------------------------------------------------------------------
class Shape:
    """Device buffers of one workload on one GPU: sequence-sharded inputs drawn N(0,1) -> bf16 per shard from a seeded
    device generator (timing only; the parity tests use the CPU generator on global coordinates), head-sharded
    intermediates, and for a training workload the gradients and the backward workspace."""

    def __init__(self, basp, w: synth.Workload, dev, seed: int):
        self.w, self.basp = w, basp
        self.plan = plan = basp.basp_plan_create(w.N, w.B, w.S, w.Hq, w.Hkv, w.D, num_groups=w.G)
        N, T, Bl = w.N, plan.T, plan.Bl
        gen = torch.Generator(device=dev).manual_seed(seed)
        self.randn = lambda shape: torch.randn(shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
        empty = lambda shape: torch.empty(shape, dtype=torch.bfloat16, device=dev)
        self.q_seq = [self.randn((Bl, T, w.Hq, w.D)) for _ in range(N)]
        self.k_seq = [self.randn((Bl, T, w.Hkv, w.D)) for _ in range(N)]
        self.v_seq = [self.randn((Bl, T, w.Hkv, w.D)) for _ in range(N)]
        self.o_seq = [torch.empty_like(t) for t in self.q_seq]
        self.q_head = [empty((Bl, w.S, plan.Hq_l, w.D)) for _ in range(N)]
        self.k_head = [empty((Bl, w.S, plan.Hkv_l, w.D)) for _ in range(N)]
        self.v_head = [empty((Bl, w.S, plan.Hkv_l, w.D)) for _ in range(N)]
        self.o_head = [torch.empty_like(t) for t in self.q_head]
        self.lse = None
        if w.train:
            self.do_seq = [self.randn((Bl, T, w.Hq, w.D)) for _ in range(N)]
            self.do_head = [torch.empty_like(t) for t in self.q_head]
            self.dq_head = [torch.empty_like(t) for t in self.q_head]
            self.dk_head = [torch.empty_like(t) for t in self.k_head]
            self.dv_head = [torch.empty_like(t) for t in self.k_head]
            self.dq_seq = [torch.empty_like(t) for t in self.q_seq]
            self.dk_seq = [torch.empty_like(t) for t in self.k_seq]
            self.dv_seq = [torch.empty_like(t) for t in self.k_seq]
            self.lse = [torch.empty((Bl, plan.Hq_l, w.S), dtype=torch.float32, device=dev) for _ in range(N)]
            self.bwd_ws = torch.empty(basp.basp_attn_bwd_workspace_bytes(plan), dtype=torch.uint8, device=dev)
        self.n_events = 7 if w.train else 4
        self.seed = seed

    def checksum(self) -> dict:
        """Sum of the bf16 bit patterns of every input shard (what identifies the drawn inputs of a run)."""
        tot = lambda ts: int(sum(int(t.view(torch.int16).to(torch.int64).sum().item()) for t in ts))
        out = {"generator": f"torch device generator, seed {self.seed}, N(0,1) in fp32 rounded to bf16, per shard in the order Q, K, V",
               "q": tot(self.q_seq), "k": tot(self.k_seq), "v": tot(self.v_seq)}
        if self.w.train:
            out["do"] = tot(self.do_seq)
        return out

    def step(self, events=None):
        """a2 -> a3 -> a4 (what basp_layer_fwd launches) and, for a training workload, a7 -> a6 -> a7 (what
        basp_layer_bwd launches), with optional events between the launches."""
        b, p, w = self.basp, self.plan, self.w

        def mark(i):
            if events:
                events[i].record()
        mark(0)
        b.basp_reshard_qkv_s2h(p, self.q_seq, self.k_seq, self.v_seq, self.q_head, self.k_head, self.v_head)
        mark(1)
        b.basp_attn_fwd(p, self.q_head, self.k_head, self.v_head, self.o_head, self.lse)
        mark(2)
        b.basp_reshard_h2s(p, w.Hq, self.o_head, self.o_seq)
        mark(3)
        if w.train:
            b.basp_reshard_s2h(p, w.Hq, self.do_seq, self.do_head)
            mark(4)
            b.basp_attn_bwd(p, self.q_head, self.k_head, self.v_head, self.o_head, self.do_head, self.lse, self.dq_head,
                            self.dk_head, self.dv_head, self.bwd_ws)
            mark(5)
            b.basp_reshard_grads_h2s(p, self.dq_head, self.dk_head, self.dv_head, self.dq_seq, self.dk_seq, self.dv_seq)
            mark(6)


def time_steps(shape: Shape, steps: int, warmup: int, rank: int, local_rank: int):
    """W untimed steps, then exactly `steps` timed ones between barriers and device synchronisations, CUDA events on the
    launching stream around every launch, the clocks sampled meanwhile.  Returns a dict of per-launch means (ms)."""
    basp = shape.basp
    basp.basp_clear_status()
    for _ in range(warmup):
        shape.step()
    torch.cuda.synchronize()
    basp.basp_get_status()
    n_ev = shape.n_events
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(steps)]
    sampler = ClockSampler(local_rank) if rank == 0 else None
    launches0 = basp.basp_launch_count()
    pdist.barrier()
    torch.cuda.synchronize()
    for i in range(steps):
        shape.step(ev[i])
    torch.cuda.synchronize()
    pdist.barrier()
    launches = basp.basp_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    basp.basp_get_status()
    mean = lambda i: statistics.mean(e[i].elapsed_time(e[i + 1]) for e in ev)
    per_step = [e[0].elapsed_time(e[n_ev - 1]) for e in ev]
    out = {"total_ms": ev[0][0].elapsed_time(ev[-1][n_ev - 1]), "per_step": per_step, "launches": launches, "clocks": clocks,
           "ms_s2h": mean(0), "ms_attn": mean(1), "ms_h2s": mean(2)}
    if shape.w.train:
        out.update(ms_s2h_do=mean(3), ms_attn_bwd=mean(4), ms_h2s_grads=mean(5))
    return out


def time_fused(shape: Shape, steps: int, warmup: int) -> float:
    """basp_layer_fwd_fused (one kernel straight from / to the sequence-sharded shards): ms per call."""
    b = shape.basp
    for _ in range(max(1, warmup // 2)):
        b.basp_layer_fwd_fused(shape.plan, shape.q_seq, shape.k_seq, shape.v_seq, shape.o_seq)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    f0.record()
    for _ in range(steps):
        b.basp_layer_fwd_fused(shape.plan, shape.q_seq, shape.k_seq, shape.v_seq, shape.o_seq)
    f1.record()
    torch.cuda.synchronize()
    b.basp_get_status()
    return f0.elapsed_time(f1) / steps


def time_e2e_host(shape: Shape, steps: int, dev):
    """End to end through the C ABI with HOST buffers: basp_layer_fwd_host copies the pinned Q, K, V shards to the device,
    runs the fused kernel per arrived piece and copies O back, all inside the timed region (wall clock around the
    synchronous call).  Returns (ms per call, H2D bytes, D2H bytes)."""
    b, plan = shape.basp, shape.plan
    hq = [t.cpu().pin_memory() for t in shape.q_seq]
    hk = [t.cpu().pin_memory() for t in shape.k_seq]
    hv = [t.cpu().pin_memory() for t in shape.v_seq]
    ho = [torch.empty_like(t).pin_memory() for t in hq]
    arena = torch.empty(b.basp_host_arena_bytes(plan), dtype=torch.uint8, device=dev)
    b.basp_layer_fwd_host(plan, hq, hk, hv, ho, arena)
    pdist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        b.basp_layer_fwd_host(plan, hq, hk, hv, ho, arena)       # synchronises the stream itself
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3 / steps
    return ms, sum(t.numel() * 2 for t in hq + hk + hv), sum(t.numel() * 2 for t in ho)


def time_e2e_train(shape: Shape, steps: int, dev):
    """The training step through the layer entry points of the C ABI (basp_layer_fwd, then basp_layer_bwd on the
    head-sharded activations the forward left in its workspace), wall clock around the calls and a device
    synchronisation.  The activations and the loss gradient of a training step are produced and consumed on the
    device by the layers around this one, so the step has no host boundary: zero bytes cross the bus."""
    b, plan, w = shape.basp, shape.plan, shape.w
    ws = torch.empty(b.basp_workspace_bytes(plan), dtype=torch.uint8, device=dev)
    ws2 = torch.empty(b.basp_layer_bwd_workspace_bytes(plan), dtype=torch.uint8, device=dev)

    def one():
        b.basp_layer_fwd(plan, shape.q_seq, shape.k_seq, shape.v_seq, shape.o_seq, ws, shape.lse)
        qh, kh, vh, oh = (b.as_shards(a) for a in b.basp_layer_workspace_shards(plan, ws))
        b.basp_layer_bwd(plan, qh, kh, vh, oh, shape.lse, shape.do_seq, shape.dq_seq, shape.dk_seq, shape.dv_seq, ws2)
    one()
    torch.cuda.synchronize()
    pdist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3 / steps
    b.basp_get_status()
    return ms


def rates(w: synth.Workload, t: dict, peaks: dict) -> dict:
    """Kernel rates of one timed shape: attention TFLOP/s against the measured sustained and burst cuBLAS bf16 rates and
    the nominal 2250, both exchanges in GB/s against the measured copy bandwidth and the nominal 8 TB/s."""
    def tensor(flops, ms):
        tf = flops / (ms * 1e-3) / 1e12
        return {"ms": ms, "tflops": tf, "frac_of_sustained": tf / peaks["bf16_sustained"],
                "frac_of_burst": tf / peaks["bf16_burst"], "frac_of_nominal_2250": tf / 2250.0}

    def hbm(nbytes, ms):
        g = nbytes / (ms * 1e-3) / 1e9
        return {"ms": ms, "gbs": g, "frac_of_measured_copy": g / peaks["hbm_gbs"], "frac_of_nominal_8000": g / 8000.0,
                "bytes": nbytes}
    out = {"attn_fwd": tensor(w.attn_flops_fwd(), t["ms_attn"]),
           "reshard_qkv_s2h": hbm(w.reshard_bytes_s2h(), t["ms_s2h"]),
           "reshard_h2s": hbm(w.reshard_bytes_h2s(), t["ms_h2s"])}
    if w.train:
        out["attn_bwd"] = tensor(w.attn_flops_bwd(), t["ms_attn_bwd"])
        out["attn_bwd"]["launches"] = "memset + Delta + main kernel + dQ conversion"
        out["reshard_s2h_do"] = hbm(w.reshard_bytes_h2s(), t["ms_s2h_do"])
        out["reshard_grads_h2s"] = hbm(w.reshard_bytes_s2h(), t["ms_h2s_grads"])
    return out


def measure_shape(basp, w: synth.Workload, dev, rank: int, local_rank: int, steps: int, warmup: int, peaks: dict,
                  e2e_steps: int = 3) -> dict:
    """One entry of `configs`: the three-launch step (plus the backward for a training shape), the fused form, the
    end-to-end number, rates and clocks of one shape."""
    shape = Shape(basp, w, dev, seed=1000 + rank)
    t = time_steps(shape, steps, warmup, rank, local_rank)
    ms = t["total_ms"] / steps
    entry = {"config": config_dict(w), "steps": steps, "warmup": warmup, "ms_per_step": ms,
             "tokens_per_s": w.tokens / (ms * 1e-3), "kernels": rates(w, t, peaks), "clocks": t["clocks"],
             "gpu_launches": t["launches"]}
    if w.train:
        e_ms = time_e2e_train(shape, min(steps, e2e_steps), dev)
        entry["e2e"] = {"ms_per_step": e_ms, "value": w.tokens / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0,
                        "call": "basp_layer_fwd + basp_layer_bwd from device buffers (a training step has no host boundary)"}
    else:
        f_ms = time_fused(shape, steps, warmup)
        entry["fused"] = {"ms_per_step": f_ms, "tokens_per_s": w.tokens / (f_ms * 1e-3),
                          "tflops": w.attn_flops_fwd() / (f_ms * 1e-3) / 1e12,
                          "ms_minus_attention_launch": f_ms - t["ms_attn"]}
        del shape.q_head, shape.k_head, shape.v_head, shape.o_head
        e_ms, h2d, d2h = time_e2e_host(shape, min(steps, e2e_steps), dev)
        entry["e2e"] = {"ms_per_step": e_ms, "value": w.tokens / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "call": "basp_layer_fwd_host (pinned host shards)"}
    del shape
    torch.cuda.empty_cache()
    return entry


def measure_span(basp, dev, rank: int, world: int, steps: int, warmup: int) -> dict:
    """One micro-batch whose single group of eight ranks is spread over the GPUs of the run (on one GPU: all eight
    local): the fused form (Q/K/V tiles fetched from wherever the group's sequence shards live, O tiles stored into
    the owner's shard) and the three-step form (push exchange, attention, pull exchange), both through the `*_ranks`
    entry points over a symmetric shard table, host barriers between the steps.  Peer loads and stores only."""
    w = synth.WORKLOADS[SPAN_WORKLOAD]
    if w.N % world != 0:
        return {"skipped": f"{w.N} ranks do not divide over {world} GPUs"}
    plan = basp.basp_plan_create(w.N, w.B, w.S, w.Hq, w.Hkv, w.D)
    T, S = plan.T, w.S
    qb, kb = T * w.Hq * w.D * 2, T * w.Hkv * w.D * 2
    qhb, khb = S * plan.Hq_l * w.D * 2, S * plan.Hkv_l * w.D * 2
    sh = pdist.SymmetricShards(w.N, {"q": qb, "k": kb, "v": kb, "o": qb, "qh": qhb, "kh": khb, "vh": khb, "oh": qhb})
    gen = torch.Generator(device=dev).manual_seed(2000 + rank)
    for r in sh.local:
        for name in ("q", "k", "v"):
            t = sh.local_shard(name, r).view(torch.bfloat16)
            t.copy_(torch.randn(t.shape, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16))
    out = {"workload": w.name, "group_size": plan.K, "gpus": world, "ranks_per_gpu": len(sh.local),
           "remote_fraction_of_exchange_bytes": sh.remote_fraction(plan.K), "tokens": w.tokens}
    basp.basp_clear_status()
    for name, fn in (("fused", pdist.layer_fwd_fused_multi_gpu), ("three_step", pdist.layer_fwd_three_step_multi_gpu)):
        for _ in range(max(1, warmup // 2)):
            fn(plan, sh)
        torch.cuda.synchronize()
        pdist.barrier()
        t0 = time.perf_counter()
        for _ in range(steps):
            fn(plan, sh)
        torch.cuda.synchronize()
        ms = pdist.max_over_ranks((time.perf_counter() - t0) * 1e3 / steps)
        out[name] = {"ms_per_step": ms, "tokens_per_s": w.tokens / (ms * 1e-3)}
        if name == "fused":
            fused_o = [sh.local_shard("o", r).clone() for r in sh.local]
    basp.basp_get_status()
    same = all(torch.equal(a, sh.local_shard("o", r)) for a, r in zip(fused_o, sh.local))
    out["three_step_equals_fused_bitwise"] = bool(same)
    if world == 1:      # every rank local: the call must reproduce the single-GPU fused layer bit for bit
        view = lambda name, r, h: sh.local_shard(name, r).view(torch.bfloat16).view(1, T, h, w.D)
        q, k, v = ([view(n, r, h) for r in range(w.N)] for n, h in (("q", w.Hq), ("k", w.Hkv), ("v", w.Hkv)))
        o = [torch.empty_like(t) for t in q]
        basp.basp_layer_fwd_fused(plan, q, k, v, o)
        torch.cuda.synchronize()
        out["equals_single_gpu_fused_bitwise"] = bool(all(torch.equal(a.view(torch.uint8).reshape(-1), b)
                                                          for a, b in zip(o, fused_o)))
    del sh
    torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------------------------------
def run_gpu(args, w: synth.Workload):
    from paper_2609_03151_b200 import binding as basp

    rank, local_rank, world = pdist.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback of the product path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = measured_peaks()

    if args.quick:     # kernel timings of one shape only (what the profiler recipes in profiles/ run)
        shape = Shape(basp, w, dev, seed=1000 + rank)
        t = time_steps(shape, args.steps, args.warmup, rank, local_rank)
        proj = time_projections(basp, shape, args, dev) if args.proj else None
        ms_fused = time_fused(shape, args.steps, args.warmup) if (args.fused and not w.train) else None
        if rank == 0:
            k = rates(w, t, peaks)
            print(json.dumps({"workload": w.name, "ms_per_step": t["total_ms"] / args.steps, "ms_s2h": t["ms_s2h"],
                              "ms_attn": t["ms_attn"], "ms_h2s": t["ms_h2s"], "gpu_launches": t["launches"],
                              "attn_tflops": k["attn_fwd"]["tflops"], "clocks": t["clocks"],
                              "bwd_ms_s2h_attn_h2s": [t["ms_s2h_do"], t["ms_attn_bwd"], t["ms_h2s_grads"]] if w.train else None,
                              "projections": proj, "ms_fused": ms_fused,
                              "attn_bwd_tflops": k["attn_bwd"]["tflops"] if w.train else None}), flush=True)
        pdist.finalize()
        return

    # ---- the headline shape: exactly args.steps timed steps after args.warmup untimed ones
    shape = Shape(basp, w, dev, seed=1000 + rank)
    inputs = shape.checksum()
    t = time_steps(shape, args.steps, args.warmup, rank, local_rank)
    ms_per_step = pdist.max_over_ranks(t["total_ms"] / args.steps)
    k = rates(w, t, peaks)
    tokens_all = w.tokens * world
    fused = None
    if w.train:
        e2e_steps = max(1, min(args.steps, 3))
        e2e_ms = pdist.max_over_ranks(time_e2e_train(shape, e2e_steps, dev))
        e2e = {"value": tokens_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
               "ms_per_step": e2e_ms, "steps": e2e_steps,
               "call": "basp_layer_fwd + basp_layer_bwd from device buffers (a training step has no host boundary)"}
        top, top_name = k["attn_bwd"], "attn_bwd"
    else:
        f_ms = pdist.max_over_ranks(time_fused(shape, args.steps, args.warmup))
        fused = {"ms_per_step": f_ms, "value": tokens_all / (f_ms * 1e-3), "unit": UNIT,
                 "tflops": w.attn_flops_fwd() / (f_ms * 1e-3) / 1e12, "launches_per_step": 1,
                 "ms_minus_attention_launch": f_ms - t["ms_attn"]}
        del shape.q_head, shape.k_head, shape.v_head, shape.o_head
        e2e_steps = max(1, min(args.steps, 5))
        e_ms, h2d, d2h = time_e2e_host(shape, e2e_steps, dev)
        e2e_ms = pdist.max_over_ranks(e_ms)
        e2e = {"value": tokens_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": e2e_ms, "steps": e2e_steps,
               "call": "basp_layer_fwd_host (fused kernel per arrived piece of query rows, copies and kernels pipelined, pinned host shards)"}
        top, top_name = k["attn_fwd"], "attn_fwd"
    del shape
    torch.cuda.empty_cache()

    # ---- every benchmark shape under the same clock (one GPU only: the scaling runs stay short)
    configs = None
    if world == 1 and not args.no_configs:
        configs = {}
        for name in ALL_SHAPES:
            ww = synth.WORKLOADS[name]
            configs[name] = measure_shape(basp, ww, dev, rank, local_rank, 3 if ww.train else min(args.steps, 10),
                                          max(3, min(args.warmup, 5)), peaks)
    span = None
    if not args.no_configs:
        try:
            span = measure_span(basp, dev, rank, world, max(2, min(args.steps, 10)), args.warmup)
        except Exception as e:      # the group-spanning leg must not take the headline number down with it (it needs
            span = {"error": f"{type(e).__name__}: {e}"[:300]}       # symmetric memory across the run's GPUs)

    if rank == 0:
        cpu = None
        if world == 1:
            v, cores, desc, _ = oracle_sample(w, budget_rows=2048 if w.train else 8192)
            if w.train:
                v, desc = v / 3.5, desc + "; forward sample scaled by 3.5 for forward + backward (4*D + 10*D flop per pair)"
            cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
        line = {
            "metric": METRIC, "value": tokens_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(w), "inputs": inputs, "clocks": t["clocks"], "e2e": e2e, "gpu_launches": t["launches"],
            "ms_per_step_median": statistics.median(t["per_step"]), "ms_per_step_best": min(t["per_step"]),
            "roofline": {"kernel": top_name, "bound": "tensor", "achieved": top["tflops"], "peak": peaks["bf16_sustained"],
                         "unit": "TFLOP/s", "frac": top["frac_of_sustained"], "traffic": ncu_traffic(w.name, top_name),
                         "peak_source": f"cuBLAS bf16 sustained (the kernel is timed inside a loop), of {peaks['source']}",
                         "ms": top["ms"], "frac_of_burst": top["frac_of_burst"],
                         "frac_of_nominal_2250": top["frac_of_nominal_2250"],
                         "flops_per_launch": w.attn_flops_bwd() if w.train else w.attn_flops_fwd()},
            "kernels": k, "fused": fused, "configs": configs, "span": span, "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    pdist.finalize()


def time_projections(basp, shape: Shape, args, dev):
    """The projections on either side of the core (not part of the step): X W_qkv^T (plain and with the rotary
    embedding in its epilogue) and O W_o^T."""
    w, plan = shape.w, shape.plan
    N, T, Bl = w.N, plan.T, plan.Bl
    hidden = w.Hq * w.D
    xs = [shape.randn((Bl * T, hidden)) for _ in range(N)]
    w_qkv = (torch.randn(((w.Hq + 2 * w.Hkv) * w.D, hidden), device=dev) / hidden ** 0.5).to(torch.bfloat16)
    w_o = (torch.randn((hidden, w.Hq * w.D), device=dev) / hidden ** 0.5).to(torch.bfloat16)
    ys = [torch.empty((Bl * T, hidden), dtype=torch.bfloat16, device=dev) for _ in range(N)]
    pe = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    for it in range(args.warmup + args.steps):
        if it == args.warmup:
            pe[0].record()
        basp.basp_qkv_proj(plan, hidden, xs, w_qkv, shape.q_seq, shape.k_seq, shape.v_seq)
    pe[1].record()
    for it in range(args.steps):
        basp.basp_out_proj(plan, hidden, shape.o_seq, w_o, ys)
    pe[2].record()
    ms_rope = None
    if w.D in (64, 128):
        cos, sin = (t.t().contiguous().to(dev) for t in synth.rope_tables(w.S, w.D))      # feature-major
        re = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for it in range(args.warmup + args.steps):
            if it == args.warmup:
                re[0].record()
            basp.basp_qkv_proj_rope(plan, hidden, xs, w_qkv, cos, sin, shape.q_seq, shape.k_seq, shape.v_seq)
        re[1].record()
        torch.cuda.synchronize()
        ms_rope = re[0].elapsed_time(re[1]) / args.steps
    torch.cuda.synchronize()
    basp.basp_get_status()
    ms_qkv, ms_out = pe[0].elapsed_time(pe[1]) / args.steps, pe[1].elapsed_time(pe[2]) / args.steps
    f_qkv = 2.0 * N * Bl * T * hidden * (w.Hq + 2 * w.Hkv) * w.D
    f_out = 2.0 * N * Bl * T * hidden * w.Hq * w.D
    return {"hidden": hidden, "qkv_ms": ms_qkv, "qkv_tflops": f_qkv / ms_qkv / 1e9, "out_ms": ms_out,
            "out_tflops": f_out / ms_out / 1e9, "qkv_rope_ms": ms_rope,
            "qkv_rope_tflops": f_qkv / ms_rope / 1e9 if ms_rope else None}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="basp", choices=["basp", "reference"])
    ap.add_argument("--proj", action="store_true", help="also time the QKV and output projection GEMMs (with --quick)")
    ap.add_argument("--quick", action="store_true", help="time the kernels of one shape only (for profiler runs)")
    ap.add_argument("--fused", action="store_true", help="with --quick: also time basp_layer_fwd_fused after the three launches")
    ap.add_argument("--no-configs", action="store_true", help="the headline shape only (no `configs`, no `span`)")
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
