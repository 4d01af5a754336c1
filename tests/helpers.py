"""Shared test plumbing: move oracle-built shards to the GPU and back, error measures."""
import numpy as np
import torch

import oracle
from paper_2609_03151_b200 import synth

MAX_ABS_TOL = 2e-2     # attention vs the fp64 oracle, bf16 inputs / fp32 accumulation
MEAN_ABS_TOL = 2e-3


def to_dev(arena_bits: np.ndarray, dev="cuda"):
    """[N, ...] uint16 arena -> list of N bf16 device tensors (separate allocations)."""
    return [synth.from_bits(arena_bits[r]).to(dev) for r in range(arena_bits.shape[0])]


def to_bits(tensors) -> np.ndarray:
    return np.stack([synth.bits(t.cpu()) for t in tensors])


def to_f64(tensors) -> np.ndarray:
    return np.stack([t.float().cpu().numpy().astype(np.float64) for t in tensors])


def oracle_inputs(w, seed=0):
    """Global bf16 bit tensors and the oracle plan of a workload."""
    q, k, v = synth.make_qkv(w, seed)
    return synth.bits(q), synth.bits(k), synth.bits(v), oracle.plan(w.N, w.B, w.S, w.G)


def make_plan(basp, w, causal=True):
    return basp.basp_plan_create(w.N, w.B, w.S, w.Hq, w.Hkv, w.D, num_groups=w.G, causal=causal)


def attn_errors(got_f64: np.ndarray, ref_f64: np.ndarray):
    e = np.abs(got_f64 - ref_f64)
    return float(e.max()), float(e.mean())


def assert_attn_close(got_f64, ref_f64, what=""):
    mx, mean = attn_errors(got_f64, ref_f64)
    assert mx <= MAX_ABS_TOL and mean <= MEAN_ABS_TOL, f"{what}: max-abs {mx:.3e} mean-abs {mean:.3e}"
    return mx, mean
