"""Seeded random plans and shapes through the whole forward path (three-launch layer, fused kernel where its
precondition holds) against the oracle's layer: group counts between Ulysses and BASP, several sequences per group,
GQA ratios including replicated KV heads, head dimensions that are padded inside the kernel, sequence lengths with
ragged last tiles, with and without the causal mask.  The hand-offs between the kernel's roles depend on the shape
(number of key blocks per item, one or two query tiles per item, items per CTA), which is what this walks through."""
import random
import zlib

import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def _random_workload(rng: random.Random) -> tuple[synth.Workload, bool]:
    while True:
        N = rng.choice([1, 2, 4, 8])
        G = rng.choice([g for g in (1, 2, 4, 8) if N % g == 0])
        Bl = rng.choice([1, 1, 2])
        B = G * Bl
        K = N // G
        D = rng.choice([16, 32, 48, 64, 64, 80, 96, 128, 128])
        hq_l = rng.choice([1, 2, 3, 4])
        Hq = hq_l * K
        ratios = [r for r in (1, 2, 3, 4, 8) if Hq % r == 0]
        Hkv = Hq // rng.choice(ratios)
        if not (Hkv % K == 0 or K % Hkv == 0):
            continue
        if ((Hq // K) * D * 2) % 16 or (max(Hkv // K, 1) * D * 2) % 16:
            continue
        T = rng.choice([1, 7, 64, 128, 128, 200, 256, 384, 512])
        S = T * K
        if B * S * Hq * D > 3_000_000 or S > 2048:       # keep the oracle to a second or two
            continue
        causal = rng.random() < 0.8
        return synth.Workload(f"fuzz_N{N}_G{G}_Bl{Bl}_S{S}_H{Hq}-{Hkv}_D{D}", N=N, B=B, S=S, Hq=Hq, Hkv=Hkv, D=D, G=G), causal


CASES = []
_rng = random.Random(20260925)
for _ in range(60):
    CASES.append(_random_workload(_rng))


@pytest.mark.parametrize("w,causal", CASES, ids=lambda x: x.name if isinstance(x, synth.Workload) else f"causal{int(x)}")
def test_random_plan_matches_oracle(basp, w, causal):
    q, k, v = synth.make_qkv(w, seed=zlib.crc32(w.name.encode()) % 1000)
    Xq, Xk, Xv = synth.bits(q), synth.bits(k), synth.bits(v)
    op = oracle.plan(w.N, w.B, w.S, w.G)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op, causal=causal)
    pl = make_plan(basp, w, causal=causal)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    variants = ["three_launch"] + (["fused"] if pl.T % 128 == 0 else [])
    for variant in variants:
        do = [torch.zeros_like(t) for t in dq]
        lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
        basp.basp_clear_status()
        if variant == "fused":
            basp.basp_layer_fwd_fused(pl, dq, dk, dv, do, lse)
        else:
            ws = torch.empty(max(basp.basp_workspace_bytes(pl), 16), dtype=torch.uint8, device="cuda")
            basp.basp_layer_fwd(pl, dq, dk, dv, do, ws, lse_shards=lse)
        basp.basp_get_status()
        assert_attn_close(to_f64(do), ref["o_seq"], f"{w.name} {variant} causal={causal}")
        got_lse = np.stack([t.cpu().numpy().astype(np.float64) for t in lse])
        assert np.abs(got_lse - ref["lse_head"]).max() < 2e-3, (w.name, variant)
