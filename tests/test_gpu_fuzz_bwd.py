"""Seeded random plans and shapes through the whole training path (forward layer, backward layer from the sequence-
sharded activations) against the oracle's layer backward: group counts between Ulysses and BASP, several sequences
per group, GQA ratios including replicated KV heads, padded head dimensions, ragged sequence lengths, lengths the
group size does not divide, with and without the causal mask."""
import random
import zlib

import numpy as np
import pytest
import torch

import oracle
from helpers import make_plan
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def _random_workload(rng: random.Random):
    while True:
        N = rng.choice([1, 2, 4, 8])
        G = rng.choice([g for g in (1, 2, 4, 8) if N % g == 0])
        Bl = rng.choice([1, 1, 2])
        B, K = G * Bl, N // G
        D = rng.choice([16, 32, 48, 64, 80, 96, 128, 128])
        Hq = rng.choice([1, 2, 4]) * K
        Hkv = Hq // rng.choice([r for r in (1, 2, 4) if Hq % r == 0])
        if not (Hkv % K == 0 or K % Hkv == 0):
            continue
        if ((Hq // K) * D * 2) % 16 or (max(Hkv // K, 1) * D * 2) % 16:
            continue
        S = rng.choice([1, 7, 64, 128, 200, 256, 384, 500]) * K - rng.choice([0, 0, 0, 1, K - 1])
        if S <= 0 or S - (K - 1) * -(-S // K) <= 0:
            continue
        if B * S * Hq * D > 1_500_000 or S > 1536:       # keep the oracle's backward to a second or two
            continue
        causal = rng.random() < 0.75
        return synth.Workload(f"bfuzz_N{N}_G{G}_Bl{Bl}_S{S}_H{Hq}-{Hkv}_D{D}", N=N, B=B, S=S, Hq=Hq, Hkv=Hkv, D=D, G=G), causal


CASES = []
_rng = random.Random(20261125)
for _ in range(30):
    CASES.append(_random_workload(_rng))


def _dev(arrays):
    return [synth.from_bits(np.ascontiguousarray(a)).cuda() for a in arrays]


def _cat(arrays):
    return np.concatenate([np.asarray(a, dtype=np.float64).ravel() for a in arrays])


@pytest.mark.parametrize("w,causal", CASES, ids=lambda x: x.name if isinstance(x, synth.Workload) else f"causal{int(x)}")
def test_random_plan_backward_matches_oracle(basp, w, causal):
    tensors = synth.make_qkv(w, seed=zlib.crc32(w.name.encode()) % 1000, with_dO=True)
    Xq, Xk, Xv, Xdo = (synth.bits(t) for t in tensors)
    op = oracle.plan(w.N, w.B, w.S, w.G) if w.S % w.K == 0 else oracle.plan_uneven(w.N, w.B, w.S, w.G)
    ref = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op, causal=causal)
    cut = (lambda X: oracle.partition_uneven(X, op)) if op.uneven else (lambda X: list(oracle.partition(X, op)))
    pl = make_plan(basp, w, causal=causal)
    dq, dk, dv, ddo = (_dev(cut(X)) for X in (Xq, Xk, Xv, Xdo))
    o = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    ws = torch.empty(max(basp.basp_workspace_bytes(pl), 16), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse)
    gq, gk, gv = ([torch.full_like(t, float("nan")) for t in x] for x in (dq, dk, dv))
    ws2 = torch.empty(max(basp.basp_layer_bwd_seq_workspace_bytes(pl), 16), dtype=torch.uint8, device="cuda")
    basp.basp_layer_bwd_seq(pl, dq, dk, dv, o, lse, ddo, gq, gk, gv, ws2)
    basp.basp_get_status()
    for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
        r = _cat(ref[name + "_seq"])
        g = _cat([t.float().cpu().numpy() for t in got])
        err = np.abs(g - r)
        assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (w.name, name, float(err.max()))
        assert err.mean() <= 2e-3 * max(1.0, float(np.abs(r).mean())), (w.name, name)
