"""Parity of the attention kernel (head-sharded entry) with the fp64 oracle, through the C ABI.
Tolerance (bf16 inputs, fp32 accumulation, bf16 P and bf16 output): max-abs 2e-2, mean-abs 2e-3."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, oracle_inputs, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def run_attn(basp, w, causal=True, scale=0.0, seed=0, with_lse=True):
    Xq, Xk, Xv, op = oracle_inputs(w, seed)
    pl = make_plan(basp, w, causal)
    qh, kh, vh = (oracle.s2h(oracle.partition(X, op), op) for X in (Xq, Xk, Xv))
    dq, dk, dv = to_dev(qh), to_dev(kh), to_dev(vh)
    do = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((op.Bl, w.Hq // op.K, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)] if with_lse else None
    basp.basp_clear_status()
    basp.basp_attn_fwd(pl, dq, dk, dv, do, lse, softmax_scale=scale)
    basp.basp_get_status()
    ref_o, ref_l = [], []
    for r in range(w.N):
        o, l = oracle.attn_fwd(qh[r], kh[r], vh[r], scale=(scale or None), causal=causal)
        ref_o.append(o)
        ref_l.append(l)
    return to_f64(do), np.stack(ref_o), (to_f64(lse) if with_lse else None), np.stack(ref_l)


@pytest.mark.parametrize("name,w", [
    ("tiny", synth.WORKLOADS["tiny"]),
    ("llama_T512", synth.shrink(synth.WORKLOADS["llama3_8b_32k"], 512)),
    ("qwen_T256", synth.shrink(synth.WORKLOADS["qwen25_7b_64k"], 256)),
    ("one_tile", synth.Workload("one_tile", N=1, B=1, S=128, Hq=1, Hkv=1, D=128)),
    ("ragged_tiles", synth.Workload("ragged", N=2, B=2, S=640, Hq=2, Hkv=1, D=64)),
    ("ulysses", synth.Workload("ulysses", N=4, B=2, S=512, Hq=8, Hkv=4, D=128, G=1)),
    ("head_dim_96", synth.Workload("d96", N=4, B=2, S=640, Hq=8, Hkv=4, D=96)),       # hidden 3072 / 32 heads
    ("head_dim_96_ragged", synth.Workload("d96r", N=2, B=2, S=333, Hq=4, Hkv=2, D=96)),
    ("head_dim_80", synth.shrink(synth.WORKLOADS["t2_qwen25_3b"], 256)),                # hidden 2560 / 32 heads
    ("head_dim_48", synth.Workload("d48", N=2, B=2, S=384, Hq=4, Hkv=4, D=48)),
    ("head_dim_112", synth.Workload("d112", N=2, B=1, S=512, Hq=4, Hkv=2, D=112)),
])
def test_attn_fwd_matches_oracle(basp, name, w):
    got, ref, lse, ref_lse = run_attn(basp, w)
    assert_attn_close(got, ref, name)
    assert np.abs(lse - ref_lse).max() < 2e-3, np.abs(lse - ref_lse).max()


@pytest.mark.parametrize("S,causal", [(1, True), (77, True), (200, True), (333, False), (129, False), (1000, True)])
def test_ragged_sequence_lengths(basp, S, causal):
    """S not a multiple of the 128-row tile: the last tile is masked, rows past the end are not stored
    (two sequences per rank, so what follows a ragged end is the next sequence, not padding)."""
    w = synth.Workload("ragged_S", N=2, B=4, S=S, Hq=4, Hkv=2, D=128, G=2)
    got, ref, lse, ref_lse = run_attn(basp, w, causal=causal, seed=S)
    assert_attn_close(got, ref, f"S={S}")
    assert np.abs(lse - ref_lse).max() < 2e-3


def test_noncausal_and_explicit_scale(basp):
    w = synth.Workload("nc", N=2, B=2, S=384, Hq=4, Hkv=2, D=64)
    got, ref, lse, ref_lse = run_attn(basp, w, causal=False, scale=0.2, seed=5)
    assert_attn_close(got, ref, "noncausal")
    assert np.abs(lse - ref_lse).max() < 2e-3


def test_without_lse(basp):
    w = synth.Workload("nolse", N=2, B=2, S=256, Hq=2, Hkv=2, D=128)
    got, ref, _, _ = run_attn(basp, w, with_lse=False, seed=7)
    assert_attn_close(got, ref, "nolse")


def test_closed_forms_on_gpu(basp):
    """Row 0 returns V[0] exactly; Q = 0 returns the running mean of V."""
    w = synth.Workload("cf", N=1, B=1, S=512, Hq=2, Hkv=1, D=128)
    pl = make_plan(basp, w)
    g = torch.Generator().manual_seed(3)
    v = synth.randn_bf16(g, (1, w.S, 1, w.D)).cuda()
    k = synth.randn_bf16(g, (1, w.S, 1, w.D)).cuda()
    q = synth.randn_bf16(g, (1, w.S, 2, w.D)).cuda()
    o = torch.zeros_like(q)
    basp.basp_attn_fwd(pl, [q], [k], [v], [o])
    basp.basp_get_status()
    assert torch.equal(o[0, 0, 0], v[0, 0, 0]) and torch.equal(o[0, 0, 1], v[0, 0, 0])
    basp.basp_attn_fwd(pl, [torch.zeros_like(q)], [k], [v], [o])
    basp.basp_get_status()
    want = torch.cumsum(v.double(), 1) / torch.arange(1, w.S + 1, device="cuda").view(1, -1, 1, 1)
    assert (o.double() - want).abs().max() < 2e-2
