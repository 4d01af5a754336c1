"""Plans with more than 8 ranks (up to BASP_MAX_RANKS = 32) run on the kernels' larger parameter blocks (32 tensor maps
per operand): every entry of the path once, against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, oracle_inputs, to_bits, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [
    synth.Workload("n16_k8", N=16, B=2, S=1024, Hq=16, Hkv=8, D=128),            # two groups of 8
    synth.Workload("n32_k8_d64", N=32, B=4, S=1024, Hq=8, Hkv=8, D=64),          # four groups of 8, T = 128
    synth.Workload("n32_ulysses", N=32, B=1, S=4096, Hq=32, Hkv=32, D=64, G=1),  # one group of 32 ranks
    synth.Workload("n32_k1", N=32, B=32, S=256, Hq=2, Hkv=1, D=128),             # 32 groups of one rank
    synth.Workload("n24_rep", N=24, B=3, S=1024, Hq=8, Hkv=4, D=128),            # K = 8 > Hkv: replicated KV heads
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_forward_layer_and_exchanges(basp, w):
    Xq, Xk, Xv, op = oracle_inputs(w)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    pl = make_plan(basp, w)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    # the exchange alone, bit for bit
    hq = [torch.zeros((pl.Bl, pl.S, pl.Hq_l, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    basp.basp_reshard_s2h(pl, w.Hq, dq, hq)
    assert np.array_equal(to_bits(hq), oracle.s2h(oracle.partition(Xq, op), op))
    back = [torch.zeros_like(t) for t in dq]
    basp.basp_reshard_h2s(pl, w.Hq, hq, back)
    assert np.array_equal(to_bits(back), oracle.partition(Xq, op))
    for variant in ["three_launch"] + (["fused"] if pl.T % 128 == 0 else []):
        o = [torch.full_like(t, float("nan")) for t in dq]
        lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
        basp.basp_clear_status()
        if variant == "fused":
            basp.basp_layer_fwd_fused(pl, dq, dk, dv, o, lse)
        else:
            ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
            basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse)
        basp.basp_get_status()
        assert_attn_close(to_f64(o), ref["o_seq"], f"{w.name} {variant}")


@pytest.mark.parametrize("deterministic", [False, True])
@pytest.mark.parametrize("w", [CASES[0], CASES[1], CASES[4]], ids=lambda w: w.name)
def test_backward_layer(basp, w, deterministic):
    q, k, v, do_ = synth.make_qkv(w, seed=21, with_dO=True)
    Xq, Xk, Xv, Xdo = (synth.bits(t) for t in (q, k, v, do_))
    op = oracle.plan(w.N, w.B, w.S, w.G)
    ref = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op)
    pl = make_plan(basp, w)
    dq, dk, dv, ddo = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv, Xdo))
    o = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse)
    qh, kh, vh, oh = basp.basp_layer_workspace_shards(pl, ws)
    mk = lambda h: [torch.full((pl.Bl, pl.S, h, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    doh, gqh, gkh, gvh = mk(pl.Hq_l), mk(pl.Hq_l), mk(pl.Hkv_l), mk(pl.Hkv_l)
    basp.basp_reshard_s2h(pl, w.Hq, ddo, doh)
    bws = torch.empty(basp.basp_attn_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_attn_bwd(pl, qh, kh, vh, oh, doh, lse, gqh, gkh, gvh, bws, deterministic=deterministic)
    gq, gk, gv = ([torch.full_like(t, float("nan")) for t in x] for x in (dq, dk, dv))
    basp.basp_reshard_grads_h2s(pl, gqh, gkh, gvh, gq, gk, gv)
    basp.basp_get_status()
    for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
        r = ref[name + "_seq"]
        err = np.abs(to_f64(got) - r)
        assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (name, float(err.max()))


def test_projections_and_host_entry(basp):
    w = CASES[0]
    pl = make_plan(basp, w)
    hidden = 256
    g = torch.Generator().manual_seed(3)
    M = pl.Bl * pl.T
    x = [synth.randn_bf16(g, (M, hidden)) for _ in range(w.N)]
    w_qkv = (torch.randn(((w.Hq + 2 * w.Hkv) * w.D, hidden), generator=g) / hidden ** 0.5).to(torch.bfloat16)
    mk = lambda h: [torch.full((pl.Bl, pl.T, h, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    dq, dk, dv = mk(w.Hq), mk(w.Hkv), mk(w.Hkv)
    basp.basp_clear_status()
    basp.basp_qkv_proj(pl, hidden, [t.cuda() for t in x], w_qkv.cuda(), dq, dk, dv)
    basp.basp_get_status()
    for r in (0, 9, w.N - 1):
        Y = oracle.linear(synth.bits(x[r]), synth.bits(w_qkv))
        got = torch.cat([dq[r].reshape(M, -1), dk[r].reshape(M, -1), dv[r].reshape(M, -1)], dim=1).float().cpu().numpy()
        err = np.abs(got.astype(np.float64) - Y)
        assert (err <= 1e-2 + 2.0 ** -8 * np.abs(Y)).all(), (r, float(err.max()))
    # host-buffer entry with the plan's own inputs
    Xq, Xk, Xv, op = oracle_inputs(w, seed=4)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    host = [[synth.from_bits(a[r]).pin_memory() for r in range(w.N)] for a in (ref["q_seq"], ref["k_seq"], ref["v_seq"])]
    out = [torch.zeros_like(t).pin_memory() for t in host[0]]
    arena = torch.empty(basp.basp_host_arena_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_layer_fwd_host(pl, host[0], host[1], host[2], out, arena)
    basp.basp_get_status()
    assert_attn_close(to_f64(out), ref["o_seq"], "host entry, 16 ranks")
