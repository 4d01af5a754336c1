"""A group with more ranks than KV heads on the GPU: the replicating exchange is bit-exact against the oracle, the
three-launch layer and the fused kernel match the oracle's layer (which equals the unpartitioned definition), the
backward pass adds the copies' gradients up."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, oracle_inputs, to_bits, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [
    synth.Workload("llama_k16_like", N=8, B=1, S=2048, Hq=32, Hkv=4, D=128),      # K = 8, each KV head on 2 ranks
    synth.Workload("mqa", N=4, B=1, S=1024, Hq=8, Hkv=1, D=128),                  # one KV head for the whole group
    synth.Workload("two_groups_d64", N=8, B=2, S=1024, Hq=8, Hkv=2, D=64),        # K = 4, 2 copies, D = 64
    synth.Workload("ragged", N=4, B=1, S=1000, Hq=4, Hkv=2, D=128),               # T = 250: head-sharded path only
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_replicating_exchange_is_bit_exact(basp, w):
    _, Xk, _, op = oracle_inputs(w)
    pl = make_plan(basp, w)
    assert pl.Hkv_l == 1 and pl.K > w.Hkv
    seq = oracle.partition(Xk, op)
    dk = to_dev(seq)
    hk = [torch.zeros((pl.Bl, pl.S, 1, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    basp.basp_reshard_s2h(pl, w.Hkv, dk, hk)
    assert np.array_equal(to_bits(hk), oracle.s2h_replicated(seq, op))
    # the way back adds the copies up (it carries gradients): with identical copies that is K/Hkv times the tensor
    back = [torch.zeros_like(t) for t in dk]
    basp.basp_reshard_h2s(pl, w.Hkv, hk, back)
    want = oracle.bf16_bits_to_f64(seq) * (pl.K // w.Hkv)
    got = np.stack([t.float().cpu().numpy().astype(np.float64) for t in back])
    assert np.abs(got - want).max() <= np.abs(want).max() * 2.0 ** -8


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_layer_matches_oracle(basp, w, fused):
    if fused and (w.S // w.K) % 128 != 0:
        pytest.skip("the fused kernel needs T to be a multiple of 128")
    Xq, Xk, Xv, op = oracle_inputs(w)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    pl = make_plan(basp, w)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    do = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    basp.basp_clear_status()
    if fused:
        basp.basp_layer_fwd_fused(pl, dq, dk, dv, do, lse)
    else:
        ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
        basp.basp_layer_fwd(pl, dq, dk, dv, do, ws, lse_shards=lse)
    basp.basp_get_status()
    assert_attn_close(to_f64(do), ref["o_seq"], f"{w.name} fused={fused}")
    got_lse = np.stack([t.cpu().numpy().astype(np.float64) for t in lse])
    assert np.abs(got_lse - ref["lse_head"]).max() < 2e-3


@pytest.mark.parametrize("w", [
    synth.Workload("bwd_rep2", N=4, B=1, S=512, Hq=8, Hkv=2, D=128),
    synth.Workload("bwd_mqa_two_groups", N=8, B=2, S=512, Hq=8, Hkv=1, D=128),
], ids=lambda w: w.name)
def test_layer_backward_with_replication(basp, w):
    """Forward through basp_layer_fwd, backward through basp_layer_bwd: every rank's attention backward sees one KV head,
    the gradient exchange adds the copies' dK and dV.  Against the oracle's layer backward (= the global gradients)."""
    q, k, v, do_ = synth.make_qkv(w, seed=11, with_dO=True)
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
    gq, gk, gv = ([torch.zeros_like(t) for t in x] for x in (dq, dk, dv))
    ws2 = torch.empty(basp.basp_layer_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_layer_bwd(pl, qh, kh, vh, oh, lse, ddo, gq, gk, gv, ws2)
    basp.basp_get_status()
    for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
        r = ref[name + "_seq"]
        err = np.abs(to_f64(got) - r)
        assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (name, float(err.max()))
        assert err.mean() <= 2e-3 * max(1.0, float(np.abs(r).mean())), name
