"""A group with more ranks than KV heads on the GPU: the replicating exchange is bit-exact against the oracle, the
three-launch layer and the fused kernel match the oracle's layer (which equals the unpartitioned definition), the
backward pass declines."""
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
    with pytest.raises(basp.BaspError) as e:          # the way back would have to add the copies up
        basp.basp_reshard_h2s(pl, w.Hkv, hk, dk)
    assert e.value.code == basp.BASP_ERR_UNSUPPORTED


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


def test_backward_declines(basp):
    w = synth.Workload("bwd", N=4, B=1, S=512, Hq=8, Hkv=2, D=128)
    pl = make_plan(basp, w)
    mk = lambda h: [torch.zeros((pl.Bl, pl.S, h, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    q, k, v, o, do, dq, dk, dv = mk(2), mk(1), mk(1), mk(2), mk(2), mk(2), mk(1), mk(1)
    lse = [torch.zeros((pl.Bl, 2, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    ws = torch.empty(max(basp.basp_attn_bwd_workspace_bytes(pl), 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(basp.BaspError) as e:
        basp.basp_attn_bwd(pl, q, k, v, o, do, lse, dq, dk, dv, ws)
    assert e.value.code == basp.BASP_ERR_UNSUPPORTED
