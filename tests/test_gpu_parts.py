"""Unequal groups (micro-batch does not divide the rank count: groups of ceil and floor(N/B) ranks) on the GPU: every
part runs the ordinary calls on its own ranks; together they must equal the oracle's layer over the same groups,
which equals attention on the unpartitioned tensors."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [  # N, B, S, Hq, Hkv, D
    (8, 3, 1536, 12, 6, 64),       # groups of 3, 3, 2 ranks: T = 512 / 768
    (5, 2, 768, 6, 6, 128),        # groups of 3 and 2: T = 256 / 384
    (7, 3, 1000, 6, 6, 64),        # groups of 3, 2, 2; the group of 3 cuts 1000 tokens unevenly (334, 334, 332)
]


def dev(arrays):
    return [synth.from_bits(np.ascontiguousarray(a)).cuda() for a in arrays]


def f64(tensors):
    return np.concatenate([t.float().cpu().numpy().astype(np.float64).ravel() for t in tensors])


@pytest.mark.parametrize("N,B,S,Hq,Hkv,D", CASES)
def test_layer_forward_and_backward_over_unequal_groups(basp, N, B, S, Hq, Hkv, D):
    w = synth.Workload("parts", N=B, B=B, S=S, Hq=Hq, Hkv=Hkv, D=D)      # tensor shapes only
    Xq, Xk, Xv, Xdo = (synth.bits(t) for t in synth.make_qkv(w, seed=4, with_dO=True))
    oparts = oracle.plan_parts(N, B, S)
    ref = oracle.layer_fwd_parts(Xq, Xk, Xv, oparts)
    refb = oracle.layer_bwd_parts(Xq, Xk, Xv, Xdo, oparts)
    parts = basp.basp_plan_create_parts(N, B, S, Hq, Hkv, D)
    assert len(parts) == len(oparts) == 2
    o_glob = np.empty((B, S, Hq, D))
    basp.basp_clear_status()
    for pt, opt, rf, rb in zip(parts, oparts, ref["parts"], refb["parts"]):
        pl, op = pt.plan, opt.plan
        sl = slice(pt.seq_begin, pt.seq_begin + pt.n_seqs)
        cut = (lambda X: oracle.partition_uneven(X[sl], op)) if op.uneven else (lambda X: list(oracle.partition(X[sl], op)))
        dq, dk, dv, ddo = (dev(cut(X)) for X in (Xq, Xk, Xv, Xdo))
        variants = ["three_launch"] + (["fused"] if pl.T % 128 == 0 else [])
        for variant in variants:
            o = [torch.full_like(t, float("nan")) for t in dq]
            lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(pl.N)]
            ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
            if variant == "fused":
                basp.basp_layer_fwd_fused(pl, dq, dk, dv, o, lse)
            else:
                basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse)
            basp.basp_get_status()
            want = np.concatenate([np.asarray(a).ravel() for a in rf["o_seq"]])
            assert_attn_close(f64(o), want, f"part at rank {pt.rank_begin} {variant}")
        # the part's share of the global output, put back by the oracle's own gather
        shards = [t.float().cpu().numpy().astype(np.float64) for t in o]
        o_glob[sl] = oracle.gather_uneven(shards, op) if op.uneven else oracle.gather(np.stack(shards), op)
        # backward from the sequence-sharded activations
        gq, gk, gv = ([torch.full_like(t, float("nan")) for t in x] for x in (dq, dk, dv))
        ws2 = torch.empty(basp.basp_layer_bwd_seq_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
        basp.basp_layer_bwd_seq(pl, dq, dk, dv, o, lse, ddo, gq, gk, gv, ws2)
        basp.basp_get_status()
        for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
            r = np.concatenate([np.asarray(a).ravel() for a in rb[name + "_seq"]])
            err = np.abs(f64(got) - r)
            assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (name, float(err.max()))
    full, _ = oracle.attn_fwd(Xq, Xk, Xv)
    assert_attn_close(o_glob, full, "unequal groups against unpartitioned attention")
