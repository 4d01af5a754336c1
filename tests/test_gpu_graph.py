"""The layer's calls are asynchronous on the caller's stream, allocate nothing and never synchronise, so a training
step's forward and backward can be captured into a CUDA graph and replayed: the replay must reproduce the eager results
bit for bit (the forward) and within the summation-order freedom of the dQ reduction (the backward), also after the inputs
have been overwritten in place with new values."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def test_forward_and_backward_replay_from_a_cuda_graph(basp):
    w = synth.Workload("graph", N=4, B=2, S=1024, Hq=8, Hkv=4, D=128)
    pl = make_plan(basp, w)
    op = oracle.plan(w.N, w.B, w.S, w.G)

    def shards(seed):
        ts = synth.make_qkv(w, seed=seed, with_dO=True)
        return [synth.bits(t) for t in ts], [[synth.from_bits(a).cuda() for a in oracle.partition(synth.bits(t), op)] for t in ts]

    (Xq, Xk, Xv, Xdo), (dq, dk, dv, ddo) = shards(1)
    o = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    gq, gk, gv = ([torch.zeros_like(t) for t in x] for x in (dq, dk, dv))
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(basp.basp_layer_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    qh, kh, vh, oh = basp.basp_layer_workspace_shards(pl, ws)

    def step(stream):
        basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse, stream=stream)
        basp.basp_layer_bwd(pl, qh, kh, vh, oh, lse, ddo, gq, gk, gv, ws2, stream=stream)

    basp.basp_clear_status()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step(side)                                   # eager once: modules loaded, attributes set
    side.synchronize()
    basp.basp_get_status()
    eager_o = [t.clone() for t in o]
    eager_g = [t.clone() for t in gq + gk + gv]

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(side)
    for t in o + gq + gk + gv:
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    basp.basp_get_status()
    assert all(torch.equal(a, b) for a, b in zip(o, eager_o))
    for a, b in zip(gq + gk + gv, eager_g):
        assert (a.float() - b.float()).abs().max().item() <= 2e-2

    # new inputs written into the same buffers, same graph
    (Xq, Xk, Xv, Xdo), fresh = shards(2)
    for dst, src in zip((dq, dk, dv, ddo), fresh):
        for a, b in zip(dst, src):
            a.copy_(b)
    graph.replay()
    torch.cuda.synchronize()
    basp.basp_get_status()
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    refb = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op)
    assert_attn_close(np.stack([t.float().cpu().numpy().astype(np.float64) for t in o]), ref["o_seq"], "graph replay, forward")
    for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
        r = refb[name + "_seq"]
        err = np.abs(np.stack([t.float().cpu().numpy().astype(np.float64) for t in got]) - r)
        assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (name, float(err.max()))
