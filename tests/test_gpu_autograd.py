"""The differentiable wrapper: forward and gradients through torch.autograd against the oracle's layer."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("w", [
    synth.shrink(synth.WORKLOADS["llama3_8b_32k"], 128),
    synth.Workload("tiny_like_d64", N=4, B=2, S=512, Hq=8, Hkv=8, D=64),
], ids=lambda w: w.name)
@pytest.mark.parametrize("fused", [False, True])
def test_autograd_matches_oracle(basp, w, fused):
    from paper_2609_03151_b200.autograd import basp_attention
    q, k, v, do_ = synth.make_qkv(w, seed=5, with_dO=True)
    Xq, Xk, Xv, Xdo = (synth.bits(t) for t in (q, k, v, do_))
    op = oracle.plan(w.N, w.B, w.S, w.G)
    ref_f = oracle.layer_fwd(Xq, Xk, Xv, op)
    ref_b = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op)
    pl = make_plan(basp, w)
    qs, ks, vs = ([t.requires_grad_() for t in to_dev(oracle.partition(X, op))] for X in (Xq, Xk, Xv))
    dos = to_dev(oracle.partition(Xdo, op))
    basp.basp_clear_status()
    o = basp_attention(pl, qs, ks, vs, fused=fused)
    torch.autograd.backward(o, dos)
    basp.basp_get_status()
    assert_attn_close(to_f64([t.detach() for t in o]), ref_f["o_seq"], w.name)
    for name, xs in (("dq", qs), ("dk", ks), ("dv", vs)):
        r = ref_b[name + "_seq"]
        err = np.abs(to_f64([t.grad for t in xs]) - r)
        assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (name, float(err.max()))
