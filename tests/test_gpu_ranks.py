"""The `*_ranks` entry points (one physical GPU's share when the ranks are spread over several GPUs), checked on
one GPU: the shares of P emulated GPUs are launched one after the other (no launch waits for another), every pointer
is local, and the union must equal the single-GPU call bit for bit and the oracle within tolerance.  Shards a share
does not touch are passed as NULL, which also checks that it really does not touch them."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, oracle_inputs, to_bits, to_dev, to_f64
from paper_2609_03151_b200 import dist as pdist
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [  # (workload, emulated GPUs)
    (synth.Workload("span4_on2", N=4, B=1, S=1024, Hq=8, Hkv=4, D=128), 2),    # one group of 4 ranks over 2 GPUs
    (synth.Workload("span4_on4", N=4, B=1, S=512, Hq=8, Hkv=8, D=64), 4),      # one rank per GPU
    (synth.Workload("two_groups_on4", N=8, B=2, S=1024, Hq=8, Hkv=4, D=128), 4),  # each group of 4 over 2 GPUs
    (synth.Workload("whole_groups", N=8, B=4, S=512, Hq=4, Hkv=2, D=128), 2),  # groups of 2, two groups per GPU
]


def _masked(shards, keep):
    return [t if r in keep else None for r, t in enumerate(shards)]


def _group_members(pl, ranks):
    lo, hi = ranks.start // pl.K * pl.K, (ranks.stop + pl.K - 1) // pl.K * pl.K
    return range(lo, hi)


@pytest.mark.parametrize("w,world", CASES, ids=lambda x: getattr(x, "name", str(x)))
def test_three_step_path_by_shares(basp, w, world):
    Xq, Xk, Xv, op = oracle_inputs(w)
    pl = make_plan(basp, w)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    shape = lambda h: (pl.Bl, pl.S, h // pl.K, w.D)
    mk = lambda h: [torch.zeros(shape(h), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    hq, hk, hv, ho = mk(w.Hq), mk(w.Hkv), mk(w.Hkv), mk(w.Hq)
    o_seq = [torch.zeros_like(t) for t in dq]
    basp.basp_clear_status()
    for gpu in range(world):        # step 1 on every "GPU", then a host barrier, then step 2, ...
        mine = pdist.ranks_of_gpu(w.N, world, gpu)
        grp = _group_members(pl, mine)
        basp.basp_reshard_qkv_s2h_ranks(pl, _masked(dq, mine), _masked(dk, mine), _masked(dv, mine),
                                        _masked(hq, grp), _masked(hk, grp), _masked(hv, grp), mine.start, len(mine))
    for gpu in range(world):
        mine = pdist.ranks_of_gpu(w.N, world, gpu)
        basp.basp_attn_fwd_ranks(pl, _masked(hq, mine), _masked(hk, mine), _masked(hv, mine), _masked(ho, mine),
                                 mine.start, len(mine))
    for gpu in range(world):
        mine = pdist.ranks_of_gpu(w.N, world, gpu)
        basp.basp_reshard_h2s_ranks(pl, w.Hq, _masked(ho, _group_members(pl, mine)), _masked(o_seq, mine),
                                    mine.start, len(mine))
    basp.basp_get_status()
    # the single-GPU calls
    hq1, hk1, hv1, ho1 = mk(w.Hq), mk(w.Hkv), mk(w.Hkv), mk(w.Hq)
    o1 = [torch.zeros_like(t) for t in dq]
    basp.basp_reshard_qkv_s2h(pl, dq, dk, dv, hq1, hk1, hv1)
    basp.basp_attn_fwd(pl, hq1, hk1, hv1, ho1)
    basp.basp_reshard_h2s(pl, w.Hq, ho1, o1)
    basp.basp_get_status()
    for a, b in ((hq, hq1), (hk, hk1), (hv, hv1), (ho, ho1), (o_seq, o1)):
        assert np.array_equal(to_bits(a), to_bits(b))
    assert np.array_equal(to_bits(hq), oracle.s2h(oracle.partition(Xq, op), op))      # the exchange itself: bit-exact
    assert_attn_close(to_f64(o_seq), oracle.layer_fwd(Xq, Xk, Xv, op)["o_seq"], w.name)


@pytest.mark.parametrize("w,world", CASES, ids=lambda x: getattr(x, "name", str(x)))
def test_fused_kernel_by_shares(basp, w, world):
    Xq, Xk, Xv, op = oracle_inputs(w)
    pl = make_plan(basp, w)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    o_seq = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    basp.basp_clear_status()
    for gpu in range(world):
        mine = pdist.ranks_of_gpu(w.N, world, gpu)
        grp = _group_members(pl, mine)
        basp.basp_layer_fwd_fused_ranks(pl, _masked(dq, grp), _masked(dk, grp), _masked(dv, grp), _masked(o_seq, grp),
                                        mine.start, len(mine), lse_shards=_masked(lse, mine))
    basp.basp_get_status()
    o1 = [torch.zeros_like(t) for t in dq]
    lse1 = [torch.zeros_like(t) for t in lse]
    basp.basp_layer_fwd_fused(pl, dq, dk, dv, o1, lse1)
    basp.basp_get_status()
    assert np.array_equal(to_bits(o_seq), to_bits(o1))
    assert all(torch.equal(a, b) for a, b in zip(lse, lse1))
    assert_attn_close(to_f64(o_seq), oracle.layer_fwd(Xq, Xk, Xv, op)["o_seq"], w.name)


def test_range_errors(basp):
    w = synth.WORKLOADS["tiny"]
    pl = make_plan(basp, w)
    t = [torch.zeros((pl.Bl, pl.T, w.Hq, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    o = [torch.zeros_like(x) for x in t]
    for begin, count in ((-1, 1), (3, 2), (0, 5)):
        with pytest.raises(basp.BaspError) as e:
            basp.basp_layer_fwd_fused_ranks(pl, t, t, t, o, begin, count)
        assert e.value.code == basp.BASP_ERR_INVALID
    with pytest.raises(basp.BaspError) as e:      # a member of the group is missing
        basp.basp_layer_fwd_fused_ranks(pl, [None] + t[1:], t, t, o, 1, 1)
    assert e.value.code == basp.BASP_ERR_NULL
    basp.basp_layer_fwd_fused_ranks(pl, t, t, t, o, 2, 0)      # an empty share is a no-op
    basp.basp_get_status()
