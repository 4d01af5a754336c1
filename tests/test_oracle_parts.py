"""Pins of the oracle's unequal group formation (B does not divide N: the paper's future work; reading: B groups of
contiguous ranks whose sizes differ by at most one, as two uniform plans).  Checked against what the structure
fixes: the sizes, the disjoint contiguous cover of ranks and sequences, the reduction to Algorithm 1 when B divides N,
and the paper's exactness claim (Section IV-C): the layer over any grouping equals attention on the unpartitioned
tensors."""
import numpy as np
import pytest

import oracle
from paper_2609_03151_b200 import synth


@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 12, 16])
def test_group_sizes(N):
    for B in range(1, N + 1):
        sizes = oracle.group_sizes(N, B)
        assert len(sizes) == B and sum(sizes) == N and max(sizes) - min(sizes) <= 1
        assert sizes == sorted(sizes, reverse=True) and min(sizes) >= 1
        if N % B == 0:
            assert sizes == [N // B] * B                     # Algorithm 1: K = N / B


def test_more_sequences_than_ranks_is_invalid():
    with pytest.raises(ValueError):
        oracle.group_sizes(4, 5)


@pytest.mark.parametrize("N,B", [(8, 3), (8, 5), (7, 2), (5, 5), (8, 2), (6, 4)])
def test_parts_cover_ranks_and_sequences(N, B):
    S = 840                                                   # divisible by 1..8
    parts = oracle.plan_parts(N, B, S)
    assert 1 <= len(parts) <= 2
    ranks, seqs = [], []
    for pt in parts:
        assert pt.plan.G == pt.plan.B and pt.plan.Bl == 1     # one sequence per group, as in BASP
        ranks += list(range(pt.rank_begin, pt.rank_begin + pt.plan.N))
        seqs += list(range(pt.seq_begin, pt.seq_begin + pt.plan.B))
        for g in range(pt.plan.G):                            # a group is a contiguous block of ranks
            assert pt.plan.group_ranks(g) == list(range(g * pt.plan.K, (g + 1) * pt.plan.K))
    assert ranks == list(range(N)) and seqs == list(range(B))
    assert [pt.plan.K for pt in parts for _ in range(pt.plan.G)] == oracle.group_sizes(N, B)
    if N % B == 0:
        assert len(parts) == 1 and parts[0].plan == oracle.plan(N, B, S)


@pytest.mark.parametrize("N,B,S,Hq,Hkv", [(8, 3, 96, 12, 6), (5, 2, 90, 6, 6), (7, 3, 100, 6, 6)])
def test_layer_over_unequal_groups_equals_unpartitioned_attention(N, B, S, Hq, Hkv):
    D = 8
    w = synth.Workload("parts", N=B, B=B, S=S, Hq=Hq, Hkv=Hkv, D=D)          # only the tensor shapes matter here
    Xq, Xk, Xv, XdO = (synth.bits(t) for t in synth.make_qkv(w, seed=9, with_dO=True))
    parts = oracle.plan_parts(N, B, S)
    assert len(parts) == 2
    ref_o, _ = oracle.attn_fwd(Xq, Xk, Xv)
    got = oracle.layer_fwd_parts(Xq, Xk, Xv, parts)
    assert np.abs(got["o_global"] - ref_o).max() < 1e-13
    ref = oracle.attn_bwd(Xq, Xk, Xv, XdO)
    gb = oracle.layer_bwd_parts(Xq, Xk, Xv, XdO, parts)
    for n, key in (("dq", "dQ"), ("dk", "dK"), ("dv", "dV")):
        assert np.abs(gb[n + "_global"] - ref[key]).max() < 1e-12 * max(1.0, np.abs(ref[key]).max()), n
