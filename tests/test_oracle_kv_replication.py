"""Pins of the oracle's reading for a group with more ranks than KV heads (the paper does not treat grouped-query
attention): each KV head goes to the K/Hkv consecutive local ranks whose query heads read it."""
import numpy as np
import pytest

import oracle
from paper_2609_03151_b200 import synth


def _inputs(w, seed=3):
    q, k, v = synth.make_qkv(w, seed)
    return synth.bits(q), synth.bits(k), synth.bits(v)


@pytest.mark.parametrize("N,B,Hq,Hkv", [(4, 1, 8, 2), (8, 2, 8, 1), (8, 1, 16, 4), (4, 1, 4, 1)])
def test_replicated_exchange_from_global_coordinates(N, B, Hq, Hkv):
    """Brute force from GLOBAL coordinates: local rank m of group g must hold, for its group's sequence(s), every
    token of exactly the KV head that its query heads [m Hq/K, (m+1) Hq/K) map to under h -> h / (Hq/Hkv)."""
    w = synth.Workload("r", N=N, B=B, S=32, Hq=Hq, Hkv=Hkv, D=8)
    _, Xk, _ = _inputs(w)
    pl = oracle.plan(N, B, w.S)
    assert Hkv < pl.K and pl.K % Hkv == 0
    got = oracle.s2h_replicated(oracle.partition(Xk, pl), pl)
    assert got.shape == (N, pl.Bl, w.S, 1, w.D)
    for r in range(N):
        g, m = divmod(r, pl.K)
        heads = {h // (Hq // Hkv) for h in range(m * Hq // pl.K, (m + 1) * Hq // pl.K)}
        assert len(heads) == 1                      # all query heads of a rank read the same KV head
        kv = heads.pop()
        assert oracle.Plan.rank_info(pl, r, Hq, Hkv)["kv_head_begin"] == kv
        assert oracle.Plan.rank_info(pl, r, Hq, Hkv)["kv_head_end"] == kv + 1
        for bl in range(pl.Bl):
            assert np.array_equal(got[r, bl, :, 0, :], Xk[g * pl.Bl + bl, :, kv, :])


@pytest.mark.parametrize("N,B,Hq,Hkv", [(4, 1, 8, 2), (8, 2, 8, 1), (8, 1, 16, 4)])
def test_layer_with_replication_equals_global_attention(N, B, Hq, Hkv):
    """The grouping never changes the result (Section IV-C): the layer with replicated KV heads equals the
    unpartitioned definition, and the plan without replication (fewer ranks) exactly."""
    w = synth.Workload("r", N=N, B=B, S=64, Hq=Hq, Hkv=Hkv, D=16)
    Xq, Xk, Xv = _inputs(w)
    full, full_lse = oracle.attn_fwd(Xq, Xk, Xv)
    rep = oracle.layer_fwd(Xq, Xk, Xv, oracle.plan(N, B, w.S))
    assert np.array_equal(rep["o_global"], full)
    small = oracle.layer_fwd(Xq, Xk, Xv, oracle.plan(B * Hkv, B, w.S))      # K = Hkv: one KV head per rank, no copies
    assert np.array_equal(small["o_global"], full)


def test_replicated_equals_plain_exchange_when_heads_are_repeated():
    """Repeating every KV head K/Hkv times turns the replicated exchange into the plain one."""
    w = synth.Workload("r", N=4, B=1, S=32, Hq=8, Hkv=2, D=8)
    _, Xk, _ = _inputs(w)
    pl = oracle.plan(4, 1, 32)
    a = oracle.s2h_replicated(oracle.partition(Xk, pl), pl)
    b = oracle.s2h(oracle.partition(np.repeat(Xk, 2, axis=2), pl), pl)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("N,B,Hq,Hkv", [(4, 1, 8, 2), (8, 2, 8, 1)])
def test_backward_with_replication_equals_global_gradients(N, B, Hq, Hkv):
    """dK and dV of a replicated KV head are the sums over its copies: the layer's gradients equal those of the
    unpartitioned attention (oracle.attn_bwd on the global tensors, itself pinned by autograd and finite differences)."""
    w = synth.Workload("r", N=N, B=B, S=64, Hq=Hq, Hkv=Hkv, D=16)
    Xq, Xk, Xv = _inputs(w)
    Xdo = synth.bits(synth.randn_bf16(__import__("torch").Generator().manual_seed(9), Xq.shape))
    ref = oracle.attn_bwd(Xq, Xk, Xv, Xdo)
    got = oracle.layer_bwd(Xq, Xk, Xv, Xdo, oracle.plan(N, B, w.S))
    for n, k in (("dq", "dQ"), ("dk", "dK"), ("dv", "dV")):
        assert np.abs(got[n + "_global"] - ref[k]).max() < 1e-12, n


def test_sum_of_copies_is_the_adjoint_of_the_replicating_exchange():
    """<s2h_replicated(x), y> = <x, h2s_sum_replicated(y)> for arbitrary x, y (the reverse exchange of a gradient is the
    transpose of the forward exchange)."""
    rng = np.random.default_rng(0)
    pl = oracle.plan(8, 2, 32)
    x = rng.standard_normal((8, pl.Bl, pl.T, 2, 4))
    y = rng.standard_normal((8, pl.Bl, pl.S, 1, 4))
    lhs = float((oracle.s2h_replicated(x, pl) * y).sum())
    rhs = float((x * oracle.h2s_sum_replicated(y, pl, 2)).sum())
    assert abs(lhs - rhs) < 1e-9 * max(1.0, abs(lhs))
