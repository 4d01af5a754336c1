"""Pins of the oracle's uneven-shard functions (a sequence length that the group size does not divide: chunk =
ceil(S/K), the group's last rank short).  They are checked against what the mathematics fixes: the shards are a
disjoint cover of every sequence, both exchanges are bijections that undo each other, for a divisible length they
coincide with the C loops of the even case (an independent implementation), and the layer built from them equals
attention on the unpartitioned tensors - the paper's claim that grouping is an exact re-arrangement (Section IV-C)."""
import numpy as np
import pytest

import oracle
from paper_2609_03151_b200 import synth

CASES = [  # N, B, G, S, Hq, Hkv, D
    (4, 2, 0, 1001, 4, 2, 16),      # K=2: 501 + 500
    (4, 1, 0, 1001, 8, 4, 16),      # K=4: 251 * 3 + 248
    (8, 2, 1, 203, 8, 8, 8),        # Ulysses grouping of two sequences, K=8: 26 * 7 + 21
    (8, 4, 2, 77, 4, 4, 8),         # two sequences per group, K=4: 20 * 3 + 17
    (4, 1, 0, 131, 8, 2, 8),        # replicated KV heads (K=4 > Hkv=2)
]


def _ids(shape):
    return np.arange(int(np.prod(shape)), dtype=np.int64).reshape(shape)


@pytest.mark.parametrize("N,B,G,S,Hq,Hkv,D", CASES)
def test_plan_and_cover(N, B, G, S, Hq, Hkv, D):
    pl = oracle.plan_uneven(N, B, S, G)
    assert pl.K * pl.G == N and pl.T == -(-S // pl.K) and pl.uneven
    ranges = [pl.token_range(l) for l in range(pl.K)]
    assert ranges[0][0] == 0 and ranges[-1][1] == S
    assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))           # contiguous, disjoint, in order
    assert all(e - b == pl.T for b, e in ranges[:-1]) and ranges[-1][1] - ranges[-1][0] == pl.T_last
    X = _ids((B, S, Hq, D))
    shards = oracle.partition_uneven(X, pl)
    assert sum(s.size for s in shards) == X.size
    assert np.array_equal(np.sort(np.concatenate([s.ravel() for s in shards])), X.ravel())   # every element once
    assert np.array_equal(oracle.gather_uneven(shards, pl), X)
    # Algorithm 2's slice, rank by rank
    for r in (0, N - 1):
        g, l = divmod(r, pl.K)
        t0, t1 = ranges[l]
        assert np.array_equal(shards[r], X[g * pl.Bl:(g + 1) * pl.Bl, t0:t1])


def test_empty_last_rank_is_invalid():
    with pytest.raises(ValueError):
        oracle.plan_uneven(4, 1, 5)          # ceil(5/4) = 2: ranks would hold 2, 2, 1, 0 tokens
    with pytest.raises(ValueError):
        oracle.plan(4, 1, 5)                 # the even plan still requires K | S
    assert oracle.plan_uneven(4, 1, 7).T_last == 1


@pytest.mark.parametrize("N,B,G,S,Hq,Hkv,D", CASES)
def test_exchanges_are_inverse_bijections(N, B, G, S, Hq, Hkv, D):
    pl = oracle.plan_uneven(N, B, S, G)
    X = _ids((B, S, Hq, D))
    seq = oracle.partition_uneven(X, pl)
    head = oracle.s2h_uneven(seq, pl)
    assert head.shape == (N, pl.Bl, S, Hq // pl.K, D)
    assert np.array_equal(np.sort(head.ravel()), X.ravel())
    # closed form of the destination: rank gK+m holds heads [m Hq/K, (m+1) Hq/K) of its group's whole sequences
    Hl = Hq // pl.K
    for g in range(pl.G):
        for m in range(pl.K):
            assert np.array_equal(head[g * pl.K + m], X[g * pl.Bl:(g + 1) * pl.Bl, :, m * Hl:(m + 1) * Hl, :])
    back = oracle.h2s_uneven(head, pl)
    assert all(np.array_equal(a, b) for a, b in zip(back, seq))


def test_even_length_reduces_to_the_even_functions():
    # chunk = ceil(S/K) = S/K: the slice-based functions must reproduce the C loops of the even case
    N, B, S, Hq, D = 8, 2, 64, 8, 4
    ple = oracle.plan(N, B, S)
    plu = oracle.Plan(N=N, B=B, G=ple.G, K=ple.K, Bl=ple.Bl, S=S, T=ple.T, T_last=ple.T)
    assert not plu.uneven
    X = synth.random_bits((B, S, Hq, D), seed=5)
    seq_e = oracle.partition(X, ple)
    seq_u = oracle.partition_uneven(X, plu)
    assert np.array_equal(np.stack(seq_u), seq_e)
    assert np.array_equal(oracle.s2h_uneven(seq_u, plu), oracle.s2h(seq_e, ple))
    head = oracle.s2h(seq_e, ple)
    assert np.array_equal(np.stack(oracle.h2s_uneven(head, plu)), oracle.h2s(head, ple))
    Xkv = synth.random_bits((B, S, 2, D), seed=6)              # replicated: K=4 > 2 heads
    assert np.array_equal(oracle.s2h_uneven(oracle.partition_uneven(Xkv, plu), plu),
                          oracle.s2h_replicated(oracle.partition(Xkv, ple), ple))
    gh = np.random.default_rng(0).standard_normal((N, ple.Bl, S, 1, D))
    assert np.allclose(np.stack(oracle.h2s_uneven(gh, plu, 2)), oracle.h2s_sum_replicated(gh, ple, 2), rtol=0, atol=0)


@pytest.mark.parametrize("N,B,G,S,Hq,Hkv,D", CASES)
def test_layer_equals_unpartitioned_attention(N, B, G, S, Hq, Hkv, D):
    pl = oracle.plan_uneven(N, B, S, G)
    w = synth.Workload("uneven", N=N, B=B, S=S, Hq=Hq, Hkv=Hkv, D=D, G=G)
    Xq, Xk, Xv, XdO = (synth.bits(t) for t in synth.make_qkv(w, seed=1, with_dO=True))
    for causal in (True, False):
        ref_o, ref_lse = oracle.attn_fwd(Xq, Xk, Xv, causal=causal)
        got = oracle.layer_fwd(Xq, Xk, Xv, pl, causal=causal)
        assert np.abs(got["o_global"] - ref_o).max() < 1e-13
        assert [s.shape[1] for s in got["o_seq"][:pl.K]] == [pl.T] * (pl.K - 1) + [pl.T_last]
    ref = oracle.attn_bwd(Xq, Xk, Xv, XdO)
    got = oracle.layer_bwd(Xq, Xk, Xv, XdO, pl)
    for n, key in (("dq", "dQ"), ("dk", "dK"), ("dv", "dV")):
        scale = max(1.0, np.abs(ref[key]).max())
        assert np.abs(got[n + "_global"] - ref[key]).max() < 1e-12 * scale, n
