"""Pins of the oracle's permutations (Algorithm 2 and the two all-to-alls of Section IV-C)
against independent statements of the same maps."""
import numpy as np
import pytest

import oracle

CASES = [  # N, B, G, S, H, D
    (4, 2, 0, 16, 8, 4),
    (8, 2, 0, 32, 8, 2),
    (8, 1, 0, 64, 16, 2),
    (8, 8, 0, 8, 4, 2),
    (8, 4, 1, 16, 8, 2),    # standard Ulysses, 4 sequences on every rank
    (8, 4, 2, 16, 8, 2),    # two groups of four ranks, two sequences each
    (6, 3, 0, 10, 6, 3),
]


def ids(shape):
    return np.arange(int(np.prod(shape)), dtype=np.int64).reshape(shape)


@pytest.mark.parametrize("N,B,G,S,H,D", CASES)
def test_s2h_semantics_from_global_tensor(N, B, G, S, H, D):
    """After the first all-to-all, local rank m of group g must hold the WHOLE sequence(s)
    of its group for heads [m*H/K, (m+1)*H/K): brute force on global coordinates."""
    pl = oracle.plan(N, B, S, G)
    X = ids((B, S, H, D))
    head = oracle.s2h(oracle.partition(X, pl), pl)
    Hl = H // pl.K
    for r in range(N):
        g, m = divmod(r, pl.K)
        for bl in range(pl.Bl):
            want = X[g * pl.Bl + bl][:, m * Hl:(m + 1) * Hl, :]
            assert np.array_equal(head[r, bl], want)


@pytest.mark.parametrize("N,B,G,S,H,D", CASES)
def test_partition_is_slicing(N, B, G, S, H, D):
    pl = oracle.plan(N, B, S, G)
    X = ids((B, S, H, D))
    sh = oracle.partition(X, pl)
    for r in range(N):
        g, l = divmod(r, pl.K)
        assert np.array_equal(sh[r], X[g * pl.Bl:(g + 1) * pl.Bl, l * pl.T:(l + 1) * pl.T])
    assert np.array_equal(oracle.gather(sh, pl), X)


@pytest.mark.parametrize("N,B,G,S,H,D", CASES)
def test_s2h_equals_axis_transpose(N, B, G, S, H, D):
    """Within a group the all-to-all is the transposition [l, .., t, m, ..] -> [m, .., l, t, ..]."""
    pl = oracle.plan(N, B, S, G)
    rng = np.random.default_rng(1)
    seq = rng.integers(0, 1 << 16, size=(N, pl.Bl, pl.T, H, D), dtype=np.uint16)
    K, Hl = pl.K, H // pl.K
    want = (seq.reshape(pl.G, K, pl.Bl, pl.T, K, Hl, D)      # g l bl t m h' d
               .transpose(0, 4, 2, 1, 3, 5, 6)              # g m bl l t h' d
               .reshape(N, pl.Bl, S, Hl, D))
    got = oracle.s2h(seq, pl)
    assert np.array_equal(got, want)
    back = oracle.h2s(got, pl)
    assert np.array_equal(back, seq)                         # h2s o s2h = identity, bit for bit
    assert np.array_equal(oracle.s2h(oracle.h2s(got, pl), pl), got)


@pytest.mark.parametrize("N,B,G,S,H,D", CASES)
def test_bijection_with_element_ids(N, B, G, S, H, D):
    pl = oracle.plan(N, B, S, G)
    seq = ids((N, pl.Bl, pl.T, H, D))
    head = oracle.s2h(seq, pl)
    assert np.array_equal(np.sort(head.ravel()), seq.ravel())
    seq2 = oracle.h2s(ids(head.shape), pl)
    assert np.array_equal(np.sort(seq2.ravel()), np.arange(seq2.size))


def test_k1_is_identity():
    pl = oracle.plan(8, 8, 8)
    seq = ids((8, 1, 8, 4, 2)).astype(np.uint16)
    assert np.array_equal(oracle.s2h(seq, pl), seq)
    assert np.array_equal(oracle.h2s(seq, pl), seq)


def test_h2s_semantics_from_global_tensor():
    """The reverse all-to-all returns every token to its sequence owner with all heads."""
    N, B, S, H, D = 8, 2, 32, 8, 2
    pl = oracle.plan(N, B, S)
    O = ids((B, S, H, D))
    head = oracle.s2h(oracle.partition(O, pl), pl)
    assert np.array_equal(oracle.gather(oracle.h2s(head, pl), pl), O)
