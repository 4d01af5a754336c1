"""Pins of the oracle's attention backward against finite differences of the oracle's own (pinned)
forward, fp64 autograd of a library routine, and invariants of the softmax Jacobian."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_03151_b200 import synth


def rand_bits(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return synth.bits((torch.randn(shape, generator=g) * scale).to(torch.bfloat16))


def f64(b):
    return oracle.bf16_bits_to_f64(b)


def autograd_ref(Q, K, V, dO, scale, causal):
    q, k, v = (torch.from_numpy(f64(a)).permute(0, 2, 1, 3).clone().requires_grad_(True) for a in (Q, K, V))
    rep = q.shape[1] // k.shape[1]
    o = torch.nn.functional.scaled_dot_product_attention(q, k.repeat_interleave(rep, 1), v.repeat_interleave(rep, 1),
                                                         is_causal=causal, scale=scale)
    o.backward(torch.from_numpy(f64(dO)).permute(0, 2, 1, 3))
    return tuple(t.grad.permute(0, 2, 1, 3).numpy() for t in (q, k, v))


@pytest.mark.parametrize("Bn,S,Hq,Hkv,D,causal", [(1, 40, 2, 2, 8, True), (2, 33, 4, 2, 16, True), (1, 24, 6, 2, 8, False)])
def test_library_autograd_fp64(Bn, S, Hq, Hkv, D, causal):
    Q, K, V, dO = (rand_bits(s, i) for i, s in enumerate([(Bn, S, Hq, D), (Bn, S, Hkv, D), (Bn, S, Hkv, D), (Bn, S, Hq, D)]))
    g = oracle.attn_bwd(Q, K, V, dO, scale=0.3, causal=causal)
    rq, rk, rv = autograd_ref(Q, K, V, dO, 0.3, causal)
    assert np.abs(g["dQ"] - rq).max() < 1e-11
    assert np.abs(g["dK"] - rk).max() < 1e-11
    assert np.abs(g["dV"] - rv).max() < 1e-11
    O, L = oracle.attn_fwd(Q, K, V, scale=0.3, causal=causal)
    assert np.abs(g["LSE"] - L).max() < 1e-12
    assert np.abs(g["DELTA"] - np.einsum("bshd,bshd->bhs", f64(dO), O)).max() < 1e-12


def test_finite_differences_of_the_forward():
    """d/dx of loss = sum(O * dO), central differences in fp64 on exactly representable inputs."""
    Bn, S, Hq, Hkv, D = 1, 6, 2, 1, 4
    Q, K, V, dO = (rand_bits(s, 10 + i) for i, s in enumerate([(Bn, S, Hq, D), (Bn, S, Hkv, D), (Bn, S, Hkv, D), (Bn, S, Hq, D)]))
    g = oracle.attn_bwd(Q, K, V, dO)

    def loss(q, k, v):       # the forward definition itself, in numpy fp64 (inputs no longer bf16-exact)
        rep = Hq // Hkv
        tot = 0.0
        for h in range(Hq):
            A = np.tril(np.exp((q[0, :, h] @ k[0, :, h // rep].T) / np.sqrt(D)))
            tot += (((A / A.sum(1, keepdims=True)) @ v[0, :, h // rep]) * f64(dO)[0, :, h]).sum()
        return tot

    base = [f64(Q), f64(K), f64(V)]
    eps = 1e-6
    for which, name in enumerate(("dQ", "dK", "dV")):
        num = np.zeros_like(base[which])
        for idx in np.ndindex(*base[which].shape):
            a = [x.copy() for x in base]
            a[which][idx] += eps
            b = [x.copy() for x in base]
            b[which][idx] -= eps
            num[idx] = (loss(*a) - loss(*b)) / (2 * eps)
        assert np.abs(num - g[name]).max() < 1e-8, name


def test_softmax_jacobian_invariants():
    Bn, S, Hq, Hkv, D = 1, 30, 2, 1, 8
    Q, K, V, dO = (rand_bits(s, 20 + i) for i, s in enumerate([(Bn, S, Hq, D), (Bn, S, Hkv, D), (Bn, S, Hkv, D), (Bn, S, Hq, D)]))
    # dO constant along d and V constant along positions -> O does not depend on the scores -> dQ = dK = 0
    Vc = np.broadcast_to(V[:, :1], V.shape).copy()
    g = oracle.attn_bwd(Q, K, Vc, dO)
    assert np.abs(g["dQ"]).max() < 1e-13 and np.abs(g["dK"]).max() < 1e-13
    # dV_j = sum_i P_ij dO_i: with Q = 0 the weights are 1/(i+1)
    g0 = oracle.attn_bwd(np.zeros_like(Q), K, V, dO)
    do = f64(dO)
    want = np.zeros((S, D))
    for j in range(S):
        for h in range(Hq):
            want[j] += sum(do[0, i, h] / (i + 1) for i in range(j, S))
    assert np.abs(g0["dV"][0, :, 0] - want).max() < 1e-12
    # row 0 sees only itself: P = 1, dS = 0 -> dQ_0 = 0
    g = oracle.attn_bwd(Q, K, V, dO)
    assert np.abs(g["dQ"][:, 0]).max() < 1e-13


def test_sparse_entries_match_full():
    Bn, S, Hq, Hkv, D = 2, 50, 4, 2, 8
    Q, K, V, dO = (rand_bits(s, 30 + i) for i, s in enumerate([(Bn, S, Hq, D), (Bn, S, Hkv, D), (Bn, S, Hkv, D), (Bn, S, Hq, D)]))
    g = oracle.attn_bwd(Q, K, V, dO)
    rows = np.array([(0, 0, 0), (1, 3, 49), (0, 2, 17)], dtype=np.int32)
    dq = oracle.attn_bwd_dq_rows(Q, K, V, dO, rows)
    for n, (b, h, i) in enumerate(rows):
        assert np.allclose(dq[n], g["dQ"][b, i, h], rtol=0, atol=1e-13)
    dk, dv = oracle.attn_bwd_dkdv_tail(Q, K, V, dO, b=1, kv=1, ncols=7)
    assert np.allclose(dk, g["dK"][1, S - 7:, 1], rtol=0, atol=1e-13)
    assert np.allclose(dv, g["dV"][1, S - 7:, 1], rtol=0, atol=1e-13)


@pytest.mark.parametrize("causal", [True, False])
def test_column_entry_matches_library_autograd_and_full_entry(causal):
    """The arbitrary-column dK/dV entry (used for the large shapes): unordered columns, a repeated one, the first and
    the last position, on a GQA shape; against fp64 autograd of the library routine and against the full entry."""
    Bn, S, Hq, Hkv, D = 2, 61, 6, 2, 8
    Q, K, V, dO = (rand_bits(s, 50 + i) for i, s in enumerate([(Bn, S, Hq, D), (Bn, S, Hkv, D), (Bn, S, Hkv, D), (Bn, S, Hq, D)]))
    _, rk, rv = autograd_ref(Q, K, V, dO, 0.3, causal)
    g = oracle.attn_bwd(Q, K, V, dO, scale=0.3, causal=causal)
    cols = [40, 7, 60, 0, 7, 33]
    for b, kv in ((0, 0), (1, 1)):
        dk, dv = oracle.attn_bwd_dkdv_cols(Q, K, V, dO, b=b, kv=kv, cols=cols, scale=0.3, causal=causal)
        assert np.abs(dk - rk[b, cols, kv]).max() < 1e-11
        assert np.abs(dv - rv[b, cols, kv]).max() < 1e-11
        assert np.allclose(dk, g["dK"][b, cols, kv], rtol=0, atol=1e-13)
        assert np.allclose(dv, g["dV"][b, cols, kv], rtol=0, atol=1e-13)
    # a single late column needs the statistics of the rows behind it only, and gives the same numbers
    dk1, dv1 = oracle.attn_bwd_dkdv_cols(Q, K, V, dO, b=1, kv=1, cols=[55], scale=0.3, causal=causal)
    assert np.allclose(dk1[0], g["dK"][1, 55, 1], rtol=0, atol=1e-13) and np.allclose(dv1[0], g["dV"][1, 55, 1], rtol=0, atol=1e-13)


def test_layer_bwd_grouping_equivalence():
    N, B, S, Hq, Hkv, D = 4, 2, 32, 8, 4, 4
    X = [rand_bits(s, 40 + i) for i, s in enumerate([(B, S, Hq, D), (B, S, Hkv, D), (B, S, Hkv, D), (B, S, Hq, D)])]
    full = oracle.attn_bwd(*X)
    for G in (0, 1):
        lb = oracle.layer_bwd(*X, oracle.plan(N, B, S, G))
        assert np.array_equal(lb["dq_global"], full["dQ"])
        assert np.array_equal(lb["dk_global"], full["dK"])
        assert np.array_equal(lb["dv_global"], full["dV"])
