"""Pins of the oracle's attention (Section II-A equation + causal mask) against closed
forms, brute force, a library routine, and the equivalence the paper claims between BASP,
standard Ulysses and unpartitioned attention."""
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


def brute(Q, K, V, scale, causal=True):
    """Explicit S x S matrix, no max subtraction, written independently of the C code."""
    q, k, v = f64(Q), f64(K), f64(V)
    Bn, S, Hq, D = q.shape
    rep = Hq // k.shape[2]
    O = np.zeros((Bn, S, Hq, D))
    L = np.zeros((Bn, Hq, S))
    for b in range(Bn):
        for h in range(Hq):
            A = np.exp(scale * (q[b, :, h] @ k[b, :, h // rep].T))
            if causal:
                A = np.tril(A)
            O[b, :, h] = (A / A.sum(1, keepdims=True)) @ v[b, :, h // rep]
            L[b, h] = np.log(A.sum(1))
    return O, L


@pytest.mark.parametrize("Bn,S,Hq,Hkv,D,causal", [(1, 1, 1, 1, 4, True), (2, 37, 4, 2, 8, True),
                                                    (1, 64, 6, 2, 16, True), (1, 33, 2, 1, 8, False)])
def test_brute_force(Bn, S, Hq, Hkv, D, causal):
    Q, K, V = rand_bits((Bn, S, Hq, D), 1), rand_bits((Bn, S, Hkv, D), 2), rand_bits((Bn, S, Hkv, D), 3)
    O, L = oracle.attn_fwd(Q, K, V, scale=0.3, causal=causal)
    Ob, Lb = brute(Q, K, V, 0.3, causal)
    assert np.abs(O - Ob).max() < 1e-12
    assert np.abs(L - Lb).max() < 1e-12


@pytest.mark.parametrize("S,Hq,Hkv,D", [(128, 4, 4, 64), (200, 8, 2, 32)])
def test_library_sdpa_fp64(S, Hq, Hkv, D):
    Q, K, V = rand_bits((2, S, Hq, D), 4), rand_bits((2, S, Hkv, D), 5), rand_bits((2, S, Hkv, D), 6)
    O, _ = oracle.attn_fwd(Q, K, V)            # default scale 1/sqrt(D)
    tq, tk, tv = (torch.from_numpy(f64(a)).permute(0, 2, 1, 3) for a in (Q, K, V))
    rep = Hq // Hkv
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(rep, 1), tv.repeat_interleave(rep, 1), is_causal=True)
    assert np.abs(O - ref.permute(0, 2, 1, 3).numpy()).max() < 1e-12


def test_closed_forms():
    S, H, D = 50, 2, 8
    Q, K, V = rand_bits((1, S, H, D), 7), rand_bits((1, S, H, D), 8), rand_bits((1, S, H, D), 9)
    O, L = oracle.attn_fwd(Q, K, V)
    v = f64(V)
    # row 0 attends to itself only
    assert np.array_equal(O[:, 0], v[:, 0])
    assert np.allclose(L[0, :, 0], np.einsum("hd,hd->h", f64(Q)[0, 0], f64(K)[0, 0]) / np.sqrt(D), atol=1e-14)
    # Q = 0 -> uniform weights -> prefix mean of V, LSE = ln(i+1)
    O0, L0 = oracle.attn_fwd(np.zeros_like(Q), K, V)
    want = np.cumsum(v, axis=1) / np.arange(1, S + 1)[None, :, None, None]
    assert np.abs(O0 - want).max() < 1e-13
    assert np.abs(L0 - np.log(np.arange(1, S + 1))[None, None, :]).max() < 1e-13
    # V constant per head -> O equals that constant
    Vc = np.broadcast_to(V[:, :1], V.shape).copy()
    Oc, _ = oracle.attn_fwd(Q, K, Vc)
    assert np.abs(Oc - f64(Vc)).max() < 1e-13
    # scale really multiplies the logits: doubling K's exponent (x2 exactly in bf16) == scale x2
    K2 = synth.bits(synth.from_bits(K) * 2)
    Oa, _ = oracle.attn_fwd(Q, K2, V, scale=0.25)
    Ob, _ = oracle.attn_fwd(Q, K, V, scale=0.5)
    assert np.abs(Oa - Ob).max() < 1e-13


def test_head_permutation_and_gqa_mapping():
    S, Hq, Hkv, D = 24, 6, 3, 4
    Q, K, V = rand_bits((1, S, Hq, D), 10), rand_bits((1, S, Hkv, D), 11), rand_bits((1, S, Hkv, D), 12)
    O, _ = oracle.attn_fwd(Q, K, V)
    # q head h must read kv head h // 2: compare with single-head calls
    for h in range(Hq):
        Oh, _ = oracle.attn_fwd(Q[:, :, h:h + 1], K[:, :, h // 2:h // 2 + 1], V[:, :, h // 2:h // 2 + 1])
        assert np.array_equal(Oh[:, :, 0], O[:, :, h])


def test_rows_entry_matches_full():
    S, Hq, Hkv, D = 70, 4, 2, 8
    Q, K, V = rand_bits((2, S, Hq, D), 13), rand_bits((2, S, Hkv, D), 14), rand_bits((2, S, Hkv, D), 15)
    O, L = oracle.attn_fwd(Q, K, V)
    rows = np.array([(0, 0, 0), (1, 3, 69), (0, 2, 31), (1, 1, 5)], dtype=np.int32)
    Or, Lr = oracle.attn_fwd_rows(Q, K, V, rows)
    for n, (b, h, i) in enumerate(rows):
        assert np.array_equal(Or[n], O[b, i, h]) and Lr[n] == L[b, h, i]


@pytest.mark.parametrize("N,B,S,Hq,Hkv,D", [(4, 2, 64, 8, 8, 8), (8, 2, 64, 8, 4, 4), (8, 4, 32, 16, 8, 4)])
def test_basp_equals_ulysses_equals_unpartitioned(N, B, S, Hq, Hkv, D):
    """Grouping is an exact re-arrangement: BASP (G=B), standard Ulysses (G=1) and plain
    attention on the unpartitioned batch give the same output (Section II-C, IV-B)."""
    Xq, Xk, Xv = rand_bits((B, S, Hq, D), 20), rand_bits((B, S, Hkv, D), 21), rand_bits((B, S, Hkv, D), 22)
    full, _ = oracle.attn_fwd(Xq, Xk, Xv)
    basp = oracle.layer_fwd(Xq, Xk, Xv, oracle.plan(N, B, S))
    assert np.array_equal(basp["o_global"], full)
    if Hkv % N == 0:
        ul = oracle.layer_fwd(Xq, Xk, Xv, oracle.plan(N, B, S, G=1))
        assert np.array_equal(ul["o_global"], full)
    one = oracle.layer_fwd(Xq, Xk, Xv, oracle.plan(B, B, S))   # K = 1: nothing is sharded
    assert np.array_equal(one["o_global"], full)
