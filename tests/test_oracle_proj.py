"""Pins of the oracle's projection (Section II-A: Q = X W_Q etc.) against brute force and special cases."""
import numpy as np
import torch

import oracle
from paper_2609_03151_b200 import synth


def rand_bits(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return synth.bits(torch.randn(shape, generator=g).to(torch.bfloat16))


def test_brute_force_loops():
    X, W = rand_bits((5, 7), 1), rand_bits((3, 7), 2)
    x, w = oracle.bf16_bits_to_f64(X), oracle.bf16_bits_to_f64(W)
    want = np.zeros((5, 3))
    for i in range(5):
        for n in range(3):
            for k in range(7):
                want[i, n] += x[i, k] * w[n, k]
    assert np.abs(oracle.linear(X, W) - want).max() < 1e-13


def test_identity_and_selection_weights():
    X = rand_bits((9, 8), 3)
    eye = synth.bits(torch.eye(8).to(torch.bfloat16))
    assert np.array_equal(oracle.linear(X, eye), oracle.bf16_bits_to_f64(X))
    # a weight row that is a unit vector picks one input feature: output feature n = input feature perm[n]
    perm = [3, 0, 7]
    sel = synth.bits(torch.eye(8)[perm].to(torch.bfloat16))
    assert np.array_equal(oracle.linear(X, sel), oracle.bf16_bits_to_f64(X)[:, perm])


def test_heads_are_row_blocks_of_the_weight():
    """Per-head projection (X W^i_Q for head i) equals the i-th block of D output features of the fused weight."""
    M, K, H, D = 6, 16, 3, 4
    X, W = rand_bits((M, K), 4), rand_bits((H * D, K), 5)
    full = oracle.linear(X, W)
    for i in range(H):
        assert np.array_equal(oracle.linear(X, W[i * D:(i + 1) * D]), full[:, i * D:(i + 1) * D])


# ---- rotary position embedding (rotate-half form) of the oracle
def _exact_tables(S, D, base=10000.0):
    j = np.arange(D // 2, dtype=np.float64)
    ang = np.arange(S, dtype=np.float64)[:, None] * base ** (-2.0 * j / D)[None, :]
    return np.cos(ang), np.sin(ang)


def test_rope_is_a_complex_rotation_of_each_pair():
    rng = np.random.default_rng(1)
    tokens, H, D = 7, 3, 16
    x = rng.standard_normal((tokens, H, D))
    cos, sin = _exact_tables(32, D)
    pos = np.array([0, 5, 9, 31, 2, 2, 17])
    y = oracle.rope(x, cos, sin, pos)
    z = (x[..., :D // 2] + 1j * x[..., D // 2:]) * (cos[pos] + 1j * sin[pos])[:, None, :]
    assert np.abs(y[..., :D // 2] - z.real).max() < 1e-14 and np.abs(y[..., D // 2:] - z.imag).max() < 1e-14
    # explicit loops on one element, written from the definition
    t, h, j = 3, 1, 5
    c, s = cos[pos[t], j], sin[pos[t], j]
    assert abs(y[t, h, j] - (x[t, h, j] * c - x[t, h, j + D // 2] * s)) < 1e-15
    assert abs(y[t, h, j + D // 2] - (x[t, h, j + D // 2] * c + x[t, h, j] * s)) < 1e-15


def test_rope_invariants():
    rng = np.random.default_rng(2)
    D = 32
    cos, sin = _exact_tables(64, D)
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    assert np.array_equal(oracle.rope(q, cos, sin, np.array([0])), q)                  # position 0: identity
    for m, n in ((9, 4), (40, 40), (63, 1)):
        qm, kn = oracle.rope(q, cos, sin, np.array([m])), oracle.rope(k, cos, sin, np.array([n]))
        assert abs(np.linalg.norm(qm) - np.linalg.norm(q)) < 1e-12                     # a rotation keeps lengths
        rel = oracle.rope(q, cos, sin, np.array([m - n]))                               # scores depend on m - n only
        assert abs(float((qm * kn).sum()) - float((rel * k).sum())) < 1e-12


def test_qkv_proj_rope_rotates_q_and_k_only():
    Hq, Hkv, D, hidden, tokens = 4, 2, 8, 16, 5
    X, W = rand_bits((tokens, hidden), 6), rand_bits(((Hq + 2 * Hkv) * D, hidden), 7)
    cos, sin = _exact_tables(16, D)
    pos = np.array([3, 0, 15, 7, 7])
    q, k, v = oracle.qkv_proj_rope(X, W, Hq, Hkv, D, cos, sin, pos)
    Y = oracle.linear(X, W)
    assert np.array_equal(v, Y[:, (Hq + Hkv) * D:].reshape(tokens, Hkv, D))
    assert np.array_equal(q[1], Y[1, :Hq * D].reshape(Hq, D))                            # position 0 is not rotated
    assert np.abs(q - oracle.rope(Y[:, :Hq * D].reshape(tokens, Hq, D), cos, sin, pos)).max() == 0
    assert np.abs(k - oracle.rope(Y[:, Hq * D:(Hq + Hkv) * D].reshape(tokens, Hkv, D), cos, sin, pos)).max() == 0
