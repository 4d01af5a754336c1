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
