"""Bit-exact parity of the reshard kernels with the oracle's all-to-all maps (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import to_bits, to_dev
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu

# N, B, G, S, H, D  -- several runs per row, ragged tails (shards not a multiple of the 32 KiB chunk),
# K = 1 (identity), non-power-of-two runs (Qwen: 7 heads per rank), Ulysses with several sequences per rank.
CASES = [
    (4, 2, 0, 1024, 8, 64),
    (8, 2, 0, 2048, 32, 128),
    (8, 2, 0, 2048, 8, 128),
    (8, 1, 0, 1024, 32, 128),
    (8, 8, 0, 256, 8, 128),
    (8, 2, 0, 520, 28, 128),
    (8, 2, 0, 520, 4, 128),
    (8, 4, 1, 136, 16, 64),
    (8, 4, 2, 200, 8, 8),
    (6, 3, 0, 50, 6, 24),
    (1, 1, 0, 3, 1, 8),
]


@pytest.mark.parametrize("N,B,G,S,H,D", CASES)
def test_s2h_h2s_bit_exact(basp, N, B, G, S, H, D):
    pl = basp.basp_plan_create(N, B, S, H, H, D, num_groups=G)
    op = oracle.plan(N, B, S, G)
    seq = synth.random_bits((N, op.Bl, op.T, H, D), seed=S + H)
    want_head = oracle.s2h(seq, op)
    d_seq = to_dev(seq)
    d_head = [torch.zeros(want_head.shape[1:], dtype=torch.bfloat16, device="cuda") for _ in range(N)]
    basp.basp_reshard_s2h(pl, H, d_seq, d_head)
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(d_head), want_head)
    d_back = [torch.zeros_like(t) for t in d_seq]
    basp.basp_reshard_h2s(pl, H, d_head, d_back)
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(d_back), oracle.h2s(want_head, op))
    assert np.array_equal(to_bits(d_back), seq)


def test_qkv_single_launch_gqa(basp):
    N, B, S, Hq, Hkv, D = 8, 2, 1024, 28, 4, 128
    pl = basp.basp_plan_create(N, B, S, Hq, Hkv, D)
    op = oracle.plan(N, B, S)
    arenas = [synth.random_bits((N, 1, op.T, h, D), seed=i) for i, h in enumerate((Hq, Hkv, Hkv))]
    want = [oracle.s2h(a, op) for a in arenas]
    src = [to_dev(a) for a in arenas]
    dst = [[torch.zeros(w.shape[1:], dtype=torch.bfloat16, device="cuda") for _ in range(N)] for w in want]
    n0 = basp.basp_launch_count()
    basp.basp_reshard_qkv_s2h(pl, *src, *dst)
    torch.cuda.synchronize()
    assert basp.basp_launch_count() == n0 + 1
    for d, w in zip(dst, want):
        assert np.array_equal(to_bits(d), w)


def test_arena_slices_and_guard_bands(basp):
    """Shards as consecutive slices of one allocation, with canaries around every destination."""
    N, B, S, H, D = 4, 2, 512, 8, 64
    pl = basp.basp_plan_create(N, B, S, H, H, D)
    op = oracle.plan(N, B, S)
    seq = synth.random_bits((N, 1, op.T, H, D), seed=3)
    shard = seq[0].size
    pad = 64
    arena = torch.full((N * (shard + pad) + pad,), -1, dtype=torch.int16, device="cuda")
    src = torch.from_numpy(seq.view(np.int16)).cuda()
    dst = [arena[pad + r * (shard + pad): pad + r * (shard + pad) + shard] for r in range(N)]
    basp.basp_reshard_s2h(pl, H, [src[r] for r in range(N)], dst)
    torch.cuda.synchronize()
    got = np.stack([d.cpu().numpy().view(np.uint16).reshape(1, S, H // op.K, D) for d in dst])
    assert np.array_equal(got, oracle.s2h(seq, op))
    a = arena.cpu().numpy()
    for r in range(N + 1):
        assert (a[r * (shard + pad): r * (shard + pad) + pad] == -1).all()


@pytest.mark.parametrize("name", ["llama3_8b_32k", "sweep_b1", "sweep_b4", "sweep_b8", "qwen25_7b_64k",
                                  "llama3_8b_128k_train"])
def test_full_size_reshard_sampled(basp, name):
    """The benchmark shapes from 32K to 128K tokens at full size (the launches the benchmark times): the closed-form
    destination of sampled source runs, plus the round trip being the identity."""
    w = synth.WORKLOADS[name]
    pl = basp.basp_plan_create(w.N, w.B, w.S, w.Hq, w.Hkv, w.D)
    g = torch.Generator(device="cuda").manual_seed(0)
    T, K, Hl = pl.T, pl.K, pl.Hq_l
    seq = [torch.randint(-32768, 32767, (1, T, w.Hq, w.D), dtype=torch.int16, device="cuda", generator=g) for _ in range(w.N)]
    head = [torch.zeros((1, w.S, Hl, w.D), dtype=torch.int16, device="cuda") for _ in range(w.N)]
    basp.basp_reshard_s2h(pl, w.Hq, seq, head)
    rng = np.random.default_rng(0)
    for _ in range(200):
        r, t, h = int(rng.integers(w.N)), int(rng.integers(T)), int(rng.integers(w.Hq))
        gidx, l = divmod(r, K)
        m, hp = divmod(h, Hl)
        assert torch.equal(head[gidx * K + m][0, l * T + t, hp], seq[r][0, t, h])
    back = [torch.zeros_like(s) for s in seq]
    basp.basp_reshard_h2s(pl, w.Hq, head, back)
    torch.cuda.synchronize()
    for a, b in zip(seq, back):
        assert torch.equal(a, b)


@pytest.mark.parametrize("name", ["llama3_8b_32k", "qwen25_7b_64k"])
def test_full_size_three_tensor_exchange_against_oracle(basp, name):
    """The launches the benchmark times, at full size and on every element: Q, K and V through the one-launch first
    exchange (basp_reshard_qkv_s2h) and O through the reverse one, bit for bit against the oracle's index loops."""
    w = synth.WORKLOADS[name]
    pl = basp.basp_plan_create(w.N, w.B, w.S, w.Hq, w.Hkv, w.D)
    op = oracle.plan(w.N, w.B, w.S)
    seq = [synth.random_bits((w.N, 1, pl.T, h, w.D), seed=i) for i, h in enumerate((w.Hq, w.Hkv, w.Hkv))]
    src = [to_dev(a) for a in seq]
    dst = [[torch.zeros((1, w.S, h // pl.K, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
           for h in (w.Hq, w.Hkv, w.Hkv)]
    basp.basp_reshard_qkv_s2h(pl, *src, *dst)
    torch.cuda.synchronize()
    for a, d in zip(seq, dst):
        assert np.array_equal(np.stack([synth.bits(t.cpu()) for t in d]), oracle.s2h(a, op))
    back = [torch.zeros_like(t) for t in src[0]]
    basp.basp_reshard_h2s(pl, w.Hq, dst[0], back)              # the head-sharded Q stands in for O: same shape
    torch.cuda.synchronize()
    assert np.array_equal(np.stack([synth.bits(t.cpu()) for t in back]), seq[0])
    assert np.array_equal(oracle.h2s(oracle.s2h(seq[0], op), op), seq[0])
