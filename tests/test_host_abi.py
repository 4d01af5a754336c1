"""CPU-only checks of the C ABI: every declared symbol is exported, the host planner agrees
with the oracle's Algorithm 1 / Algorithm 2, and the argument checks that need no GPU."""
import os
import re

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported(basp):
    text = open(os.path.join(ROOT, "include", "basp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(basp_[a-z0-9_]+)\s*\(", text))
    assert declared == set(basp.EXPORTS), declared ^ set(basp.EXPORTS)
    for name in declared:
        assert hasattr(basp.lib, name), name


@pytest.mark.parametrize("N,B,G", [(4, 2, 0), (8, 1, 0), (8, 2, 0), (8, 4, 0), (8, 8, 0), (8, 4, 1), (8, 4, 2), (16, 4, 0)])
def test_plan_matches_oracle(basp, N, B, G):
    S, Hq, Hkv, D = 4096, 32, 16, 128
    pl = basp.basp_plan_create(N, B, S, Hq, Hkv, D, num_groups=G)
    op = oracle.plan(N, B, S, G)
    assert (pl.K, pl.G, pl.Bl, pl.T) == (op.K, op.G, op.Bl, op.T)
    assert pl.info.q_shard_elems == B * S // N * Hq * D          # tokens per GPU = B*S/N (Table I)
    assert pl.info.kv_shard_elems == B * S // N * Hkv * D
    for g in range(pl.G):
        assert basp.basp_plan_group_ranks(pl, g) == op.group_ranks(g)
    for r in range(N):
        assert basp.basp_plan_get_rank(pl, r) == op.rank_info(r, Hq, Hkv)


@pytest.mark.parametrize("N,B,Hq,Hkv", [(8, 2, 32, 2), (8, 1, 32, 4), (4, 1, 8, 1)])
def test_plan_with_more_ranks_than_kv_heads(basp, N, B, Hq, Hkv):
    """A group with more ranks than KV heads: one (replicated) KV head per rank, as the oracle reads it."""
    S, D = 2048, 128
    pl = basp.basp_plan_create(N, B, S, Hq, Hkv, D)
    op = oracle.plan(N, B, S)
    assert pl.K > Hkv and pl.info.kv_heads_per_rank == 1 and pl.info.q_heads_per_rank == Hq // pl.K
    assert pl.info.kv_shard_elems == B * S // N * Hkv * D       # the sequence-sharded side is unchanged
    for r in range(N):
        assert basp.basp_plan_get_rank(pl, r) == op.rank_info(r, Hq, Hkv)


@pytest.mark.parametrize("N,B,G,S", [(8, 2, 0, 1022), (8, 1, 0, 1001), (4, 2, 1, 203), (8, 4, 2, 77)])
def test_plan_for_a_length_the_group_size_does_not_divide(basp, N, B, G, S):
    pl = basp.basp_plan_create(N, B, S, 8, 8, 64, num_groups=G)
    op = oracle.plan_uneven(N, B, S, G)
    assert (pl.K, pl.T, pl.T_last) == (op.K, op.T, op.T_last) and pl.T_last < pl.T
    for r in range(N):
        ri = basp.basp_plan_get_rank(pl, r)
        assert (ri["token_begin"], ri["token_end"]) == op.token_range(r % op.K)
        assert pl.rank_tokens(r) == ri["token_end"] - ri["token_begin"]
    assert sum(pl.rank_tokens(r) for r in range(pl.K)) == S


@pytest.mark.parametrize("N,B", [(8, 3), (8, 5), (7, 2), (7, 3), (6, 4), (8, 2), (5, 5)])
def test_unequal_group_formation_matches_oracle(basp, N, B):
    S, Hq = 840, 840                                   # divisible by every group size that occurs
    parts = basp.basp_plan_create_parts(N, B, S, Hq, Hq, 16)
    want = oracle.plan_parts(N, B, S)
    assert len(parts) == len(want)
    for got, ref in zip(parts, want):
        assert (got.rank_begin, got.n_ranks, got.seq_begin, got.n_seqs) == (ref.rank_begin, ref.plan.N, ref.seq_begin, ref.plan.B)
        assert (got.plan.K, got.plan.G, got.plan.Bl, got.plan.T) == (ref.plan.K, ref.plan.G, 1, ref.plan.T)
        assert got.group_size == ref.plan.K
    assert [p.group_size for p in parts for _ in range(p.n_seqs)] == oracle.group_sizes(N, B)
    if N % B == 0:
        whole = basp.basp_plan_create(N, B, S, Hq, Hq, 16)
        assert len(parts) == 1 and (parts[0].plan.K, parts[0].plan.T) == (whole.K, whole.T)


def test_unequal_group_formation_errors(basp):
    with pytest.raises(basp.BaspError) as e:
        basp.basp_plan_create_parts(4, 5, 1024, 8, 8, 64)          # more sequences than ranks, and 4 does not divide 5
    assert e.value.code == basp.BASP_ERR_INVALID
    (dp,) = basp.basp_plan_create_parts(4, 8, 1024, 8, 8, 64)      # the data-parallel fallback is one part
    assert (dp.plan.K, dp.plan.Bl, dp.n_ranks, dp.n_seqs) == (1, 2, 4, 8)
    with pytest.raises(basp.BaspError) as e:
        basp.basp_plan_create_parts(8, 3, 1536, 8, 8, 64)          # groups of 3 ranks cannot split 8 heads
    assert e.value.code == basp.BASP_ERR_INVALID


def test_data_parallel_fallback_plan(basp):
    pl = basp.basp_plan_create(4, 8, 1024, 8, 8, 64)                 # B > N: one rank per group, two whole sequences each
    op = oracle.plan(4, 8, 1024)
    assert (pl.K, pl.G, pl.Bl, pl.T) == (op.K, op.G, op.Bl, op.T) == (1, 4, 2, 1024)
    for r in range(4):
        assert basp.basp_plan_get_rank(pl, r) == op.rank_info(r, 8, 8)


def test_paper_example_four_gpus_batch_two(basp):
    pl = basp.basp_plan_create(4, 2, 1024, 8, 8, 64)
    assert pl.K == 2 and [basp.basp_plan_group_ranks(pl, g) for g in range(2)] == [[0, 1], [2, 3]]


@pytest.mark.parametrize("kw,code", [
    (dict(n_ranks=8, micro_batch=3), -1),                 # N mod B != 0
    (dict(n_ranks=4, micro_batch=6), -1),                 # B > N and N does not divide B
    (dict(n_ranks=8, micro_batch=1, seq_len=9), -1),      # chunk = ceil(9/8) = 2 would leave the last ranks empty
    (dict(n_q_heads=30), -1),                             # Hq mod Hkv
    (dict(n_ranks=6, micro_batch=1, seq_len=1536, n_q_heads=24, n_kv_heads=4), -1),   # K = 6: neither Hkv mod K nor K mod Hkv
    (dict(num_groups=3), -1),
    (dict(dtype=1), -2),
    (dict(n_ranks=64, micro_batch=64), -2),               # more than BASP_MAX_RANKS
    (dict(head_dim=3, n_q_heads=4, n_kv_heads=4), -2),    # rows not a multiple of 16 bytes
])
def test_plan_errors(basp, kw, code):
    args = dict(n_ranks=8, micro_batch=2, seq_len=1024, n_q_heads=32, n_kv_heads=8, head_dim=128)
    args.update(kw)
    with pytest.raises(basp.BaspError) as e:
        basp.basp_plan_create(**args)
    assert e.value.code == code


def test_null_and_alignment_checks_need_no_gpu(basp):
    import ctypes
    pl = basp.basp_plan_create(4, 2, 1024, 8, 8, 64)
    n = 4
    good = (ctypes.c_void_p * n)(*[0x10000 * (i + 1) for i in range(n)])
    good2 = (ctypes.c_void_p * n)(*[0x10000000 + 0x100000 * (i + 1) for i in range(n)])
    odd = (ctypes.c_void_p * n)(*[0x10000 * (i + 1) + 8 for i in range(n)])
    null = (ctypes.c_void_p * n)(*[None] * n)
    L = basp.lib
    assert L.basp_reshard_s2h(pl.handle, 8, None, good, None) == basp.BASP_ERR_NULL
    assert L.basp_reshard_s2h(pl.handle, 8, null, good, None) == basp.BASP_ERR_NULL
    assert L.basp_reshard_s2h(pl.handle, 8, odd, good2, None) == basp.BASP_ERR_ALIGN
    assert L.basp_reshard_s2h(pl.handle, 8, good, good, None) == basp.BASP_ERR_ALIAS
    assert L.basp_reshard_s2h(pl.handle, 7, good, good2, None) == basp.BASP_ERR_INVALID
    assert L.basp_attn_fwd(pl.handle, good, good, good, None, None, 0.0, None) == basp.BASP_ERR_NULL
    assert L.basp_attn_fwd(pl.handle, good, good, good, good, None, 0.0, None) == basp.BASP_ERR_ALIAS
    assert L.basp_layer_fwd(pl.handle, good, good, good, good2, None, ctypes.c_void_p(0x1000), 16, 0.0, None) \
        == basp.BASP_ERR_WORKSPACE
    pl2 = basp.basp_plan_create(4, 2, 1000, 8, 8, 64)    # T = 500 is not a multiple of 128: tiles would straddle ranks
    assert L.basp_layer_fwd_fused(pl2.handle, good, good, good, good2, None, 0.0, None) == basp.BASP_ERR_UNSUPPORTED
    pl3 = basp.basp_plan_create(4, 2, 1024, 8, 8, 40)    # head dim the kernels do not implement (not a multiple of 16)
    assert L.basp_attn_fwd(pl3.handle, good, good, good, good2, None, 0.0, None) == basp.BASP_ERR_UNSUPPORTED
    assert basp.lib.basp_strerror(-7).decode().startswith("a bounded wait")


def test_scale_checks_need_no_gpu(basp):
    """A negative, infinite or NaN softmax scale is refused by every call that takes one, before anything is launched."""
    import ctypes
    pl = basp.basp_plan_create(4, 2, 1024, 8, 8, 64)
    a = (ctypes.c_void_p * 4)(*[0x10000 * (i + 1) for i in range(4)])
    b = (ctypes.c_void_p * 4)(*[0x10000000 + 0x100000 * (i + 1) for i in range(4)])
    ws = ctypes.c_void_p(0x40000000)
    L = basp.lib
    for bad in (-0.125, float("inf"), float("nan")):
        assert L.basp_attn_fwd(pl.handle, a, a, a, b, None, bad, None) == basp.BASP_ERR_INVALID
        assert L.basp_layer_fwd_fused(pl.handle, a, a, a, b, None, bad, None) == basp.BASP_ERR_INVALID
        assert L.basp_layer_fwd(pl.handle, a, a, a, b, None, ws, 1 << 30, bad, None) == basp.BASP_ERR_INVALID
        assert L.basp_attn_bwd(pl.handle, a, a, a, a, a, a, b, b, b, ws, 1 << 30, bad, None) == basp.BASP_ERR_INVALID
        assert L.basp_layer_bwd(pl.handle, a, a, a, a, a, a, b, b, b, ws, 1 << 30, bad, None) == basp.BASP_ERR_INVALID


def test_uneven_head_shards_may_touch_the_next_buffer(basp):
    """Where the group size does not divide the sequence length a head-sharded shard (whole sequences of S tokens) is
    smaller than K full chunks: a buffer that starts right behind the last head shard does not overlap it."""
    import ctypes
    import torch
    if torch.cuda.is_available():
        pytest.skip("made-up addresses: with a device present the accepted call would launch on them "
                    "(tests/test_gpu_uneven.py covers the case on real buffers)")
    N, S, H, D = 4, 1021, 8, 64                           # one group of 4: T = 256, last rank 253 tokens
    pl = basp.basp_plan_create(N, 1, S, H, H, D)
    assert (pl.K, pl.T, pl.T_last) == (4, 256, 253)
    head_bytes = S * (H // 4) * D * 2                     # exact size of a head shard
    seq_bytes = 256 * H * D * 2
    heads = [0x20000000 + r * head_bytes for r in range(N)]
    behind = heads[-1] + head_bytes                       # the first byte after the last head shard (16-byte aligned)
    assert behind % 16 == 0
    seqs = [behind + r * seq_bytes for r in range(N)]
    P = lambda xs: (ctypes.c_void_p * N)(*xs)
    rc = basp.lib.basp_reshard_h2s(pl.handle, H, P(heads), P(seqs), None)
    assert rc in (basp.BASP_OK, basp.BASP_ERR_CUDA)       # passed the overlap check (no GPU here: the launch may fail)
    seqs[0] -= 16                                         # one vector into the last head shard: a real overlap
    assert basp.lib.basp_reshard_h2s(pl.handle, H, P(heads), P(seqs), None) == basp.BASP_ERR_ALIAS
