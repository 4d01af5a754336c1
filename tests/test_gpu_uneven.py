"""A sequence length that the group size does not divide (chunk = ceil(S/K), the last rank of each group short, its
sequence-sharded shards compact): the exchanges bit for bit against the oracle's uneven maps, the forward layer
(three launches; one fused kernel where the chunk is a multiple of the tile), the backward layer, the projections
with and without the rotary embedding, and the host-buffer entry."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [
    synth.Workload("k2_s1001", N=4, B=2, S=1001, Hq=4, Hkv=2, D=64),              # 501 + 500
    synth.Workload("k4_s1021_fusable", N=4, B=1, S=1021, Hq=8, Hkv=4, D=128),     # 256 * 3 + 253
    synth.Workload("ulysses_two_seqs", N=8, B=2, S=1019, Hq=8, Hkv=8, D=64, G=1),  # K=8: 128 * 7 + 123, two sequences
    synth.Workload("two_per_group", N=8, B=4, S=509, Hq=8, Hkv=4, D=32, G=2),     # K=4: 128 * 3 + 125
    synth.Workload("replicated_kv", N=4, B=1, S=1022, Hq=8, Hkv=2, D=128),        # K=4 > Hkv: 256 * 3 + 254
    synth.Workload("tiny_tail", N=4, B=1, S=385, Hq=4, Hkv=4, D=64),              # 97 * 3 + 94
]


def dev_list(arrays):
    return [synth.from_bits(np.ascontiguousarray(a)).cuda() for a in arrays]


def bits_list(tensors):
    return [synth.bits(t.cpu()) for t in tensors]


def f64_list(tensors):
    return [t.float().cpu().numpy().astype(np.float64) for t in tensors]


def cat(arrays):
    return np.concatenate([np.asarray(a).ravel() for a in arrays])


def setup(basp, w, causal=True, with_dO=False):
    ts = synth.make_qkv(w, seed=3, with_dO=with_dO)
    X = [synth.bits(t) for t in ts]
    op = oracle.plan_uneven(w.N, w.B, w.S, w.G)
    pl = make_plan(basp, w, causal=causal)
    assert (pl.K, pl.T, pl.T_last) == (op.K, op.T, op.T_last) and op.uneven
    return X, op, pl


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_exchanges_bit_exact(basp, w):
    (Xq, Xk, Xv), op, pl = setup(basp, w)
    seqs = [oracle.partition_uneven(X, op) for X in (Xq, Xk, Xv)]
    dq, dk, dv = (dev_list(s) for s in seqs)
    mk = lambda h: [torch.full((pl.Bl, pl.S, h, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    hq, hk, hv = mk(pl.Hq_l), mk(pl.Hkv_l), mk(pl.Hkv_l)
    basp.basp_reshard_qkv_s2h(pl, dq, dk, dv, hq, hk, hv)
    for got, seq in ((hq, seqs[0]), (hk, seqs[1]), (hv, seqs[2])):
        assert np.array_equal(np.stack(bits_list(got)), oracle.s2h_uneven(seq, op))
    back = [torch.full_like(t, float("nan")) for t in dq]
    basp.basp_reshard_h2s(pl, w.Hq, hq, back)
    assert all(np.array_equal(a, b) for a, b in zip(bits_list(back), seqs[0]))
    if pl.Hkv_l * pl.K == w.Hkv:                    # not replicated: the way back is the inverse for K and V too
        backk = [torch.full_like(t, float("nan")) for t in dk]
        basp.basp_reshard_h2s(pl, w.Hkv, hk, backk)
        assert all(np.array_equal(a, b) for a, b in zip(bits_list(backk), seqs[1]))


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_forward_layer(basp, w, causal):
    (Xq, Xk, Xv), op, pl = setup(basp, w, causal)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op, causal=causal)
    dq, dk, dv = (dev_list(oracle.partition_uneven(X, op)) for X in (Xq, Xk, Xv))
    variants = ["three_launch"] + (["fused"] if pl.T % 128 == 0 and pl.Bl == 1 else [])
    for variant in variants:
        o = [torch.full_like(t, float("nan")) for t in dq]
        lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
        basp.basp_clear_status()
        if variant == "fused":
            basp.basp_layer_fwd_fused(pl, dq, dk, dv, o, lse)
        else:
            ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
            basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse)
        basp.basp_get_status()
        assert [tuple(t.shape) for t in o] == [a.shape for a in ref["o_seq"]]
        assert_attn_close(cat(f64_list(o)), cat(ref["o_seq"]), f"{w.name} {variant} causal={causal}")
        got_lse = np.stack([t.cpu().numpy().astype(np.float64) for t in lse])
        assert np.abs(got_lse - ref["lse_head"]).max() < 2e-3, (w.name, variant)


@pytest.mark.parametrize("w", [CASES[0], CASES[2], CASES[3]], ids=lambda w: w.name)
def test_fused_refuses_what_its_tile_addressing_cannot_serve(basp, w):
    """A chunk that is no multiple of the tile; a short last shard that holds several sequences."""
    (Xq, Xk, Xv), op, pl = setup(basp, w)
    assert pl.T % 128 != 0 or pl.Bl > 1
    dq, dk, dv = (dev_list(oracle.partition_uneven(X, op)) for X in (Xq, Xk, Xv))
    with pytest.raises(basp.BaspError) as e:
        basp.basp_layer_fwd_fused(pl, dq, dk, dv, [torch.zeros_like(t) for t in dq])
    assert e.value.code == basp.BASP_ERR_UNSUPPORTED


@pytest.mark.parametrize("w", [CASES[1], CASES[3], CASES[4], CASES[5]], ids=lambda w: w.name)
def test_backward_layer(basp, w):
    (Xq, Xk, Xv, Xdo), op, pl = setup(basp, w, with_dO=True)
    ref = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op)
    dq, dk, dv, ddo = (dev_list(oracle.partition_uneven(X, op)) for X in (Xq, Xk, Xv, Xdo))
    o = [torch.zeros_like(t) for t in dq]
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse)
    qh, kh, vh, oh = basp.basp_layer_workspace_shards(pl, ws)
    for variant in ("from_head_shards", "from_sequence_shards"):
        gq, gk, gv = ([torch.full_like(t, float("nan")) for t in x] for x in (dq, dk, dv))
        if variant == "from_head_shards":
            ws2 = torch.empty(basp.basp_layer_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
            basp.basp_layer_bwd(pl, qh, kh, vh, oh, lse, ddo, gq, gk, gv, ws2)
        else:
            ws2 = torch.empty(basp.basp_layer_bwd_seq_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
            basp.basp_layer_bwd_seq(pl, dq, dk, dv, o, lse, ddo, gq, gk, gv, ws2)
        basp.basp_get_status()
        for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
            r, g = cat(ref[name + "_seq"]), cat(f64_list(got))
            err = np.abs(g - r)
            assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (variant, name, float(err.max()))
            assert err.mean() <= 2e-3 * max(1.0, float(np.abs(r).mean())), (variant, name)


@pytest.mark.parametrize("rope", [False, True])
@pytest.mark.parametrize("w", [CASES[1], CASES[2]], ids=lambda w: w.name)
def test_projections(basp, w, rope):
    hidden = 256
    pl = make_plan(basp, w)
    op = oracle.plan_uneven(w.N, w.B, w.S, w.G)
    g = torch.Generator().manual_seed(w.S)
    rows = [op.Bl * (op.token_range(r % op.K)[1] - op.token_range(r % op.K)[0]) for r in range(w.N)]
    x = [synth.randn_bf16(g, (m, hidden)) for m in rows]
    w_qkv = (torch.randn(((w.Hq + 2 * w.Hkv) * w.D, hidden), generator=g) / hidden ** 0.5).to(torch.bfloat16)
    cos, sin = synth.rope_tables(w.S, w.D)
    mk = lambda h: [torch.full((op.Bl, m // op.Bl, h, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for m in rows]
    dq, dk, dv = mk(w.Hq), mk(w.Hkv), mk(w.Hkv)
    basp.basp_clear_status()
    if rope:
        basp.basp_qkv_proj_rope(pl, hidden, [t.cuda() for t in x], w_qkv.cuda(), cos.t().contiguous().cuda(),
                                sin.t().contiguous().cuda(), dq, dk, dv)
    else:
        basp.basp_qkv_proj(pl, hidden, [t.cuda() for t in x], w_qkv.cuda(), dq, dk, dv)
    basp.basp_get_status()
    for r in range(w.N):
        t0, t1 = op.token_range(r % op.K)
        pos = np.tile(np.arange(t0, t1), op.Bl)
        if rope:
            q, k, v = oracle.qkv_proj_rope(synth.bits(x[r]), synth.bits(w_qkv), w.Hq, w.Hkv, w.D, cos.numpy(), sin.numpy(), pos)
        else:
            Y = oracle.linear(synth.bits(x[r]), synth.bits(w_qkv))
            q, k, v = (Y[:, :w.Hq * w.D], Y[:, w.Hq * w.D:(w.Hq + w.Hkv) * w.D], Y[:, (w.Hq + w.Hkv) * w.D:])
        for got, want, name in ((dq[r], q, "Q"), (dk[r], k, "K"), (dv[r], v, "V")):
            gf = got.float().cpu().numpy().astype(np.float64).reshape(rows[r], -1)
            wf = np.asarray(want).reshape(rows[r], -1)
            err = np.abs(gf - wf)
            assert not np.isnan(gf).any() and (err <= 1e-2 + 2.0 ** -8 * np.abs(wf)).all(), (name, r, float(err.max()))


def test_host_buffer_entry(basp):
    w = CASES[1]
    (Xq, Xk, Xv), op, pl = setup(basp, w)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    pin = lambda arrays: [synth.from_bits(np.ascontiguousarray(a)).pin_memory() for a in arrays]
    hq, hk, hv = (pin(oracle.partition_uneven(X, op)) for X in (Xq, Xk, Xv))
    ho = [torch.full_like(t, float("nan")).pin_memory() for t in hq]
    arena = torch.empty(basp.basp_host_arena_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd_host(pl, hq, hk, hv, ho, arena)
    basp.basp_get_status()
    assert_attn_close(cat(f64_list(ho)), cat(ref["o_seq"]), "host entry, uneven")


def test_sequence_shard_right_behind_the_last_head_shard(basp):
    """One arena with the head shards packed back to back at their exact size (whole sequences of S tokens, smaller than
    K chunks of T tokens) and the sequence shards directly behind them: nothing overlaps, so both exchanges must accept
    the layout, and they must be bit-exact on it."""
    w = CASES[1]                                            # one group of 4, S = 1021: T = 256, last rank 253 tokens
    pl = make_plan(basp, w)
    op = oracle.plan_uneven(w.N, w.B, w.S)
    Xq = synth.random_bits((w.B, w.S, w.Hq, w.D), seed=5)
    seq_ref = oracle.partition_uneven(Xq, op)
    head_ref = oracle.s2h_uneven(seq_ref, op)
    head_elems = w.S * (w.Hq // pl.K) * w.D
    seq_elems = [a.size for a in seq_ref]
    arena = torch.zeros(w.N * head_elems + sum(seq_elems), dtype=torch.bfloat16, device="cuda")
    heads = [arena[r * head_elems:(r + 1) * head_elems] for r in range(w.N)]
    seqs, off = [], w.N * head_elems
    for n in seq_elems:
        seqs.append(arena[off:off + n])
        off += n
    assert seqs[0].data_ptr() == heads[-1].data_ptr() + head_elems * 2
    for t, a in zip(seqs, seq_ref):
        t.copy_(synth.from_bits(a).reshape(-1))
    basp.basp_reshard_s2h(pl, w.Hq, seqs, heads)
    torch.cuda.synchronize()
    assert np.array_equal(np.stack([synth.bits(h.cpu()).reshape(head_ref[r].shape) for r, h in enumerate(heads)]), head_ref)
    for t in seqs:
        t.zero_()
    basp.basp_reshard_h2s(pl, w.Hq, heads, seqs)
    torch.cuda.synchronize()
    for t, a in zip(seqs, seq_ref):
        assert np.array_equal(synth.bits(t.cpu()).reshape(a.shape), a)
