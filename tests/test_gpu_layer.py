"""The whole layer through the C ABI: three-launch path and fused kernel against the oracle's
layer, BASP = Ulysses = unpartitioned on the GPU, the host-buffer entry, and full-size sampled parity."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, oracle_inputs, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def gpu_layer(basp, w, Xq, Xk, Xv, op, fused):
    pl = make_plan(basp, w)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    do = [torch.zeros_like(t) for t in dq]
    basp.basp_clear_status()
    if fused:
        basp.basp_layer_fwd_fused(pl, dq, dk, dv, do)
    else:
        ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
        basp.basp_layer_fwd(pl, dq, dk, dv, do, ws)
    basp.basp_get_status()
    return do


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("w", [
    synth.WORKLOADS["tiny"],
    synth.shrink(synth.WORKLOADS["llama3_8b_32k"], 256),
    synth.shrink(synth.WORKLOADS["sweep_b1"], 128),
    synth.shrink(synth.WORKLOADS["sweep_b8"], 256),
    synth.shrink(synth.WORKLOADS["qwen25_7b_64k"], 128),
    synth.Workload("head_dim_96", N=4, B=2, S=512, Hq=8, Hkv=4, D=96),
    # Table I's "Standard Ulysses (SP = N/B)" row with N = 8, B = 2: two replicas of 4 GPUs, each on its own micro-batch
    # of 2 sequences (4 sequences in flight, B^2 S / N tokens per GPU)
    synth.Workload("table1_sp_n_over_b", N=8, B=4, S=1024, Hq=8, Hkv=4, D=128, G=2),
    # more sequences than ranks: the data-parallel fallback (one rank per group, two whole sequences each)
    synth.Workload("data_parallel_fallback", N=4, B=8, S=512, Hq=4, Hkv=2, D=64),
], ids=lambda w: w.name)
def test_layer_matches_oracle(basp, w, fused):
    Xq, Xk, Xv, op = oracle_inputs(w)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    do = gpu_layer(basp, w, Xq, Xk, Xv, op, fused)
    assert_attn_close(to_f64(do), ref["o_seq"], f"{w.name} fused={fused}")


def test_tiny_basp_equals_ulysses_equals_unpartitioned(basp):
    """The tiny layer (N=4, S=1024, 8 heads of 64): b=2 (two groups of 2) vs b-agnostic Ulysses (one group of 4) vs no partition.
    The per-row tile schedule does not depend on the grouping, so the GPU outputs agree bit for bit."""
    w = synth.WORKLOADS["tiny"]
    Xq, Xk, Xv, op = oracle_inputs(w)
    full, _ = oracle.attn_fwd(Xq, Xk, Xv)
    outs = {}
    for name, ww in (("basp", w), ("ulysses", synth.Workload("u", 4, 2, 1024, 8, 8, 64, G=1)),
                     ("single", synth.Workload("s", 2, 2, 1024, 8, 8, 64))):
        o = oracle.plan(ww.N, ww.B, ww.S, ww.G)
        for fused in (False, True):
            do = gpu_layer(basp, ww, Xq, Xk, Xv, o, fused)
            bits = np.stack([synth.bits(t.cpu()) for t in do])
            outs[(name, fused)] = oracle.gather(bits, o)
            assert_attn_close(oracle.bf16_bits_to_f64(outs[(name, fused)]), full, f"{name} fused={fused}")
    first = outs[("basp", False)]
    for key, val in outs.items():
        assert np.array_equal(val, first), key


@pytest.mark.parametrize("w,causal", [
    (synth.shrink(synth.WORKLOADS["llama3_8b_32k"], 128), True),                          # T = 128: one launch per group
    (synth.Workload("pieces_two_groups", N=8, B=2, S=4096, Hq=8, Hkv=4, D=128), True),    # T = 1024: several pieces per shard
    (synth.Workload("pieces_d64_two_seqs", N=4, B=4, S=2048, Hq=4, Hkv=2, D=64, G=2), True),   # D = 64, two sequences per group
    (synth.Workload("pieces_unmasked", N=4, B=2, S=1024, Hq=4, Hkv=4, D=64), False),      # every piece needs all of K and V
], ids=lambda x: getattr(x, "name", str(x)))
def test_host_buffer_entry(basp, w, causal):
    Xq, Xk, Xv, op = oracle_inputs(w, seed=2)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op, causal=causal)
    pl = make_plan(basp, w, causal=causal)
    host = [[synth.from_bits(a[r]).pin_memory() for r in range(w.N)] for a in (ref["q_seq"], ref["k_seq"], ref["v_seq"])]
    out = [torch.zeros_like(t).pin_memory() for t in host[0]]
    arena = torch.empty(basp.basp_host_arena_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd_host(pl, host[0], host[1], host[2], out, arena)
    basp.basp_get_status()
    assert_attn_close(to_f64(out), ref["o_seq"], "host entry")


@pytest.mark.parametrize("name", ["llama3_8b_32k", "sweep_b1"])
def test_host_buffer_entry_full_size_sampled_rows(basp, name):
    """The host-buffer entry at full size, in both orders of its pipeline (Llama-3-8B shape at 32K with b = 2: the link is the longer side; 64K
    at b = 1: the GPU is), on sampled output rows."""
    w = synth.WORKLOADS[name]
    q, k, v = synth.make_qkv(w, seed=0)
    pl = make_plan(basp, w)
    T, K = pl.T, pl.K
    cut = lambda x: [x[r // K: r // K + 1, (r % K) * T:(r % K + 1) * T].contiguous().pin_memory() for r in range(w.N)]
    hq, hk, hv = cut(q), cut(k), cut(v)
    ho = [torch.full_like(t, float("nan")).pin_memory() for t in hq]
    arena = torch.empty(basp.basp_host_arena_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd_host(pl, hq, hk, hv, ho, arena)
    basp.basp_get_status()
    assert not any(torch.isnan(t.float()).any() for t in ho)                 # every row of every shard came back
    rng = np.random.default_rng(1)
    cand = [0, 255, 256, 2047, 2048, T - 1, T, 2 * T - 1, 2 * T, w.S - 2049, w.S - 2048, w.S - 1]
    rows = [(b, h, i) for b in range(w.B) for h in (0, w.Hq - 1) for i in cand]
    rows += [(int(rng.integers(w.B)), int(rng.integers(w.Hq)), int(rng.integers(w.S))) for _ in range(40)]
    rows = np.array(rows, dtype=np.int32)
    ref, _ = oracle.attn_fwd_rows(synth.bits(q), synth.bits(k), synth.bits(v), rows)
    got = np.stack([ho[b * K + i // T][0, i % T, h].float().numpy().astype(np.float64) for b, h, i in rows])
    assert_attn_close(got, ref, f"{name} host entry")


def sampled_rows(S, T, B, Hq, seed=0):
    """Rows checked per (sequence, query head) at full size: rows 0..255 (both sides of the first tile boundaries
    included), both sides of every shard boundary l*T, the last 256 rows and 64 seeded random rows."""
    rng = np.random.default_rng(seed)
    out = []
    for b in range(B):
        for h in range(Hq):
            pos = set(range(min(256, S))) | set(range(max(0, S - 256), S))
            for edge in range(T, S, T):
                pos |= {edge - 1, edge}
            pos |= {int(x) for x in rng.integers(0, S, 64)}
            out += [(b, h, i) for i in sorted(pos)]
    return np.array(out, dtype=np.int32)


@pytest.mark.parametrize("name", ["llama3_8b_32k", "sweep_b1", "sweep_b4", "sweep_b8", "qwen25_7b_64k"])
def test_full_size_sampled_rows(basp, name):
    """The Llama-3-8B shape at 32K with two groups of four, the same shape with 65536 tokens over 1, 4 and 8 sequences,
    and the Qwen2.5-7B shape at 64K, at full size through the launches the benchmark times: per (sequence, query head)
    rows 0..255, both sides of every shard boundary, the last 256 rows and 64 random rows against oracle rows."""
    w = synth.WORKLOADS[name]
    q, k, v = synth.make_qkv(w, seed=0)
    pl = make_plan(basp, w)
    T, K = pl.T, pl.K

    def shards(x):   # Algorithm 2 by slicing
        return [x[r // K: r // K + 1, (r % K) * T:(r % K + 1) * T].contiguous().cuda() for r in range(w.N)]

    dq, dk, dv = shards(q), shards(k), shards(v)
    rows = sampled_rows(w.S, T, w.B, w.Hq)
    ref, _ = oracle.attn_fwd_rows(synth.bits(q), synth.bits(k), synth.bits(v), rows)
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    for fused in (False, True):
        do = [torch.zeros_like(t) for t in dq]
        basp.basp_clear_status()
        if fused:
            basp.basp_layer_fwd_fused(pl, dq, dk, dv, do)
        else:
            basp.basp_layer_fwd(pl, dq, dk, dv, do, ws)
        basp.basp_get_status()
        flat = torch.stack(do).reshape(w.B, w.S, w.Hq, w.D)          # the shards in rank order are the global tensor
        ix = torch.from_numpy(rows.astype(np.int64)).cuda()
        got = flat[ix[:, 0], ix[:, 2], ix[:, 1]].float().cpu().numpy().astype(np.float64)
        assert_attn_close(got, ref, f"{name} fused={fused}")


@pytest.mark.parametrize("scale", [0.0, 0.05])
def test_four_sequences_per_group_and_custom_scale_forward_and_backward(basp, scale):
    """Bl = 4 sequences per group (K = 2) with a caller-supplied softmax scale, through the forward layer (both forms)
    and the backward layer; scale = 0 selects 1/sqrt(D)."""
    w = synth.Workload("bl4", N=4, B=8, S=512, Hq=4, Hkv=2, D=128, G=2)
    q, k, v, do_ = synth.make_qkv(w, seed=8, with_dO=True)
    Xq, Xk, Xv, Xdo = (synth.bits(t) for t in (q, k, v, do_))
    op = oracle.plan(w.N, w.B, w.S, w.G)
    osc = None if scale == 0.0 else scale
    ref = oracle.layer_fwd(Xq, Xk, Xv, op, scale=osc)
    refb = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op, scale=osc)
    pl = make_plan(basp, w)
    assert pl.Bl == 4 and pl.K == 2
    dq, dk, dv, ddo = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv, Xdo))
    lse = [torch.zeros((pl.Bl, pl.Hq_l, pl.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    for fused in (True, False):
        o = [torch.full_like(t, float("nan")) for t in dq]
        if fused:
            basp.basp_layer_fwd_fused(pl, dq, dk, dv, o, lse, softmax_scale=scale)
        else:
            basp.basp_layer_fwd(pl, dq, dk, dv, o, ws, lse_shards=lse, softmax_scale=scale)
        basp.basp_get_status()
        assert_attn_close(to_f64(o), ref["o_seq"], f"bl4 fused={fused} scale={scale}")
    qh, kh, vh, oh = basp.basp_layer_workspace_shards(pl, ws)
    gq, gk, gv = ([torch.full_like(t, float("nan")) for t in x] for x in (dq, dk, dv))
    ws2 = torch.empty(basp.basp_layer_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_layer_bwd(pl, qh, kh, vh, oh, lse, ddo, gq, gk, gv, ws2, softmax_scale=scale)
    basp.basp_get_status()
    for name, got in (("dq", gq), ("dk", gk), ("dv", gv)):
        r = refb[name + "_seq"]
        err = np.abs(to_f64(got) - r)
        assert (err <= 2e-2 + 2.0 ** -8 * np.abs(r)).all(), (name, float(err.max()))
