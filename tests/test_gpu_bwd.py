"""Parity of the attention backward (and the layer backward with its gradient reshards) with the
fp64 oracle, through the C ABI.

Tolerance for gradients (bf16 operands and outputs, bf16 P and dS, fp32 accumulation): element-wise
|err| <= 2e-2 + 2^-8 |ref| and mean-abs error <= 2e-3 * max(1, mean |ref|).  dK/dV sum up to S * Hq/Hkv
terms and exceed magnitude 4, where one bf16 ulp is already 0.016, hence the relative term."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_plan, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def assert_grad_close(got, ref, what):
    err = np.abs(got - ref)
    bound = 2e-2 + 2.0 ** -8 * np.abs(ref)
    worst = float((err - bound).max())
    mean_ok = err.mean() <= 2e-3 * max(1.0, float(np.abs(ref).mean()))
    assert worst <= 0 and mean_ok, f"{what}: max-abs {err.max():.3e} (excess {worst:.3e}) mean-abs {err.mean():.3e} ref mean {np.abs(ref).mean():.3e}"


def inputs(w, seed=0):
    q, k, v, do = synth.make_qkv(w, seed, with_dO=True)
    return [synth.bits(t) for t in (q, k, v, do)], oracle.plan(w.N, w.B, w.S, w.G)


def run_attn_bwd(basp, w, causal=True, seed=0, deterministic=False):
    (Xq, Xk, Xv, Xdo), op = inputs(w, seed)
    pl = make_plan(basp, w, causal)
    qh, kh, vh, doh = (oracle.s2h(oracle.partition(X, op), op) for X in (Xq, Xk, Xv, Xdo))
    dq_, dk_, dv_, ddo = to_dev(qh), to_dev(kh), to_dev(vh), to_dev(doh)
    o = [torch.zeros_like(t) for t in dq_]
    lse = [torch.zeros((op.Bl, w.Hq // op.K, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    basp.basp_clear_status()
    basp.basp_attn_fwd(pl, dq_, dk_, dv_, o, lse)
    gq = [torch.full_like(t, float("nan")) for t in dq_]
    gk = [torch.full_like(t, float("nan")) for t in dk_]
    gv = [torch.full_like(t, float("nan")) for t in dk_]
    ws = torch.empty(basp.basp_attn_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_attn_bwd(pl, dq_, dk_, dv_, o, ddo, lse, gq, gk, gv, ws, deterministic=deterministic)
    basp.basp_get_status()
    if deterministic:      # the two-pass kernels add nothing up across thread blocks: a second run gives the same bits
        again = [[torch.full_like(t, float("nan")) for t in x] for x in (gq, gk, gv)]
        basp.basp_attn_bwd(pl, dq_, dk_, dv_, o, ddo, lse, again[0], again[1], again[2], ws, deterministic=True)
        basp.basp_get_status()
        for first, second in zip((gq, gk, gv), again):
            assert all(torch.equal(a.view(torch.int16), b.view(torch.int16)) for a, b in zip(first, second))
    ref = [oracle.attn_bwd(qh[r], kh[r], vh[r], doh[r], causal=causal) for r in range(w.N)]
    return (to_f64(gq), to_f64(gk), to_f64(gv)), tuple(np.stack([g[n] for g in ref]) for n in ("dQ", "dK", "dV"))


@pytest.mark.parametrize("name,w", [
    ("one_tile", synth.Workload("one_tile", N=1, B=1, S=128, Hq=1, Hkv=1, D=128)),
    ("gqa4", synth.Workload("gqa4", N=1, B=1, S=384, Hq=4, Hkv=1, D=128)),
    ("llama_T128", synth.shrink(synth.WORKLOADS["llama3_8b_128k_train"], 128)),
    ("llama_b2_T256", synth.shrink(synth.WORKLOADS["llama3_8b_32k"], 256)),
    ("ulysses", synth.Workload("ulysses", N=4, B=2, S=512, Hq=8, Hkv=4, D=128, G=1)),
    ("head_dim_64_tiny", synth.WORKLOADS["tiny"]),                                           # N=4, b=2, S=1024, 8 heads of 64
    ("head_dim_96", synth.Workload("d96", N=2, B=1, S=512, Hq=4, Hkv=2, D=96)),             # hidden 3072 / 32 heads
    ("head_dim_80", synth.shrink(synth.WORKLOADS["t2_qwen25_3b"], 128)),                    # hidden 2560 / 32 heads
    ("head_dim_48", synth.Workload("d48", N=2, B=2, S=256, Hq=2, Hkv=1, D=48)),
])
@pytest.mark.parametrize("deterministic", [False, True])
def test_attn_bwd_matches_oracle(basp, name, w, deterministic):
    got, ref = run_attn_bwd(basp, w, deterministic=deterministic)
    for g, r, n in zip(got, ref, ("dQ", "dK", "dV")):
        assert np.isfinite(g).all(), f"{name} {n}: not fully written"
        assert_grad_close(g, r, f"{name} {n}")


@pytest.mark.parametrize("deterministic", [False, True])
@pytest.mark.parametrize("S,causal", [(200, True), (333, True), (1000, True), (77, False), (129, True)])
def test_attn_bwd_ragged_sequence_lengths(basp, S, causal, deterministic):
    """S not a multiple of the 128-row tile, two sequences per rank: what follows a ragged end is the next sequence (its
    rows must neither be read into the gradients nor be written), and the LSE / Delta rows are not 16-byte aligned."""
    w = synth.Workload("ragged_S", N=2, B=4, S=S, Hq=4, Hkv=2, D=128, G=2)
    got, ref = run_attn_bwd(basp, w, causal=causal, seed=S, deterministic=deterministic)
    for g, r, n in zip(got, ref, ("dQ", "dK", "dV")):
        assert np.isfinite(g).all(), f"S={S} {n}: not fully written"
        assert_grad_close(g, r, f"S={S} {n}")


def test_attn_bwd_noncausal(basp):
    w = synth.Workload("nc", N=2, B=2, S=256, Hq=2, Hkv=1, D=128)
    got, ref = run_attn_bwd(basp, w, causal=False, seed=3)
    for g, r, n in zip(got, ref, ("dQ", "dK", "dV")):
        assert_grad_close(g, r, f"noncausal {n}")


def test_layer_bwd_with_gradient_reshards(basp):
    """Forward through basp_layer_fwd, backward through basp_layer_bwd on the saved head-sharded
    activations, gradients back in the sequence-sharded layout; against the oracle's layer backward."""
    w = synth.shrink(synth.WORKLOADS["llama3_8b_128k_train"], 256)
    (Xq, Xk, Xv, Xdo), op = inputs(w, seed=1)
    ref = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op)
    pl = make_plan(basp, w)
    qs, ks, vs, dos = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv, Xdo))
    o = [torch.zeros_like(t) for t in qs]
    lse = [torch.zeros((op.Bl, pl.Hq_l, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_layer_fwd(pl, qs, ks, vs, o, ws, lse)
    qh, kh, vh, oh = (basp.as_shards(a) for a in basp.basp_layer_workspace_shards(pl, ws))
    gq = [torch.full_like(t, float("nan")) for t in qs]
    gk = [torch.full_like(t, float("nan")) for t in ks]
    gv = [torch.full_like(t, float("nan")) for t in ks]
    ws2 = torch.empty(basp.basp_layer_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_layer_bwd(pl, qh, kh, vh, oh, lse, dos, gq, gk, gv, ws2)
    basp.basp_get_status()
    for g, n in ((gq, "dq_seq"), (gk, "dk_seq"), (gv, "dv_seq")):
        assert_grad_close(to_f64(g), ref[n], n)


def test_grads_reshard_single_launch_bit_exact(basp):
    N, B, S, Hq, Hkv, D = 8, 2, 1024, 32, 8, 128
    pl = basp.basp_plan_create(N, B, S, Hq, Hkv, D)
    op = oracle.plan(N, B, S)
    heads = [synth.random_bits((N, 1, S, h // op.K, D), seed=i) for i, h in enumerate((Hq, Hkv, Hkv))]
    want = [oracle.h2s(a, op) for a in heads]
    src = [to_dev(a) for a in heads]
    dst = [[torch.zeros(x.shape[1:], dtype=torch.bfloat16, device="cuda") for _ in range(N)] for x in want]
    n0 = basp.basp_launch_count()
    basp.basp_reshard_grads_h2s(pl, *src, *dst)
    torch.cuda.synchronize()
    assert basp.basp_launch_count() == n0 + 1
    for d, x in zip(dst, want):
        assert np.array_equal(np.stack([synth.bits(t.cpu()) for t in d]), x)


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


def load_golden_columns():
    """The stored dK / dV columns of the 128K training shape and the module that wrote them (tests/golden/)."""
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_dkdv_columns", os.path.join(here, "make_dkdv_columns.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def head_sharded(x, hl, n_ranks):
    """Rank r of the single group owns heads [r*hl, (r+1)*hl) of the whole sequence (what the first exchange delivers)."""
    return [x[:, :, r * hl:(r + 1) * hl].contiguous().cuda() for r in range(n_ranks)]


_column_refs = {}


def column_reference(w, Q, K, V, DO, kvh):
    """Oracle dK / dV of the sampled key positions of one KV head (shared by the kernels tested on the same inputs)."""
    key = (w.name, kvh)
    if key not in _column_refs:
        cols = load_golden_columns().sampled_columns(w.S, -(-w.S // w.K), 0)
        _column_refs[key] = (cols,) + oracle.attn_bwd_dkdv_cols(Q, K, V, DO, b=0, kv=kvh, cols=cols)
    return _column_refs[key]


@pytest.mark.parametrize("name,deterministic", [
    ("llama3_8b_16k_train", False),          # head dimension 128, one-pass kernel
    ("llama3_8b_16k_train", True),           # the two-pass kernels
    ("llama32_1b_16k_train", False),         # head dimension 64: the pipelined 64-wide kernel
])
def test_dkdv_columns_summed_over_many_rows(basp, name, deterministic):
    """dK / dV columns that are sums over up to 16384 query rows x 4 query heads (bf16 P and dS, fp32 accumulation over
    128 query tiles): the first 128 key positions, both sides of tile and shard boundaries, the last positions and 64
    random ones of one KV head, against the oracle's column entry; plus dQ and O on rows spread over the sequence."""
    w = synth.WORKLOADS.get(name) or synth.Workload(name, N=8, B=1, S=16384, Hq=32, Hkv=8, D=64, train=True)
    q, k, v, do = synth.make_qkv(w, seed=0, with_dO=True)
    pl = make_plan(basp, w)
    Hl, Hkl = pl.Hq_l, pl.Hkv_l
    dq_, dk_, dv_, ddo = (head_sharded(x, hl, w.N) for x, hl in ((q, Hl), (k, Hkl), (v, Hkl), (do, Hl)))
    o = [torch.empty_like(t) for t in dq_]
    lse = [torch.empty((1, Hl, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    gq = [torch.full_like(t, float("nan")) for t in dq_]
    gk = [torch.full_like(t, float("nan")) for t in dk_]
    gv = [torch.full_like(t, float("nan")) for t in dk_]
    ws = torch.empty(basp.basp_attn_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_attn_fwd(pl, dq_, dk_, dv_, o, lse)
    basp.basp_attn_bwd(pl, dq_, dk_, dv_, o, ddo, lse, gq, gk, gv, ws, deterministic=deterministic)
    basp.basp_get_status()
    assert not any(torch.isnan(t.float()).any() for t in gq + gk + gv), "gradients not fully written"
    Q, K, V, DO = (synth.bits(t) for t in (q, k, v, do))
    kvh = 5
    cols, ref_dk, ref_dv = column_reference(w, Q, K, V, DO, kvh)
    idx = torch.from_numpy(cols.astype(np.int64)).cuda()
    got_dk = gk[kvh // Hkl][0, idx, kvh % Hkl].float().cpu().numpy().astype(np.float64)
    got_dv = gv[kvh // Hkl][0, idx, kvh % Hkl].float().cpu().numpy().astype(np.float64)
    assert_grad_close(got_dk, ref_dk, f"{name} dK columns")
    assert_grad_close(got_dv, ref_dv, f"{name} dV columns")
    rng = np.random.default_rng(3)
    pos = [0, 127, 128, 2047, 2048, 8191, 8192, w.S - 129, w.S - 1] + [int(x) for x in rng.integers(0, w.S, 23)]
    rows = np.array([(0, h, i) for h in (1, 14, 30) for i in pos], dtype=np.int32)
    ref_dq = oracle.attn_bwd_dq_rows(Q, K, V, DO, rows)
    got_dq = np.stack([gq[h // Hl][0, i, h % Hl].float().cpu().numpy().astype(np.float64) for _, h, i in rows])
    assert_grad_close(got_dq, ref_dq, f"{name} dQ rows")


@pytest.mark.parametrize("S,Hq", [(4096, 8), (4228, 16)])
def test_gang_schedule_of_long_sweeps(basp, S, Hq):
    """Shapes on which the 128-wide kernel takes its gang schedule (few CTAs per (rank, sequence, KV head) against the
    number of key tiles: 64 such streams on 148 SMs, 32 and 34 key tiles): groups of CTAs start every query-head sweep
    together.  The second shape has a ragged last tile, two query heads per KV head and a mirrored last round with a
    gap.  Sampled dQ rows and dK / dV columns of two streams against the oracle."""
    w = synth.Workload(f"gang_{S}", N=8, B=8, S=S, Hq=Hq, Hkv=8, D=128)
    q, k, v, do = synth.make_qkv(w, seed=4, with_dO=True)
    pl = make_plan(basp, w)
    assert pl.K == 1 and pl.Hkv_l == 8
    dq_, dk_, dv_, ddo = ([x[r:r + 1].contiguous().cuda() for r in range(w.N)] for x in (q, k, v, do))   # K = 1: rank r = sequence r
    o = [torch.empty_like(t) for t in dq_]
    lse = [torch.empty((1, Hq, S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    gq = [torch.full_like(t, float("nan")) for t in dq_]
    gk = [torch.full_like(t, float("nan")) for t in dk_]
    gv = [torch.full_like(t, float("nan")) for t in dk_]
    ws = torch.empty(basp.basp_attn_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_attn_fwd(pl, dq_, dk_, dv_, o, lse)
    basp.basp_attn_bwd(pl, dq_, dk_, dv_, o, ddo, lse, gq, gk, gv, ws)
    basp.basp_get_status()
    assert not any(torch.isnan(t.float()).any() for t in gq + gk + gv), "gradients not fully written"
    Q, K, V, DO = (synth.bits(t) for t in (q, k, v, do))
    rng = np.random.default_rng(S)
    cols = np.array(sorted({0, 1, 127, 128, 2047, 2048, S - 129, S - 1} | {int(x) for x in rng.integers(0, S, 40)}), dtype=np.int32)
    for b, kvh in ((0, 0), (5, 7)):
        ref_dk, ref_dv = oracle.attn_bwd_dkdv_cols(Q, K, V, DO, b=b, kv=kvh, cols=cols)
        idx = torch.from_numpy(cols.astype(np.int64)).cuda()
        assert_grad_close(gk[b][0, idx, kvh].float().cpu().numpy().astype(np.float64), ref_dk, f"gang dK ({b},{kvh})")
        assert_grad_close(gv[b][0, idx, kvh].float().cpu().numpy().astype(np.float64), ref_dv, f"gang dV ({b},{kvh})")
    rows = np.array([(b, h, int(i)) for b, h in ((0, 0), (3, Hq - 1), (7, Hq // 2)) for i in cols[::2]], dtype=np.int32)
    ref_dq = oracle.attn_bwd_dq_rows(Q, K, V, DO, rows)
    got_dq = np.stack([gq[b][0, i, h].float().cpu().numpy().astype(np.float64) for b, h, i in rows])
    assert_grad_close(got_dq, ref_dq, "gang dQ rows")


def test_full_size_train_step_sampled(basp):
    """The long-context training shape at full size (Llama-3-8B heads, N=8, b=1, S=131072), forward + backward: O and dQ
    on the sampled row set of every query head, dK / dV of one KV head on 339 key positions spread over the sequence
    (first 128, tile and shard boundaries, last 130, 64 random) against the stored oracle columns (tests/golden/, keyed
    by the CRC-32 of the regenerated inputs), and the last 165 positions of another head against the oracle run here."""
    w = synth.WORKLOADS["llama3_8b_128k_train"]
    q, k, v, do = synth.make_qkv(w, seed=0, with_dO=True)
    pl = make_plan(basp, w)
    Hl, Hkl = pl.Hq_l, pl.Hkv_l
    dq_, dk_, dv_, ddo = (head_sharded(x, hl, w.N) for x, hl in ((q, Hl), (k, Hkl), (v, Hkl), (do, Hl)))
    o = [torch.empty_like(t) for t in dq_]
    lse = [torch.empty((1, Hl, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    gq = [torch.empty_like(t) for t in dq_]
    gk = [torch.empty_like(t) for t in dk_]
    gv = [torch.empty_like(t) for t in dk_]
    ws = torch.empty(basp.basp_attn_bwd_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_clear_status()
    basp.basp_attn_fwd(pl, dq_, dk_, dv_, o, lse)
    basp.basp_attn_bwd(pl, dq_, dk_, dv_, o, ddo, lse, gq, gk, gv, ws)
    basp.basp_get_status()

    Q, K, V, DO = (synth.bits(t) for t in (q, k, v, do))
    # stored columns: the inputs must be the ones the reference was computed from
    mod = load_golden_columns()
    g = np.load(mod.path_for(w.name, 0))
    assert [int(c) for c in g["crc32_q_k_v_do"]] == [mod.crc(a) for a in (Q, K, V, DO)], "inputs differ from the stored reference's"
    assert list(g["shape_N_B_S_Hq_Hkv_D"]) == [w.N, w.B, w.S, w.Hq, w.Hkv, w.D]
    kvh, idx = int(g["kv"]), torch.from_numpy(g["cols"].astype(np.int64)).cuda()
    got_dk = gk[kvh // Hkl][0, idx, kvh % Hkl].float().cpu().numpy().astype(np.float64)
    got_dv = gv[kvh // Hkl][0, idx, kvh % Hkl].float().cpu().numpy().astype(np.float64)
    assert_grad_close(got_dk, g["dK"], "128K dK columns (stored reference)")
    assert_grad_close(got_dv, g["dV"], "128K dV columns (stored reference)")

    rows = sampled_rows(w.S, pl.T, w.B, w.Hq)
    ref_o, _ = oracle.attn_fwd_rows(Q, K, V, rows)
    gather = lambda ts: np.concatenate([
        ts[h // Hl][0, torch.from_numpy(rows[rows[:, 1] == h][:, 2].astype(np.int64)).cuda(), h % Hl].float().cpu().numpy()
        for h in range(w.Hq)]).astype(np.float64)          # rows are ordered by head
    err = np.abs(gather(o) - ref_o)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    dq_rows = rows[(rows[:, 1] % 5 == 3) | (rows[:, 2] < 256) & (rows[:, 1] < 4)]      # 6 heads in full, 4 more on the first rows
    ref_dq = oracle.attn_bwd_dq_rows(Q, K, V, DO, dq_rows)
    got_dq = np.stack([gq[h // Hl][0, i, h % Hl].float().cpu().numpy().astype(np.float64) for _, h, i in dq_rows])
    assert_grad_close(got_dq, ref_dq, "128K dQ rows")
    ncols, kv2 = 165, 6
    ref_dk, ref_dv = oracle.attn_bwd_dkdv_tail(Q, K, V, DO, b=0, kv=kv2, ncols=ncols)
    got_dk = gk[kv2 // Hkl][0, w.S - ncols:, kv2 % Hkl].float().cpu().numpy().astype(np.float64)
    got_dv = gv[kv2 // Hkl][0, w.S - ncols:, kv2 % Hkl].float().cpu().numpy().astype(np.float64)
    assert_grad_close(got_dk, ref_dk, "128K dK tail")
    assert_grad_close(got_dv, ref_dv, "128K dV tail")


@pytest.mark.parametrize("w", [
    synth.shrink(synth.WORKLOADS["llama3_8b_128k_train"], 128),
    synth.Workload("two_groups_rep", N=8, B=2, S=512, Hq=8, Hkv=2, D=64),          # replicated KV heads, D = 64
], ids=lambda w: w.name)
def test_fused_forward_then_backward_from_sequence_shards(basp, w):
    """Forward through the fused kernel (no head-sharded copies exist), backward through basp_layer_bwd_seq, which redoes
    the exchanges; against the oracle's layer backward."""
    (Xq, Xk, Xv, Xdo), op = inputs(w, seed=2)
    ref = oracle.layer_bwd(Xq, Xk, Xv, Xdo, op)
    pl = make_plan(basp, w)
    qs, ks, vs, dos = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv, Xdo))
    o = [torch.zeros_like(t) for t in qs]
    lse = [torch.zeros((op.Bl, pl.Hq_l, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
    basp.basp_clear_status()
    basp.basp_layer_fwd_fused(pl, qs, ks, vs, o, lse)
    gq = [torch.full_like(t, float("nan")) for t in qs]
    gk = [torch.full_like(t, float("nan")) for t in ks]
    gv = [torch.full_like(t, float("nan")) for t in ks]
    ws = torch.empty(basp.basp_layer_bwd_seq_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    basp.basp_layer_bwd_seq(pl, qs, ks, vs, o, lse, dos, gq, gk, gv, ws)
    basp.basp_get_status()
    for g, n in ((gq, "dq_seq"), (gk, "dk_seq"), (gv, "dv_seq")):
        assert_grad_close(to_f64(g), ref[n], n)
