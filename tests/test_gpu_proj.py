"""Parity of the projection GEMMs (QKV with its three-way split write, output projection) with the fp64 oracle.
Weights ~ N(0, 1/hidden) so that outputs are O(1); tolerance: |err| <= 2e-2 + 2^-8 |ref| (bf16 result of an fp32 sum)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import make_plan, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def close(got, ref, what):
    err = np.abs(got - ref)
    bound = 2e-2 + 2.0 ** -8 * np.abs(ref)
    assert (err <= bound).all() and err.mean() < 4e-3, f"{what}: max {err.max():.3e} mean {err.mean():.3e}"


@pytest.mark.parametrize("w,hidden", [
    (synth.Workload("p1", N=2, B=2, S=256, Hq=4, Hkv=2, D=128), 512),
    (synth.Workload("p2", N=4, B=2, S=400, Hq=8, Hkv=4, D=64), 320),        # ragged row tiles (T = 200)
    (synth.Workload("p3", N=8, B=2, S=512, Hq=32, Hkv=8, D=128), 1024),
    (synth.Workload("p4", N=2, B=4, S=192, Hq=4, Hkv=2, D=128, G=1), 256),   # several sequences per rank
])
def test_qkv_and_out_projection(basp, w, hidden):
    pl = make_plan(basp, w)
    op = oracle.plan(w.N, w.B, w.S, w.G)
    g = torch.Generator().manual_seed(w.S + hidden)
    M = op.Bl * op.T
    x = [synth.randn_bf16(g, (M, hidden)) for _ in range(w.N)]
    n_qkv = (w.Hq + 2 * w.Hkv) * w.D
    w_qkv = (torch.randn((n_qkv, hidden), generator=g) / hidden ** 0.5).to(torch.bfloat16)
    w_o = (torch.randn((hidden, w.Hq * w.D), generator=g) / (w.Hq * w.D) ** 0.5).to(torch.bfloat16)
    dx = [t.cuda() for t in x]
    dq = [torch.full((op.Bl, op.T, w.Hq, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    dk = [torch.full((op.Bl, op.T, w.Hkv, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    dv = [torch.full_like(t, float("nan")) for t in dk]
    basp.basp_clear_status()
    basp.basp_qkv_proj(pl, hidden, dx, w_qkv.cuda(), dq, dk, dv)
    basp.basp_get_status()
    for r in range(w.N):
        ref = oracle.linear(synth.bits(x[r]), synth.bits(w_qkv))
        nq, nk = w.Hq * w.D, w.Hkv * w.D
        close(dq[r].float().cpu().numpy().astype(np.float64).reshape(M, nq), ref[:, :nq], "Q")
        close(dk[r].float().cpu().numpy().astype(np.float64).reshape(M, nk), ref[:, nq:nq + nk], "K")
        close(dv[r].float().cpu().numpy().astype(np.float64).reshape(M, nk), ref[:, nq + nk:], "V")
    if hidden % 256 == 0:
        dy = [torch.full((M, hidden), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
        basp.basp_out_proj(pl, hidden, dq, w_o.cuda(), dy)
        basp.basp_get_status()
        for r in range(w.N):
            ref = oracle.linear(synth.bits(dq[r].cpu().reshape(M, -1)), synth.bits(w_o))
            close(dy[r].float().cpu().numpy().astype(np.float64), ref, "Y")


def test_projection_argument_checks(basp):
    w = synth.Workload("pe", N=2, B=2, S=256, Hq=4, Hkv=2, D=128)
    pl = make_plan(basp, w)
    x = [torch.zeros((128, 100), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    q = [torch.zeros((1, 128, 4, 128), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    kv = [torch.zeros((1, 128, 2, 128), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    wq = torch.zeros((1024, 100), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(basp.BaspError) as e:
        basp.basp_qkv_proj(pl, 100, x, wq, q, kv, kv)          # hidden not a multiple of 64
    assert e.value.code == basp.BASP_ERR_UNSUPPORTED


@pytest.mark.parametrize("w,hidden", [
    (synth.Workload("r1", N=2, B=2, S=256, Hq=4, Hkv=2, D=128), 512),
    (synth.Workload("r2", N=4, B=1, S=800, Hq=8, Hkv=4, D=64), 320),        # one group of 4: positions run across ranks; T = 200
    (synth.Workload("r3", N=2, B=4, S=192, Hq=4, Hkv=2, D=128, G=1), 256),   # several sequences per rank: positions restart
])
def test_qkv_projection_with_rope(basp, w, hidden):
    """Rotary embedding in the GEMM epilogue against the oracle: rotation of the fp64 product, position of a row =
    local rank * T + its token index inside the sequence chunk."""
    pl = make_plan(basp, w)
    op = oracle.plan(w.N, w.B, w.S, w.G)
    g = torch.Generator().manual_seed(7 * w.S + hidden)
    M = op.Bl * op.T
    x = [synth.randn_bf16(g, (M, hidden)) for _ in range(w.N)]
    w_qkv = (torch.randn(((w.Hq + 2 * w.Hkv) * w.D, hidden), generator=g) / hidden ** 0.5).to(torch.bfloat16)
    cos, sin = synth.rope_tables(w.S, w.D)
    dq = [torch.full((op.Bl, op.T, w.Hq, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    dk = [torch.full((op.Bl, op.T, w.Hkv, w.D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    dv = [torch.full_like(t, float("nan")) for t in dk]
    basp.basp_clear_status()
    basp.basp_qkv_proj_rope(pl, hidden, [t.cuda() for t in x], w_qkv.cuda(), cos.t().contiguous().cuda(),
                            sin.t().contiguous().cuda(), dq, dk, dv)      # the call takes the tables feature-major
    basp.basp_get_status()
    for r in range(w.N):
        info = op.rank_info(r, w.Hq, w.Hkv)
        pos = np.tile(np.arange(info["token_begin"], info["token_end"]), op.Bl)      # row bl*T + t -> position l*T + t
        q, k, v = oracle.qkv_proj_rope(synth.bits(x[r]), synth.bits(w_qkv), w.Hq, w.Hkv, w.D, cos.numpy(), sin.numpy(), pos)
        f = lambda t, h: t.float().cpu().numpy().astype(np.float64).reshape(M, h, w.D)
        close(f(dq[r], w.Hq), q, "Q"); close(f(dk[r], w.Hkv), k, "K"); close(f(dv[r], w.Hkv), v, "V")


def test_rope_argument_checks(basp):
    w = synth.Workload("re", N=2, B=2, S=256, Hq=4, Hkv=2, D=96)
    pl = make_plan(basp, w)
    x = [torch.zeros((128, 256), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    wq = torch.zeros(((4 + 4) * 96, 256), dtype=torch.bfloat16, device="cuda")
    q = [torch.zeros((1, 128, 4, 96), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    k = [torch.zeros((1, 128, 2, 96), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    v = [torch.zeros_like(t) for t in k]
    cs = torch.zeros((48, 256), dtype=torch.float32, device="cuda")
    with pytest.raises(basp.BaspError) as e:
        basp.basp_qkv_proj_rope(pl, 256, x, wq, cs, cs, q, k, v)
    assert e.value.code == basp.BASP_ERR_UNSUPPORTED          # D = 96: a head's halves are not whole 32-column chunks
