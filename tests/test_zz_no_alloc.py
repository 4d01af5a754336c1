"""basp_layer_fwd_static -- the layer for callers that cannot allocate device memory (their heap
belongs to another pool, or they cannot afford cudaMalloc's device-wide synchronisation) and have no
workspace to lend: its scratch is a fixed array inside the library.  Checked here, through the C ABI,
against basp_layer_fwd on two calls in a row with different inputs, so that whatever the first call
left in the shared array cannot leak into the second.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from helpers import MAX_ABS_TOL, MEAN_ABS_TOL, make_plan, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_scratch_layer_matches_workspace_layer_twice(basp):
    w = synth.WORKLOADS["tiny"]                       # needs 8 MiB of the 16 MiB array
    pl = make_plan(basp, w)
    assert basp.basp_workspace_bytes(pl) <= basp.BASP_STATIC_SCRATCH_BYTES
    op = oracle.plan(w.N, w.B, w.S)
    ws = torch.empty(basp.basp_workspace_bytes(pl), dtype=torch.uint8, device="cuda")
    for call, seed in enumerate((11, 12)):
        q, k, v = (to_dev(oracle.partition(synth.bits(t), op)) for t in synth.make_qkv(w, seed))
        want = [torch.zeros_like(t) for t in q]
        got = [torch.full_like(t, float("nan")) for t in q]
        lse_w = [torch.zeros((1, pl.Hq_l, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
        lse_g = [torch.full_like(t, float("nan")) for t in lse_w]
        basp.basp_clear_status()
        basp.basp_layer_fwd(pl, q, k, v, want, ws, lse_w)
        basp.basp_layer_fwd_static(pl, q, k, v, got, lse_g)
        basp.basp_get_status()
        err = np.abs(to_f64(got) - to_f64(want))
        assert np.isfinite(err).all(), f"call {call}: output not fully written"
        assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL, (call, err.max(), err.mean())
        assert np.abs(to_f64(lse_g) - to_f64(lse_w)).max() <= 2e-3


def test_static_scratch_refuses_large_plans(basp):
    w = synth.shrink(synth.WORKLOADS["llama3_8b_32k"], 512)     # 80 MiB of head-sharded copies
    pl = make_plan(basp, w)
    assert basp.basp_workspace_bytes(pl) > basp.BASP_STATIC_SCRATCH_BYTES
    q = [torch.zeros((1, pl.T, w.Hq, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    kv = [torch.zeros((1, pl.T, w.Hkv, w.D), dtype=torch.bfloat16, device="cuda") for _ in range(w.N)]
    o = [torch.zeros_like(t) for t in q]
    with pytest.raises(basp.BaspError) as e:
        basp.basp_layer_fwd_static(pl, q, kv, kv, o)
    assert e.value.code == basp.BASP_ERR_WORKSPACE
    assert b"static array holds" in basp.lib.basp_last_cuda_error()
