"""basp_layer_fwd_static -- the layer for callers that cannot allocate device memory (their heap
belongs to another pool, or they cannot afford cudaMalloc's device-wide synchronisation) and have no
workspace to lend: its scratch is a fixed array inside the library.  Checked here, through the C ABI,
against basp_layer_fwd (bit for bit: the same kernels run) and against the fp64 oracle on two calls in a
row with different inputs, so that whatever the first call left in the shared array cannot leak into
the second; the free device memory must be the same before and after each call.  Collected last on
purpose."""
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
        Xq, Xk, Xv = (synth.bits(t) for t in synth.make_qkv(w, seed))
        ref = oracle.layer_fwd(Xq, Xk, Xv, op)
        q, k, v = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
        want = [torch.zeros_like(t) for t in q]
        got = [torch.full_like(t, float("nan")) for t in q]
        lse_w = [torch.zeros((1, pl.Hq_l, w.S), dtype=torch.float32, device="cuda") for _ in range(w.N)]
        lse_g = [torch.full_like(t, float("nan")) for t in lse_w]
        basp.basp_clear_status()
        basp.basp_layer_fwd(pl, q, k, v, want, ws, lse_w)
        # every buffer of the call exists by now
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        basp.basp_layer_fwd_static(pl, q, k, v, got, lse_g)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        # The very first call on a device is the set-up call: the CUDA runtime loads this library's device image then,
        # which is the moment the GPU commits the fixed array (no allocation call is involved, and it happens once).
        # Every later call must leave the free memory exactly where it was.
        taken = free_before - free_after
        if call == 0:
            assert 0 <= taken <= basp.BASP_STATIC_SCRATCH_BYTES + (4 << 20), f"set-up call took {taken} bytes"
        else:
            assert taken == 0, f"call {call}: free device memory changed by {taken} bytes"
        basp.basp_get_status()
        # the same kernels on the same inputs: the same bits as the entry point with caller workspace ...
        for a, b in zip(got + lse_g, want + lse_w):
            assert torch.equal(a.view(torch.int16 if a.dtype == torch.bfloat16 else torch.int32),
                               b.view(torch.int16 if b.dtype == torch.bfloat16 else torch.int32)), f"call {call}: differs from basp_layer_fwd"
        # ... and within the attention tolerance of the fp64 oracle
        err = np.abs(to_f64(got) - ref["o_seq"])
        assert np.isfinite(err).all(), f"call {call}: output not fully written"
        assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL, (call, err.max(), err.mean())
        assert np.abs(to_f64(lse_g) - ref["lse_head"]).max() <= 2e-3


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
