"""Failure detection without a fault: a wait inside a kernel that cannot complete runs into its (short) limit, the kernel
records where, ends by itself, and the context stays usable."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_attn_close, make_plan, oracle_inputs, to_dev, to_f64
from paper_2609_03151_b200 import synth

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_context_survives(basp):
    basp.basp_clear_status()
    assert basp.basp_get_status() == [0, 0, 0, 0]
    basp.basp_selftest_wait_timeout(2000)                  # 2 ms limit, nothing ever arrives
    st = basp.basp_get_status(raise_on_timeout=False)
    assert st[0] == 2 and st[1] == 100 and st[2] == 0
    assert 2000 <= st[3] < 200000, st                       # gave up after the limit, long before the 2 s default
    with pytest.raises(basp.BaspError) as e:
        basp.basp_get_status()
    assert e.value.code == basp.BASP_ERR_TIMEOUT
    basp.basp_clear_status()
    assert basp.basp_get_status() == [0, 0, 0, 0]
    # the context is intact: a real kernel runs and is right
    w = synth.Workload("after", N=1, B=1, S=256, Hq=2, Hkv=1, D=128)
    Xq, Xk, Xv, op = oracle_inputs(w, seed=9)
    ref = oracle.layer_fwd(Xq, Xk, Xv, op)
    pl = make_plan(basp, w)
    dq, dk, dv = (to_dev(oracle.partition(X, op)) for X in (Xq, Xk, Xv))
    do = [torch.zeros_like(t) for t in dq]
    basp.basp_layer_fwd_fused(pl, dq, dk, dv, do)
    basp.basp_get_status()
    assert_attn_close(to_f64(do), ref["o_seq"], "after a timed-out wait")


def test_selftest_rejects_bad_limits(basp):
    for bad in (0, 2_000_000):
        with pytest.raises(basp.BaspError) as e:
            basp.basp_selftest_wait_timeout(bad)
        assert e.value.code == basp.BASP_ERR_INVALID
