"""World-size-2 check (gloo, CPU) of the multi-GPU plumbing: groups are sharded over processes with
no data-path collective, only results/timings are reduced."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_03151_b200 import dist as pdist
from paper_2609_03151_b200 import synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, lr, w = pdist.init(backend="gloo")
    assert (r, w) == (rank, world)
    wl = synth.Workload("g", N=4, B=2, S=64, Hq=4, Hkv=2, D=8)
    Xq, Xk, Xv = (synth.bits(t) for t in synth.make_qkv(wl, seed=0))
    pl = oracle.plan(wl.N, wl.B, wl.S)
    mine = pdist.groups_of_gpu(pl.G, world, rank)
    # each process handles only its groups' sequences (BASP: group g <-> sequence g); no exchange
    sub = oracle.plan(pl.K * len(mine), len(mine), wl.S)
    sl = slice(mine.start * pl.Bl, mine.stop * pl.Bl)
    o = oracle.layer_fwd(Xq[sl], Xk[sl], Xv[sl], sub)["o_global"]
    gathered = [torch.zeros_like(torch.from_numpy(o)) for _ in range(world)]
    dist.all_gather(gathered, torch.from_numpy(o))
    full, _ = oracle.attn_fwd(Xq, Xk, Xv)
    assert np.array_equal(torch.cat(gathered).numpy(), full)
    # timing reduction: slowest rank wins, totals add
    assert pdist.max_over_ranks(10.0 + rank) == 10.0 + world - 1
    assert pdist.sum_over_ranks(1.0) == float(world)
    pdist.barrier()
    pdist.finalize()
    open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")


def test_two_process_group_sharding(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(2))


def test_groups_of_gpu():
    assert list(pdist.groups_of_gpu(8, 2, 1)) == [4, 5, 6, 7]
    assert list(pdist.groups_of_gpu(2, 2, 0)) == [0]
    try:
        pdist.groups_of_gpu(2, 4, 0)
        assert False
    except ValueError:
        pass
