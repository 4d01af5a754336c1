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


def _worker_span(rank, world, port, out_dir):
    """A group that spans both processes (K = 4 ranks on 2 'GPUs'): address tables and the push exchange."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    pdist.init(backend="gloo")
    wl = synth.Workload("g", N=4, B=1, S=64, Hq=4, Hkv=4, D=8)
    Xq, _, _ = (synth.bits(t) for t in synth.make_qkv(wl, seed=1))
    pl = oracle.plan(wl.N, wl.B, wl.S)
    mine = pdist.ranks_of_gpu(wl.N, world, rank)
    assert len(mine) == 2 and pdist.gpu_of_rank(wl.N, world, mine.start) == rank
    # every process publishes where its buffer is "mapped": the tables built from the gathered bases must agree
    shard_bytes = pl.Bl * pl.T * wl.Hq * wl.D * 2
    bases = [None] * world
    dist.all_gather_object(bases, 0x10000000 * (rank + 1))
    table = pdist.shard_addresses(bases, wl.N, shard_bytes, offset=256)
    assert table == [0x10000000 * (r // 2 + 1) + 256 + (r % 2) * shard_bytes for r in range(wl.N)]
    tables = [None] * world
    dist.all_gather_object(tables, table)
    assert tables[0] == tables[1]
    # push model of the s2h exchange: every process scatters only ITS ranks' sequence shards; the pieces are disjoint
    # and their union is the whole exchange
    seq = oracle.partition(Xq, pl)
    masked = seq.copy()
    for r in range(wl.N):
        if r not in mine:
            masked[r] = 0
    part = oracle.s2h(masked, pl).astype(np.int64)
    total = torch.from_numpy(part.copy())
    dist.all_reduce(total, op=dist.ReduceOp.SUM)
    full = oracle.s2h(seq, pl).astype(np.int64)
    assert np.array_equal(total.numpy(), full)
    nz = torch.from_numpy((part != 0).astype(np.int64))
    dist.all_reduce(nz, op=dist.ReduceOp.SUM)
    assert int(nz.max()) <= 1                      # no element written by two processes
    pdist.finalize()
    open(os.path.join(out_dir, f"span{rank}"), "w").write("ok")


def test_two_process_group_spanning_exchange(tmp_path):
    port = _free_port()
    mp.spawn(_worker_span, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert all((tmp_path / f"span{r}").exists() for r in range(2))


def test_ranks_of_gpu_and_addresses():
    assert list(pdist.ranks_of_gpu(8, 2, 1)) == [4, 5, 6, 7]
    assert list(pdist.ranks_of_gpu(8, 8, 3)) == [3]
    assert [pdist.gpu_of_rank(8, 4, r) for r in range(8)] == [0, 0, 1, 1, 2, 2, 3, 3]
    for bad in ((8, 3, 0), (8, 2, 2)):
        try:
            pdist.ranks_of_gpu(*bad)
            assert False
        except ValueError:
            pass
    assert pdist.shard_addresses([1000 * 16, 5000 * 16], 4, 32) == [16000, 16032, 80000, 80032]
    try:
        pdist.shard_addresses([0, 0], 4, 24)
        assert False
    except ValueError:
        pass


def _cpu_allocator(world, gpu, base=0x7000_0000_0000):
    """Stand-in for symmetric memory: a host buffer and invented base addresses, one per 'GPU' (1 TiB apart)."""
    def alloc(nbytes, group):
        buf = torch.zeros(nbytes, dtype=torch.uint8)
        return buf, [base + g * (1 << 40) for g in range(world)]
    return alloc


def test_symmetric_shards_layout_on_cpu():
    """Layout arithmetic of the per-GPU shard buffer: tensors back to back (256-byte aligned blocks), this GPU's ranks
    consecutive inside each block, the same offsets on every GPU."""
    n_ranks, world, gpu = 8, 4, 2
    sizes = {"q": 4096, "k": 1040, "v": 1040, "o": 4096}          # 1040: a block that needs padding to 256
    sh = pdist.SymmetricShards(n_ranks, sizes, allocator=_cpu_allocator(world, gpu), world=world, gpu=gpu)
    assert list(sh.local) == [4, 5]
    offs = {"q": 0, "k": 8192, "v": 8192 + 2304, "o": 8192 + 2 * 2304}
    assert sh.nbytes == offs["o"] + 8192
    base = lambda g: 0x7000_0000_0000 + g * (1 << 40)
    for name, sz in sizes.items():
        assert sh.addresses(name) == [base(r // 2) + offs[name] + (r % 2) * sz for r in range(n_ranks)]
        assert all(a % 16 == 0 for a in sh.addresses(name))
    sh.local_shard("k", 5)[:] = 7
    assert int(sh.buffer[offs["k"] + 1040: offs["k"] + 2080].sum()) == 7 * 1040 and int(sh.buffer.sum()) == 7 * 1040
    for bad in (3, 6):
        try:
            sh.local_shard("k", bad)
            assert False
        except ValueError:
            pass
    assert sh.remote_fraction(8) == 0.75 and sh.remote_fraction(2) == 0.0 and sh.remote_fraction(4) == 0.5
    try:
        pdist.SymmetricShards(n_ranks, {"q": 24}, allocator=_cpu_allocator(world, gpu), world=world, gpu=gpu)
        assert False
    except ValueError:
        pass


class _RecordingStream:
    def __init__(self, log, name):
        self.log, self.name = log, name

    def synchronize(self):
        self.log.append(("sync", self.name))


def _worker_multi_gpu_order(rank, world, port, out_dir):
    """Host ordering of the group-spanning layer (synchronise the launch stream, barrier, launch, synchronise the same
    stream, barrier) with the oracle standing in for the kernel: each process produces only its ranks' output shards
    and the union is the whole layer."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    pdist.init(backend="gloo")
    wl = synth.Workload("g", N=4, B=1, S=64, Hq=4, Hkv=2, D=8)             # one group of 4 ranks over 2 'GPUs'
    Xq, Xk, Xv = (synth.bits(t) for t in synth.make_qkv(wl, seed=3))
    pl = oracle.plan(wl.N, wl.B, wl.S)
    ref = oracle.layer_fwd(Xq, Xk, Xv, pl)
    shard_bytes = {"q": pl.T * wl.Hq * wl.D * 2, "k": pl.T * wl.Hkv * wl.D * 2, "v": pl.T * wl.Hkv * wl.D * 2,
                   "o": pl.T * wl.Hq * wl.D * 2}
    sh = pdist.SymmetricShards(wl.N, shard_bytes, allocator=_cpu_allocator(world, rank), world=world, gpu=rank)
    log, produced = [], {}

    class StubBinding:
        @staticmethod
        def basp_layer_fwd_fused_ranks(plan, q, k, v, o, rank_begin, rank_count, lse_shards=None, softmax_scale=0.0,
                                       stream=None):
            log.append(("launch", stream.name, rank_begin, rank_count))
            assert q == sh.addresses("q") and o == sh.addresses("o") and len(q) == wl.N
            for r in range(rank_begin, rank_begin + rank_count):
                produced[r] = ref["o_seq"][r]

    def barrier():
        log.append(("barrier",))
        dist.barrier()

    side = _RecordingStream(log, "side")
    pdist.layer_fwd_fused_multi_gpu("plan", sh, stream=side, binding=StubBinding, barrier=barrier)
    mine = pdist.ranks_of_gpu(wl.N, world, rank)
    assert log == [("sync", "side"), ("barrier",), ("launch", "side", mine.start, len(mine)), ("sync", "side"), ("barrier",)]
    assert sorted(produced) == list(mine)
    gathered = [None] * world
    dist.all_gather_object(gathered, {r: a for r, a in produced.items()})
    union = {}
    for d in gathered:
        assert not (set(d) & set(union))
        union.update(d)
    got = oracle.gather(np.stack([union[r] for r in range(wl.N)]), pl)
    full, _ = oracle.attn_fwd(Xq, Xk, Xv)
    assert np.array_equal(got, full)
    pdist.finalize()
    open(os.path.join(out_dir, f"order{rank}"), "w").write("ok")


def test_two_process_multi_gpu_layer_ordering(tmp_path):
    port = _free_port()
    mp.spawn(_worker_multi_gpu_order, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert all((tmp_path / f"order{r}").exists() for r in range(2))


def test_three_step_multi_gpu_host_ordering():
    """The three-step group-spanning layer on one process with stand-ins: every step is launched on the given stream and
    followed by a synchronisation of that stream and a barrier (a step reads what other GPUs wrote in the step before),
    with this GPU's rank range and the eight shard tables."""
    n_ranks, world, gpu = 8, 4, 1
    sizes = {n: 4096 for n in ("q", "k", "v", "o", "qh", "kh", "vh", "oh")}
    sh = pdist.SymmetricShards(n_ranks, sizes, allocator=_cpu_allocator(world, gpu), world=world, gpu=gpu)
    log = []

    class Plan:
        Hq = 32

    class StubBinding:
        @staticmethod
        def basp_reshard_qkv_s2h_ranks(plan, q, k, v, qh, kh, vh, r0, cnt, stream=None):
            assert (q, qh, vh) == (sh.addresses("q"), sh.addresses("qh"), sh.addresses("vh"))
            log.append(("s2h", stream.name, r0, cnt))

        @staticmethod
        def basp_attn_fwd_ranks(plan, qh, kh, vh, oh, r0, cnt, lse_shards=None, softmax_scale=0.0, stream=None):
            assert (kh, oh) == (sh.addresses("kh"), sh.addresses("oh"))
            log.append(("attn", stream.name, r0, cnt))

        @staticmethod
        def basp_reshard_h2s_ranks(plan, n_heads, oh, o, r0, cnt, stream=None):
            assert n_heads == 32 and (oh, o) == (sh.addresses("oh"), sh.addresses("o"))
            log.append(("h2s", stream.name, r0, cnt))

    s = _RecordingStream(log, "s")
    pdist.layer_fwd_three_step_multi_gpu(Plan, sh, stream=s, binding=StubBinding, barrier=lambda: log.append(("barrier",)))
    sync_bar = [("sync", "s"), ("barrier",)]
    assert log == sync_bar + [("s2h", "s", 2, 2)] + sync_bar + [("attn", "s", 2, 2)] + sync_bar + [("h2s", "s", 2, 2)] + sync_bar
