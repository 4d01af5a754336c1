"""Multi-GPU plumbing (one process per GPU, torch.distributed).

The path shards without any data-path collective: BASP groups are independent units (each
group's all-to-all stays inside the group), so different GPUs take different groups -- or,
for weak scaling, different micro-batches -- and only timing is reduced across ranks.

When a group does span GPUs (K > N / world) the exchange is real: every GPU then runs the
`*_ranks` calls for the ranks it hosts over shard tables that point into its peers' memory
(`SymmetricShards`, `layer_fwd_fused_multi_gpu`); the kernels use plain loads/stores and TMA tile
loads on that memory (every thread block fetches its own tile) and never wait for one another.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment (1 process -> 0, 0, 1)."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def init(backend: str | None = None) -> tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        kw = {}
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
            kw["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    """Slowest rank's value (how every multi-GPU time is reported)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def groups_of_gpu(num_groups: int, world: int, rank: int) -> range:
    """Contiguous block of BASP groups that physical GPU `rank` of `world` hosts when ONE
    micro-batch is spread over several GPUs (virtual rank r -> GPU floor(r * world / N), the
    contiguous assignment of the paper's Section IV-A).  Needs world to divide num_groups."""
    if num_groups % world != 0:
        raise ValueError("the number of groups must be a multiple of the number of GPUs "
                         "(a group split across GPUs would need a real all-to-all)")
    per = num_groups // world
    return range(rank * per, (rank + 1) * per)


def ranks_of_gpu(n_ranks: int, world: int, gpu: int) -> range:
    """The contiguous block of virtual ranks that physical GPU `gpu` of `world` hosts (rank r lives on GPU
    floor(r * world / N), Section IV-A).  Needs world to divide n_ranks.  A group (K consecutive ranks) then lies on
    one GPU when K <= N / world and otherwise spans K * world / N GPUs."""
    if world <= 0 or n_ranks % world != 0:
        raise ValueError("the number of GPUs must divide the number of ranks")
    per = n_ranks // world
    if not 0 <= gpu < world:
        raise ValueError("gpu out of range")
    return range(gpu * per, (gpu + 1) * per)


def gpu_of_rank(n_ranks: int, world: int, rank: int) -> int:
    return rank // (n_ranks // world)


def shard_addresses(buffer_ptrs, n_ranks: int, shard_bytes: int, offset: int = 0) -> list[int]:
    """Addresses, valid in THIS process, of every rank's shard of one tensor when each GPU keeps the shards of its
    ranks back to back in one symmetric buffer: `buffer_ptrs[g]` is the address at which GPU g's buffer is mapped
    here (the local allocation for g = this GPU, peer memory otherwise), `offset` the tensor's byte offset inside
    every buffer.  The result is what the `*_ranks` calls take as their shard arrays."""
    world = len(buffer_ptrs)
    per = len(ranks_of_gpu(n_ranks, world, 0))
    if offset % 16 or shard_bytes % 16:
        raise ValueError("shards must stay 16-byte aligned")
    return [int(buffer_ptrs[r // per]) + offset + (r % per) * shard_bytes for r in range(n_ranks)]


def _symmetric_allocator(nbytes: int, group):
    """Default allocator of SymmetricShards: torch symmetric memory (every process maps every GPU's buffer), or, for a
    single process, an ordinary device buffer (there is no peer to map)."""
    dev = torch.device("cuda", torch.cuda.current_device())
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        buf = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        return buf, [buf.data_ptr()]
    import torch.distributed._symmetric_memory as symm_mem
    buf = symm_mem.empty(nbytes, dtype=torch.uint8, device=dev)
    handle = symm_mem.rendezvous(buf, group)
    buf._basp_symm_handle = handle          # keeps the mapping alive as long as the buffer
    return buf, [int(p) for p in handle.buffer_ptrs]


class SymmetricShards:
    """One buffer per GPU holding this GPU's shards of several tensors, mapped into every process of the group (torch
    symmetric memory over NVLink).  `tensors` = {name: shard_bytes}.  With more than one process it needs an
    initialised NCCL process group with one process per GPU.  `allocator(nbytes, group) -> (buffer, base addresses of
    every GPU's buffer as mapped here)` replaces the symmetric-memory allocation (tests of the layout arithmetic run on
    CPU with it); `world` / `gpu` default to the process group's size and this process's rank."""

    def __init__(self, n_ranks: int, tensors: dict, group=None, allocator=None, world: int | None = None,
                 gpu: int | None = None):
        initialised = dist.is_available() and dist.is_initialized()
        self.group = group if group is not None else (dist.group.WORLD if initialised else None)
        self.world = world if world is not None else (dist.get_world_size(self.group) if initialised else 1)
        self.gpu = gpu if gpu is not None else (dist.get_rank(self.group) if initialised else 0)
        self.n_ranks, self.local = n_ranks, ranks_of_gpu(n_ranks, self.world, self.gpu)
        self.layout, off = {}, 0
        for name, shard_bytes in tensors.items():
            if int(shard_bytes) % 16:
                raise ValueError("shards must stay 16-byte aligned")
            self.layout[name] = (off, int(shard_bytes))
            off += (len(self.local) * int(shard_bytes) + 255) // 256 * 256
        self.nbytes = off
        self.buffer, ptrs = (allocator or _symmetric_allocator)(off, self.group)
        self.buffer_ptrs = [int(p) for p in ptrs]
        if len(self.buffer_ptrs) != self.world:
            raise ValueError("the allocator must return one base address per GPU")

    def addresses(self, name: str) -> list[int]:
        off, shard_bytes = self.layout[name]
        return shard_addresses(self.buffer_ptrs, self.n_ranks, shard_bytes, off)

    def local_shard(self, name: str, rank: int) -> torch.Tensor:
        """This GPU's shard of rank `rank` as a byte tensor (view it as bf16 and reshape)."""
        off, shard_bytes = self.layout[name]
        i = rank - self.local.start
        if not 0 <= i < len(self.local):
            raise ValueError("rank lives on another GPU")
        return self.buffer[off + i * shard_bytes: off + (i + 1) * shard_bytes]

    def remote_fraction(self, group_size: int) -> float:
        """Share of a rank's exchange partners that live on another GPU: 1 - min(ranks per GPU, K) / K (what crosses
        NVLink of the bytes that the all-to-alls of a K-rank group move)."""
        return 1.0 - min(len(self.local), group_size) / float(group_size)


def _group_barrier(group):
    if dist.is_available() and dist.is_initialized():
        dist.barrier(group)


def _resolve_stream(stream):
    return stream if stream is not None else torch.cuda.current_stream()


def layer_fwd_fused_multi_gpu(plan, shards: "SymmetricShards", softmax_scale: float = 0.0, stream=None, binding=None,
                              barrier=None, lse=None):
    """The layer when a group spans GPUs: every GPU runs the fused kernel for its own ranks over the group's
    sequence shards (`shards` holds tensors "q", "k", "v", "o").  The kernels never wait for one another: the two
    host barriers order the GPUs (inputs complete before anyone reads them, nobody reuses a buffer before all are
    done), and both follow a synchronisation of the SAME stream the kernel is launched on.  `binding` and `barrier`
    default to the CUDA binding and the process group's barrier (tests pass stand-ins)."""
    if binding is None:
        from . import binding
    barrier = barrier or (lambda: _group_barrier(shards.group))
    s = _resolve_stream(stream)
    s.synchronize()
    barrier()
    binding.basp_layer_fwd_fused_ranks(plan, shards.addresses("q"), shards.addresses("k"), shards.addresses("v"),
                                       shards.addresses("o"), shards.local.start, len(shards.local), lse_shards=lse,
                                       softmax_scale=softmax_scale, stream=s)
    s.synchronize()
    barrier()


def layer_fwd_three_step_multi_gpu(plan, shards: "SymmetricShards", softmax_scale: float = 0.0, stream=None,
                                   binding=None, barrier=None, lse=None):
    """The same layer as three exchanges-and-kernels, for comparison with the fused form: push this GPU's sequence
    shards of Q, K, V into the head shards of its groups' members ("qh", "kh", "vh"; remote members over NVLink),
    attention over its own head shards, pull its sequence shards of O out of the group's "oh".  A host barrier after
    each step: a step reads what other GPUs wrote in the step before."""
    if binding is None:
        from . import binding
    barrier = barrier or (lambda: _group_barrier(shards.group))
    s = _resolve_stream(stream)
    r0, cnt = shards.local.start, len(shards.local)
    a = shards.addresses
    s.synchronize()
    barrier()
    binding.basp_reshard_qkv_s2h_ranks(plan, a("q"), a("k"), a("v"), a("qh"), a("kh"), a("vh"), r0, cnt, stream=s)
    s.synchronize()
    barrier()
    binding.basp_attn_fwd_ranks(plan, a("qh"), a("kh"), a("vh"), a("oh"), r0, cnt, lse_shards=lse,
                                softmax_scale=softmax_scale, stream=s)
    s.synchronize()
    barrier()
    binding.basp_reshard_h2s_ranks(plan, plan.Hq, a("oh"), a("o"), r0, cnt, stream=s)
    s.synchronize()
    barrier()


def finalize():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
