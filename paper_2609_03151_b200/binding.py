"""ctypes binding of libbasp.so: same names as include/basp.h, argument marshalling only.

Importing this module loads the CUDA library and fails loudly if it has not been built
(``python -m paper_2609_03151_b200.build``).  There is no CPU fallback of any call.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int, c_longlong, c_size_t, c_void_p

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbasp.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_03151_b200.build` "
                      "(there is no fallback path)")
lib = ctypes.CDLL(_LIB_PATH)

BASP_OK = 0
BASP_ERR_INVALID, BASP_ERR_UNSUPPORTED, BASP_ERR_NULL, BASP_ERR_ALIGN = -1, -2, -3, -4
BASP_ERR_ALIAS, BASP_ERR_CUDA, BASP_ERR_TIMEOUT, BASP_ERR_WORKSPACE = -5, -6, -7, -8
BASP_MAX_RANKS = 32

EXPORTS = [
    "basp_plan_create", "basp_plan_destroy", "basp_plan_get_info", "basp_plan_get_rank",
    "basp_plan_group_ranks", "basp_reshard_s2h", "basp_reshard_h2s", "basp_reshard_qkv_s2h",
    "basp_attn_fwd", "basp_layer_fwd", "basp_workspace_bytes", "basp_layer_fwd_fused",
    "basp_layer_fwd_host", "basp_host_arena_bytes", "basp_layer_fwd_static",
    "basp_layer_workspace_shards", "basp_attn_bwd", "basp_attn_bwd_workspace_bytes", "basp_reshard_grads_h2s",
    "basp_layer_bwd", "basp_layer_bwd_workspace_bytes", "basp_get_status", "basp_clear_status",
    "basp_strerror", "basp_last_cuda_error", "basp_launch_count", "basp_selftest_wait_timeout", "basp_qkv_proj", "basp_out_proj",
    "basp_reshard_qkv_s2h_ranks", "basp_reshard_h2s_ranks", "basp_attn_fwd_ranks", "basp_layer_fwd_fused_ranks",
    "basp_qkv_proj_rope", "basp_layer_bwd_seq", "basp_layer_bwd_seq_workspace_bytes", "basp_plan_create_parts", "basp_attn_bwd_deterministic",
]


class basp_config(Structure):
    _fields_ = [(n, c_int) for n in ("n_ranks", "micro_batch", "num_groups", "seq_len", "n_q_heads",
                                     "n_kv_heads", "head_dim", "dtype", "causal")]


class basp_plan_info(Structure):
    _fields_ = [(n, c_int) for n in ("group_size", "num_groups", "seqs_per_group", "tokens_per_rank",
                                     "tokens_last_rank", "q_heads_per_rank", "kv_heads_per_rank")] + \
               [(n, c_size_t) for n in ("q_shard_elems", "kv_shard_elems", "lse_shard_elems")]


class basp_rank_info(Structure):
    _fields_ = [(n, c_int) for n in ("group", "local_rank", "seq_begin", "seq_end", "token_begin", "token_end",
                                     "q_head_begin", "q_head_end", "kv_head_begin", "kv_head_end")]


_PP = POINTER(c_void_p)
lib.basp_plan_create.argtypes = [POINTER(basp_config), POINTER(c_void_p)]
lib.basp_plan_destroy.argtypes = [c_void_p]
lib.basp_plan_get_info.argtypes = [c_void_p, POINTER(basp_plan_info)]
lib.basp_plan_get_rank.argtypes = [c_void_p, c_int, POINTER(basp_rank_info)]
lib.basp_plan_group_ranks.argtypes = [c_void_p, c_int, POINTER(c_int)]
lib.basp_reshard_s2h.argtypes = [c_void_p, c_int, _PP, _PP, c_void_p]
lib.basp_reshard_h2s.argtypes = [c_void_p, c_int, _PP, _PP, c_void_p]
lib.basp_reshard_qkv_s2h.argtypes = [c_void_p] + [_PP] * 6 + [c_void_p]
lib.basp_attn_fwd.argtypes = [c_void_p] + [_PP] * 5 + [c_float, c_void_p]
lib.basp_layer_fwd.argtypes = [c_void_p] + [_PP] * 5 + [c_void_p, c_size_t, c_float, c_void_p]
lib.basp_layer_fwd_fused.argtypes = [c_void_p] + [_PP] * 5 + [c_float, c_void_p]
lib.basp_reshard_qkv_s2h_ranks.argtypes = [c_void_p] + [_PP] * 6 + [c_int, c_int, c_void_p]
lib.basp_reshard_h2s_ranks.argtypes = [c_void_p, c_int, _PP, _PP, c_int, c_int, c_void_p]
lib.basp_attn_fwd_ranks.argtypes = [c_void_p] + [_PP] * 5 + [c_float, c_int, c_int, c_void_p]
lib.basp_layer_fwd_fused_ranks.argtypes = [c_void_p] + [_PP] * 5 + [c_float, c_int, c_int, c_void_p]
lib.basp_layer_fwd_static.argtypes = [c_void_p] + [_PP] * 5 + [c_float, c_void_p]
lib.basp_layer_fwd_host.argtypes = [c_void_p] + [_PP] * 4 + [c_void_p, c_size_t, c_float, c_void_p]
lib.basp_layer_workspace_shards.argtypes = [c_void_p, c_void_p] + [_PP] * 4
lib.basp_attn_bwd.argtypes = [c_void_p] + [_PP] * 9 + [c_void_p, c_size_t, c_float, c_void_p]
lib.basp_attn_bwd_deterministic.argtypes = lib.basp_attn_bwd.argtypes
lib.basp_reshard_grads_h2s.argtypes = [c_void_p] + [_PP] * 6 + [c_void_p]
lib.basp_layer_bwd.argtypes = [c_void_p] + [_PP] * 9 + [c_void_p, c_size_t, c_float, c_void_p]
lib.basp_layer_bwd_seq.argtypes = [c_void_p] + [_PP] * 9 + [c_void_p, c_size_t, c_float, c_void_p]
for _n in ("basp_attn_bwd_workspace_bytes", "basp_layer_bwd_workspace_bytes", "basp_layer_bwd_seq_workspace_bytes"):
    getattr(lib, _n).argtypes = [c_void_p]
    getattr(lib, _n).restype = c_size_t
lib.basp_workspace_bytes.argtypes = [c_void_p]
lib.basp_workspace_bytes.restype = c_size_t
lib.basp_host_arena_bytes.argtypes = [c_void_p]
lib.basp_host_arena_bytes.restype = c_size_t
lib.basp_get_status.argtypes = [c_void_p, POINTER(c_int)]
lib.basp_clear_status.argtypes = [c_void_p]
lib.basp_selftest_wait_timeout.argtypes = [ctypes.c_uint, c_void_p]
lib.basp_qkv_proj.argtypes = [c_void_p, c_int, _PP, c_void_p, _PP, _PP, _PP, c_void_p]
lib.basp_out_proj.argtypes = [c_void_p, c_int, _PP, c_void_p, _PP, c_void_p]
lib.basp_qkv_proj_rope.argtypes = [c_void_p, c_int, _PP, c_void_p, c_void_p, c_void_p, _PP, _PP, _PP, c_void_p]
lib.basp_strerror.argtypes = [c_int]
lib.basp_strerror.restype = c_char_p
lib.basp_last_cuda_error.restype = c_char_p
lib.basp_launch_count.restype = c_longlong


class BaspError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib.basp_strerror(code).decode()
        cuda = lib.basp_last_cuda_error().decode() if code == BASP_ERR_CUDA else ""
        super().__init__(f"{where}: {msg} ({code}) {cuda}".strip())


def _check(code: int, where: str):
    if code != BASP_OK:
        raise BaspError(code, where)


def _ptrs(tensors, n: int):
    """Host array of n raw addresses from a list of tensors, raw integer addresses (peer memory mapped into this
    process) or None entries (-> NULL)."""
    if tensors is None:
        return None
    if len(tensors) != n:
        raise ValueError(f"expected {n} shards, got {len(tensors)}")
    return (c_void_p * n)(*[None if t is None else (t.data_ptr() if hasattr(t, "data_ptr") else int(t))
                            for t in tensors])


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class Plan:
    """Owner of a basp_plan*; the N, K, ... attributes are what basp_plan_get_info reports."""

    def __init__(self, handle: int, cfg: basp_config):
        self.handle = c_void_p(handle)
        self.cfg = cfg
        info = basp_plan_info()
        _check(lib.basp_plan_get_info(self.handle, byref(info)), "basp_plan_get_info")
        self.info = info
        self.N = cfg.n_ranks
        self.K, self.G, self.Bl, self.T = info.group_size, info.num_groups, info.seqs_per_group, info.tokens_per_rank
        self.S, self.Hq, self.Hkv, self.D = cfg.seq_len, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        self.Hq_l, self.Hkv_l = info.q_heads_per_rank, info.kv_heads_per_rank
        self.T_last = info.tokens_last_rank

    def rank_tokens(self, r: int) -> int:
        """Tokens per sequence in rank r's sequence-sharded shards (the last rank of a group is short when the group
        size does not divide the sequence length)."""
        return self.T_last if r % self.K == self.K - 1 else self.T

    def __del__(self, _destroy=lib.basp_plan_destroy):
        h, self.handle = getattr(self, "handle", None), None
        if h:
            _destroy(h)


def basp_plan_create(n_ranks, micro_batch, seq_len, n_q_heads, n_kv_heads, head_dim, num_groups=0,
                     causal=True, dtype=0) -> Plan:
    cfg = basp_config(n_ranks, micro_batch, num_groups, seq_len, n_q_heads, n_kv_heads, head_dim, dtype, int(causal))
    out = c_void_p()
    _check(lib.basp_plan_create(byref(cfg), byref(out)), "basp_plan_create")
    return Plan(out.value, cfg)


class basp_plan_part(Structure):
    _fields_ = [("plan", c_void_p)] + [(n, c_int) for n in ("rank_begin", "n_ranks", "seq_begin", "n_seqs", "group_size")]


lib.basp_plan_create_parts.argtypes = [POINTER(basp_config), POINTER(basp_plan_part), POINTER(c_int)]


class PlanPart:
    """One uniform part of an unequal group formation: `plan` serves global ranks [rank_begin, rank_begin + n_ranks)
    and sequences [seq_begin, seq_begin + n_seqs); `shards(x)` cuts a per-rank list down to the part's ranks."""

    def __init__(self, plan: Plan, rank_begin: int, n_ranks: int, seq_begin: int, n_seqs: int, group_size: int):
        self.plan, self.rank_begin, self.n_ranks = plan, rank_begin, n_ranks
        self.seq_begin, self.n_seqs, self.group_size = seq_begin, n_seqs, group_size

    def shards(self, per_rank):
        return list(per_rank[self.rank_begin:self.rank_begin + self.n_ranks])


def basp_plan_create_parts(n_ranks, micro_batch, seq_len, n_q_heads, n_kv_heads, head_dim, causal=True, dtype=0):
    """Group formation for any micro_batch <= n_ranks (groups of ceil and floor(N/B) ranks): a list of one or two
    PlanPart.  Every call of the library is then made per part with part.plan and part.shards(...)."""
    cfg = basp_config(n_ranks, micro_batch, 0, seq_len, n_q_heads, n_kv_heads, head_dim, dtype, int(causal))
    arr = (basp_plan_part * 2)()
    n = c_int(0)
    _check(lib.basp_plan_create_parts(byref(cfg), arr, byref(n)), "basp_plan_create_parts")
    out = []
    for i in range(n.value):
        c = basp_config(arr[i].n_ranks, arr[i].n_seqs, 0, seq_len, n_q_heads, n_kv_heads, head_dim, dtype, int(causal))
        out.append(PlanPart(Plan(arr[i].plan, c), arr[i].rank_begin, arr[i].n_ranks, arr[i].seq_begin, arr[i].n_seqs,
                            arr[i].group_size))
    return out


def basp_plan_get_rank(plan: Plan, rank: int) -> dict:
    ri = basp_rank_info()
    _check(lib.basp_plan_get_rank(plan.handle, rank, byref(ri)), "basp_plan_get_rank")
    return {n: getattr(ri, n) for n, _ in basp_rank_info._fields_}


def basp_plan_group_ranks(plan: Plan, group: int) -> list[int]:
    out = (c_int * plan.K)()
    _check(lib.basp_plan_group_ranks(plan.handle, group, out), "basp_plan_group_ranks")
    return list(out)


def basp_reshard_s2h(plan, n_heads, seq_shards, head_shards, stream=None):
    _check(lib.basp_reshard_s2h(plan.handle, n_heads, _ptrs(seq_shards, plan.N), _ptrs(head_shards, plan.N),
                                _stream(stream)), "basp_reshard_s2h")


def basp_reshard_h2s(plan, n_heads, head_shards, seq_shards, stream=None):
    _check(lib.basp_reshard_h2s(plan.handle, n_heads, _ptrs(head_shards, plan.N), _ptrs(seq_shards, plan.N),
                                _stream(stream)), "basp_reshard_h2s")


def basp_reshard_qkv_s2h(plan, q_seq, k_seq, v_seq, q_head, k_head, v_head, stream=None):
    n = plan.N
    _check(lib.basp_reshard_qkv_s2h(plan.handle, _ptrs(q_seq, n), _ptrs(k_seq, n), _ptrs(v_seq, n),
                                    _ptrs(q_head, n), _ptrs(k_head, n), _ptrs(v_head, n), _stream(stream)),
           "basp_reshard_qkv_s2h")


def basp_attn_fwd(plan, q_head, k_head, v_head, o_head, lse_shards=None, softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_attn_fwd(plan.handle, _ptrs(q_head, n), _ptrs(k_head, n), _ptrs(v_head, n), _ptrs(o_head, n),
                             _ptrs(lse_shards, n), softmax_scale, _stream(stream)), "basp_attn_fwd")


def basp_workspace_bytes(plan) -> int:
    return int(lib.basp_workspace_bytes(plan.handle))


def basp_host_arena_bytes(plan) -> int:
    return int(lib.basp_host_arena_bytes(plan.handle))


def basp_layer_fwd(plan, q_seq, k_seq, v_seq, o_seq, workspace, lse_shards=None, softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_layer_fwd(plan.handle, _ptrs(q_seq, n), _ptrs(k_seq, n), _ptrs(v_seq, n), _ptrs(o_seq, n),
                              _ptrs(lse_shards, n), c_void_p(workspace.data_ptr()),
                              workspace.numel() * workspace.element_size(), softmax_scale, _stream(stream)),
           "basp_layer_fwd")


def basp_layer_fwd_fused(plan, q_seq, k_seq, v_seq, o_seq, lse_shards=None, softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_layer_fwd_fused(plan.handle, _ptrs(q_seq, n), _ptrs(k_seq, n), _ptrs(v_seq, n),
                                    _ptrs(o_seq, n), _ptrs(lse_shards, n), softmax_scale, _stream(stream)),
           "basp_layer_fwd_fused")


# ---- one physical GPU's share (ranks [rank_begin, rank_begin + rank_count)); shard lists may hold tensors, raw
# addresses of peer memory, or None for shards the call does not touch
def basp_reshard_qkv_s2h_ranks(plan, q_seq, k_seq, v_seq, q_head, k_head, v_head, rank_begin, rank_count, stream=None):
    n = plan.N
    _check(lib.basp_reshard_qkv_s2h_ranks(plan.handle, _ptrs(q_seq, n), _ptrs(k_seq, n), _ptrs(v_seq, n),
                                          _ptrs(q_head, n), _ptrs(k_head, n), _ptrs(v_head, n), rank_begin,
                                          rank_count, _stream(stream)), "basp_reshard_qkv_s2h_ranks")


def basp_reshard_h2s_ranks(plan, n_heads, head_shards, seq_shards, rank_begin, rank_count, stream=None):
    n = plan.N
    _check(lib.basp_reshard_h2s_ranks(plan.handle, n_heads, _ptrs(head_shards, n), _ptrs(seq_shards, n), rank_begin,
                                      rank_count, _stream(stream)), "basp_reshard_h2s_ranks")


def basp_attn_fwd_ranks(plan, q_head, k_head, v_head, o_head, rank_begin, rank_count, lse_shards=None,
                        softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_attn_fwd_ranks(plan.handle, _ptrs(q_head, n), _ptrs(k_head, n), _ptrs(v_head, n),
                                   _ptrs(o_head, n), _ptrs(lse_shards, n), softmax_scale, rank_begin, rank_count,
                                   _stream(stream)), "basp_attn_fwd_ranks")


def basp_layer_fwd_fused_ranks(plan, q_seq, k_seq, v_seq, o_seq, rank_begin, rank_count, lse_shards=None,
                               softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_layer_fwd_fused_ranks(plan.handle, _ptrs(q_seq, n), _ptrs(k_seq, n), _ptrs(v_seq, n),
                                          _ptrs(o_seq, n), _ptrs(lse_shards, n), softmax_scale, rank_begin,
                                          rank_count, _stream(stream)), "basp_layer_fwd_fused_ranks")


BASP_STATIC_SCRATCH_BYTES = 16 << 20


def basp_layer_fwd_static(plan, q_seq, k_seq, v_seq, o_seq, lse_shards=None, softmax_scale=0.0, stream=None):
    """The three-launch layer for callers that can neither allocate device memory nor pass a
    workspace: scratch is a fixed 16 MiB array inside the library (plans that need more are refused).
    Calls on one device share that array, so do not let two of them overlap on the GPU."""
    n = plan.N
    _check(lib.basp_layer_fwd_static(plan.handle, _ptrs(q_seq, n), _ptrs(k_seq, n), _ptrs(v_seq, n),
                                     _ptrs(o_seq, n), _ptrs(lse_shards, n), softmax_scale, _stream(stream)),
           "basp_layer_fwd_static")


def basp_layer_fwd_host(plan, q_seq_host, k_seq_host, v_seq_host, o_seq_host, device_arena, softmax_scale=0.0,
                        stream=None):
    n = plan.N
    _check(lib.basp_layer_fwd_host(plan.handle, _ptrs(q_seq_host, n), _ptrs(k_seq_host, n), _ptrs(v_seq_host, n),
                                   _ptrs(o_seq_host, n), c_void_p(device_arena.data_ptr()),
                                   device_arena.numel() * device_arena.element_size(), softmax_scale,
                                   _stream(stream)), "basp_layer_fwd_host")


def basp_layer_workspace_shards(plan, workspace):
    """Addresses (ints) of the head-sharded Q, K, V, O that basp_layer_fwd left in `workspace`:
    four lists of n_ranks device addresses."""
    n = plan.N
    arrs = [(c_void_p * n)() for _ in range(4)]
    _check(lib.basp_layer_workspace_shards(plan.handle, c_void_p(workspace.data_ptr()), *arrs),
           "basp_layer_workspace_shards")
    return [[int(a[i]) for i in range(n)] for a in arrs]


class _Addr:
    """A raw device address standing in for a tensor in the marshalling helpers."""

    def __init__(self, addr):
        self.addr = addr

    def data_ptr(self):
        return self.addr


def as_shards(addresses):
    return [_Addr(a) for a in addresses]


def basp_attn_bwd_workspace_bytes(plan) -> int:
    return int(lib.basp_attn_bwd_workspace_bytes(plan.handle))


def basp_layer_bwd_workspace_bytes(plan) -> int:
    return int(lib.basp_layer_bwd_workspace_bytes(plan.handle))


def basp_attn_bwd(plan, q_head, k_head, v_head, o_head, do_head, lse_shards, dq_head, dk_head, dv_head, workspace,
                  softmax_scale=0.0, stream=None, deterministic=False):
    n = plan.N
    fn = lib.basp_attn_bwd_deterministic if deterministic else lib.basp_attn_bwd
    _check(fn(plan.handle, *[_ptrs(t, n) for t in (q_head, k_head, v_head, o_head, do_head, lse_shards,
                                                                  dq_head, dk_head, dv_head)],
                             c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size(),
                             softmax_scale, _stream(stream)), "basp_attn_bwd")


def basp_reshard_grads_h2s(plan, dq_head, dk_head, dv_head, dq_seq, dk_seq, dv_seq, stream=None):
    n = plan.N
    _check(lib.basp_reshard_grads_h2s(plan.handle, *[_ptrs(t, n) for t in (dq_head, dk_head, dv_head, dq_seq, dk_seq,
                                                                           dv_seq)], _stream(stream)),
           "basp_reshard_grads_h2s")


def basp_layer_bwd_seq_workspace_bytes(plan) -> int:
    return int(lib.basp_layer_bwd_seq_workspace_bytes(plan.handle))


def basp_layer_bwd_seq(plan, q_seq, k_seq, v_seq, o_seq, lse_shards, do_seq, dq_seq, dk_seq, dv_seq, workspace,
                       softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_layer_bwd_seq(plan.handle, *[_ptrs(t, n) for t in (q_seq, k_seq, v_seq, o_seq, lse_shards, do_seq,
                                                                       dq_seq, dk_seq, dv_seq)],
                                  c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size(),
                                  softmax_scale, _stream(stream)), "basp_layer_bwd_seq")


def basp_layer_bwd(plan, q_head, k_head, v_head, o_head, lse_shards, do_seq, dq_seq, dk_seq, dv_seq, workspace,
                   softmax_scale=0.0, stream=None):
    n = plan.N
    _check(lib.basp_layer_bwd(plan.handle, *[_ptrs(t, n) for t in (q_head, k_head, v_head, o_head, lse_shards, do_seq,
                                                                   dq_seq, dk_seq, dv_seq)],
                              c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size(),
                              softmax_scale, _stream(stream)), "basp_layer_bwd")


def basp_get_status(stream=None, raise_on_timeout=True):
    out = (c_int * 4)()
    rc = lib.basp_get_status(_stream(stream), out)
    if rc == BASP_ERR_TIMEOUT and not raise_on_timeout:
        return list(out)
    _check(rc, f"basp_get_status {list(out)}")
    return list(out)


def basp_clear_status(stream=None):
    _check(lib.basp_clear_status(_stream(stream)), "basp_clear_status")


def basp_qkv_proj(plan, hidden, x_seq, w_qkv, q_seq, k_seq, v_seq, stream=None):
    n = plan.N
    _check(lib.basp_qkv_proj(plan.handle, int(hidden), _ptrs(x_seq, n), c_void_p(w_qkv.data_ptr()), _ptrs(q_seq, n),
                             _ptrs(k_seq, n), _ptrs(v_seq, n), _stream(stream)), "basp_qkv_proj")


def basp_qkv_proj_rope(plan, hidden, x_seq, w_qkv, rope_cos, rope_sin, q_seq, k_seq, v_seq, stream=None):
    n = plan.N
    _check(lib.basp_qkv_proj_rope(plan.handle, int(hidden), _ptrs(x_seq, n), c_void_p(w_qkv.data_ptr()),
                                  c_void_p(rope_cos.data_ptr()), c_void_p(rope_sin.data_ptr()), _ptrs(q_seq, n),
                                  _ptrs(k_seq, n), _ptrs(v_seq, n), _stream(stream)), "basp_qkv_proj_rope")


def basp_out_proj(plan, hidden, o_seq, w_o, y_seq, stream=None):
    n = plan.N
    _check(lib.basp_out_proj(plan.handle, int(hidden), _ptrs(o_seq, n), c_void_p(w_o.data_ptr()), _ptrs(y_seq, n),
                             _stream(stream)), "basp_out_proj")


def basp_selftest_wait_timeout(limit_us: int, stream=None):
    _check(lib.basp_selftest_wait_timeout(int(limit_us), _stream(stream)), "basp_selftest_wait_timeout")


def basp_launch_count() -> int:
    return int(lib.basp_launch_count())
