"""The attention layer as a differentiable torch operation (marshalling only: forward = basp_layer_fwd, backward =
basp_layer_bwd, or with fused=True basp_layer_fwd_fused and basp_layer_bwd_seq; nothing is computed in Python).

    o_seq = basp_attention(plan, q_seq, k_seq, v_seq)          # lists of n_ranks sequence-sharded bf16 tensors
    loss(o_seq).backward()                                     # gradients arrive on q_seq, k_seq, v_seq

The forward keeps its workspace (head-sharded Q, K, V, O) and the log-sum-exp for the backward, as a training step of the
paper's setting does between the two passes; the backward needs a second workspace (basp_layer_bwd_workspace_bytes).
Both are allocated through torch's caching allocator on the current device.  With fused=True the forward is the one
fused kernel and keeps nothing but its output and the log-sum-exp (no head-sharded copies live between the passes: for
the 128K-token training shape that is 2.5 GiB less); the backward then redoes the exchanges of Q, K, V and O itself.
"""
from __future__ import annotations

import torch

from . import binding


class _BaspAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, plan, softmax_scale, fused, *shards):
        n = plan.N
        if len(shards) != 3 * n:
            raise ValueError(f"expected {3 * n} shards (q, k, v of {n} ranks), got {len(shards)}")
        q_seq, k_seq, v_seq = shards[:n], shards[n:2 * n], shards[2 * n:]
        for t in shards:
            if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
                raise ValueError("shards must be contiguous bf16 CUDA tensors")
        dev = q_seq[0].device
        o_seq = [torch.empty_like(t) for t in q_seq]
        lse = [torch.empty((plan.Bl, plan.Hq_l, plan.S), dtype=torch.float32, device=dev) for _ in range(n)]
        if fused:
            binding.basp_layer_fwd_fused(plan, list(q_seq), list(k_seq), list(v_seq), o_seq, lse, softmax_scale=softmax_scale)
            ws = None
            ctx.save_for_backward(*shards, *o_seq)
        else:
            ws = torch.empty(binding.basp_workspace_bytes(plan), dtype=torch.uint8, device=dev)
            binding.basp_layer_fwd(plan, list(q_seq), list(k_seq), list(v_seq), o_seq, ws, lse_shards=lse,
                                   softmax_scale=softmax_scale)
        ctx.plan, ctx.softmax_scale, ctx.ws, ctx.lse, ctx.fused = plan, softmax_scale, ws, lse, fused
        ctx.shapes = [t.shape for t in shards]
        return tuple(o_seq)

    @staticmethod
    def backward(ctx, *do_seq):
        plan, n = ctx.plan, ctx.plan.N
        dev = ctx.lse[0].device
        do_seq = [g.contiguous() if g is not None else None for g in do_seq]
        if any(g is None for g in do_seq):
            ref = next(g for g in do_seq if g is not None)
            do_seq = [g if g is not None else torch.zeros_like(ref) for g in do_seq]
        grads = [torch.empty(s, dtype=torch.bfloat16, device=dev) for s in ctx.shapes]
        if ctx.fused:
            saved = ctx.saved_tensors
            q_seq, k_seq, v_seq, o_seq = (list(saved[i * n:(i + 1) * n]) for i in range(4))
            ws2 = torch.empty(binding.basp_layer_bwd_seq_workspace_bytes(plan), dtype=torch.uint8, device=dev)
            binding.basp_layer_bwd_seq(plan, q_seq, k_seq, v_seq, o_seq, ctx.lse, do_seq, grads[:n], grads[n:2 * n],
                                       grads[2 * n:], ws2, softmax_scale=ctx.softmax_scale)
            return (None, None, None, *grads)
        qh, kh, vh, oh = (binding.as_shards(a) for a in binding.basp_layer_workspace_shards(plan, ctx.ws))
        ws2 = torch.empty(binding.basp_layer_bwd_workspace_bytes(plan), dtype=torch.uint8, device=dev)
        binding.basp_layer_bwd(plan, qh, kh, vh, oh, ctx.lse, do_seq, grads[:n], grads[n:2 * n], grads[2 * n:], ws2,
                               softmax_scale=ctx.softmax_scale)
        return (None, None, None, *grads)


def basp_attention(plan, q_seq, k_seq, v_seq, softmax_scale: float = 0.0, fused: bool = False):
    """Causal (or, per the plan, unmasked) attention over the group-sharded sequences of `plan`: the two group-local
    all-to-alls and the attention of Section IV-C, differentiable.  Returns the list of n_ranks output shards in the
    layout of q_seq."""
    return list(_BaspAttention.apply(plan, float(softmax_scale), bool(fused), *q_seq, *k_seq, *v_seq))
