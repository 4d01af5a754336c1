"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

Holds none of the method's arithmetic: only the workload table and a random-number
recipe.  Activations stand in for Llama/Qwen long-context training activations: dense,
equal-length sequences, i.i.d. N(0,1) drawn in fp32 on GLOBAL coordinates [B,S,H,D] in
the order Q, K, V (then dO) from one CPU generator, rounded to nearest-even bf16.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    N: int          # virtual ranks
    B: int          # micro-batch (sequences)
    S: int          # tokens per sequence
    Hq: int
    Hkv: int
    D: int
    G: int = 0      # 0 -> BASP (G = B); 1 -> standard Ulysses
    train: bool = False   # forward + backward step

    @property
    def K(self) -> int:
        return self.N // (self.G or min(self.B, self.N))     # more sequences than ranks: one rank per group

    @property
    def tokens(self) -> int:
        return self.B * self.S

    def attn_flops_fwd(self) -> float:
        """4*D flop per unmasked (i,j) pair, S(S+1)/2 pairs per (sequence, q head)."""
        return 4.0 * self.D * (self.S * (self.S + 1) / 2) * self.B * self.Hq

    def attn_flops_bwd(self) -> float:
        """10*D flop per unmasked pair (five products, the recomputed scores included)."""
        return 2.5 * self.attn_flops_fwd()

    def reshard_bytes_s2h(self) -> int:
        """Q, K and V each read once and written once."""
        return 2 * 2 * self.B * self.S * (self.Hq + 2 * self.Hkv) * self.D

    def reshard_bytes_h2s(self) -> int:
        return 2 * 2 * self.B * self.S * self.Hq * self.D


WORKLOADS = {
    "tiny": Workload("tiny", N=4, B=2, S=1024, Hq=8, Hkv=8, D=64),
    "llama3_8b_32k": Workload("llama3_8b_32k", N=8, B=2, S=32768, Hq=32, Hkv=8, D=128),
    "sweep_b1": Workload("sweep_b1", N=8, B=1, S=65536, Hq=32, Hkv=8, D=128),
    "sweep_b2": Workload("sweep_b2", N=8, B=2, S=32768, Hq=32, Hkv=8, D=128),
    "sweep_b4": Workload("sweep_b4", N=8, B=4, S=16384, Hq=32, Hkv=8, D=128),
    "sweep_b8": Workload("sweep_b8", N=8, B=8, S=8192, Hq=32, Hkv=8, D=128),
    "qwen25_7b_64k": Workload("qwen25_7b_64k", N=8, B=2, S=65536, Hq=28, Hkv=4, D=128),
    "qwen25_7b_16k": Workload("qwen25_7b_16k", N=8, B=2, S=16384, Hq=28, Hkv=4, D=128),      # the 64K shape cut down for profiler captures
    "llama3_8b_16k_train": Workload("llama3_8b_16k_train", N=8, B=1, S=16384, Hq=32, Hkv=8, D=128, train=True),
    "llama3_8b_128k_train": Workload("llama3_8b_128k_train", N=8, B=1, S=131072, Hq=32, Hkv=8, D=128, train=True),
}


# The paper's own sweep axes on one GPU (Section VI-C: S = 8K, micro-batch 1..8, Llama-3.2-1B, N = 8; Section VI-D:
# S = 1K..32K, micro-batch 2, Llama-3.2-3B).  The paper's table gives hidden size and 32 heads only; the shapes below are
# the public models' (1B: 32 query / 8 KV heads of 64; 3B: 24 / 8 heads of 128).
for _b in (1, 2, 4, 8):
    WORKLOADS[f"e5_b{_b}_basp"] = Workload(f"e5_b{_b}_basp", N=8, B=_b, S=8192, Hq=32, Hkv=8, D=64)
    WORKLOADS[f"e5_b{_b}_ulysses"] = Workload(f"e5_b{_b}_ulysses", N=8, B=_b, S=8192, Hq=32, Hkv=8, D=64, G=1)
# the same model shape as a training step (forward + backward), at the sweep's centre and at a long sequence
WORKLOADS["e5_b2_train"] = Workload("e5_b2_train", N=8, B=2, S=8192, Hq=32, Hkv=8, D=64, train=True)
WORKLOADS["llama32_1b_64k_train"] = Workload("llama32_1b_64k_train", N=8, B=1, S=65536, Hq=32, Hkv=8, D=64, train=True)
for _s in (1, 2, 4, 8, 16, 32):
    WORKLOADS[f"e6_s{_s}k_basp"] = Workload(f"e6_s{_s}k_basp", N=8, B=2, S=_s * 1024, Hq=24, Hkv=8, D=128)
    WORKLOADS[f"e6_s{_s}k_ulysses"] = Workload(f"e6_s{_s}k_ulysses", N=8, B=2, S=_s * 1024, Hq=24, Hkv=8, D=128, G=1)

# The six models of the paper's Table II exactly as printed there (hidden size, 32 attention heads, no KV-head count:
# taken as 32): head dimensions 64, 96, 128, 64, 80, 128, at the paper's S = 8K, micro-batch 2 on 8 ranks.
for _name, _hidden in (("llama32_1b", 2048), ("llama32_3b", 3072), ("llama31_8b", 4096),
                       ("qwen15_18b", 2048), ("qwen25_3b", 2560), ("qwen3_8b", 4096)):
    WORKLOADS[f"t2_{_name}"] = Workload(f"t2_{_name}", N=8, B=2, S=8192, Hq=32, Hkv=32, D=_hidden // 32)


def shrink(w: Workload, T: int = 512, name: str | None = None) -> Workload:
    """Same rank/head structure with T tokens per rank (S = T*K)."""
    return Workload(name or f"{w.name}_T{T}", w.N, w.B, T * w.K, w.Hq, w.Hkv, w.D, w.G, w.train)


def randn_bf16(gen: torch.Generator, shape) -> torch.Tensor:
    """N(0,1) in fp32, rounded to nearest-even bf16 (CPU tensor)."""
    return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16)


def make_qkv(w: Workload, seed: int = 0, with_dO: bool = False):
    """Global Q[B,S,Hq,D], K,V[B,S,Hkv,D] (and dO) as CPU bf16 tensors."""
    gen = torch.Generator().manual_seed(seed)
    q = randn_bf16(gen, (w.B, w.S, w.Hq, w.D))
    k = randn_bf16(gen, (w.B, w.S, w.Hkv, w.D))
    v = randn_bf16(gen, (w.B, w.S, w.Hkv, w.D))
    if with_dO:
        return q, k, v, randn_bf16(gen, (w.B, w.S, w.Hq, w.D))
    return q, k, v


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 CPU tensor -> numpy uint16 bit patterns (a copy)."""
    return t.contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def from_bits(a: np.ndarray) -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 CPU tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16).copy()).view(torch.bfloat16)


def random_bits(shape, seed: int = 0) -> np.ndarray:
    """Arbitrary 16-bit patterns (for bit-exact permutation checks)."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, 1 << 16, size=shape, dtype=np.uint16)


def rope_tables(S: int, D: int, base: float = 500000.0):
    """cos and sin of position * base^(-2j/D), j < D/2, as fp32 tensors [S, D/2] (angles formed in fp64; base 500000 is
    Llama 3's).  The rotary variant of the QKV projection takes them transposed, [D/2, S] contiguous."""
    j = torch.arange(D // 2, dtype=torch.float64)
    ang = torch.arange(S, dtype=torch.float64)[:, None] * (base ** (-2.0 * j / D))[None, :]
    return torch.cos(ang).to(torch.float32), torch.sin(ang).to(torch.float32)
