"""Writes the stored dK / dV reference columns of a large training workload.

    python tests/golden/make_dkdv_columns.py [--workload llama3_8b_128k_train] [--seed 0] [--kv 3]

Calls only the fp64 CPU oracle and the seeded input generator (never the CUDA path).  At S = 131072 the row
statistics of the four query heads of one KV head take tens of minutes of CPU time, which is why the result is
stored instead of being recomputed by every GPU test run.  The file is keyed by workload, seed and the CRC-32 of
each input tensor's bit pattern: the GPU test regenerates the inputs from the same seed, checks the CRCs and compares
the columns.
"""
from __future__ import annotations

import argparse
import os
import sys
import time
import zlib

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2609_03151_b200 import synth  # noqa: E402


def sampled_columns(S: int, T: int, seed: int) -> np.ndarray:
    """Key positions to check: the first 128 (summed over every row of the sequence), both sides of the first tile
    boundaries, both sides of every shard boundary l*T, the last 130, and 64 seeded random positions."""
    cols = set(range(128)) | {128, 255, 256}
    for edge in range(T, S, T):
        cols |= {edge - 1, edge}
    cols |= set(range(S - 130, S))
    rng = np.random.default_rng(seed + 1)
    cols |= {int(x) for x in rng.integers(0, S, 64)}
    return np.array(sorted(c for c in cols if 0 <= c < S), dtype=np.int32)


def crc(bits: np.ndarray) -> int:
    return zlib.crc32(memoryview(np.ascontiguousarray(bits)).cast("B")) & 0xFFFFFFFF


def path_for(workload: str, seed: int) -> str:
    return os.path.join(HERE, f"{workload}_dkdv_cols_seed{seed}.npz")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama3_8b_128k_train")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--kv", type=int, default=3, help="global KV head whose columns are stored")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    t0 = time.time()
    Q, K, V, dO = (synth.bits(t) for t in synth.make_qkv(w, seed=args.seed, with_dO=True))
    crcs = np.array([crc(a) for a in (Q, K, V, dO)], dtype=np.uint32)
    print(f"inputs ready after {time.time() - t0:.0f}s, crc32 {[hex(int(c)) for c in crcs]}", flush=True)
    cols = sampled_columns(w.S, -(-w.S // w.K), args.seed)
    dK, dV = oracle.attn_bwd_dkdv_cols(Q, K, V, dO, b=0, kv=args.kv, cols=cols)
    np.savez_compressed(path_for(args.workload, args.seed), cols=cols, dK=dK, dV=dV, crc32_q_k_v_do=crcs,
                        kv=np.int32(args.kv), seed=np.int32(args.seed),
                        shape_N_B_S_Hq_Hkv_D=np.array([w.N, w.B, w.S, w.Hq, w.Hkv, w.D], dtype=np.int64))
    print(f"wrote {path_for(args.workload, args.seed)}: {len(cols)} columns, {time.time() - t0:.0f}s, "
          f"{oracle.num_threads()} threads", flush=True)


if __name__ == "__main__":
    main()
