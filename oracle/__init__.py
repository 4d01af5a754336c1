"""fp64 CPU oracle of the BASP attention layer -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``basp_oracle.c`` (plain C, fp64, literal loops of the
paper's definitions: Algorithm 1, Algorithm 2, the two group-local all-to-alls of
Section IV-C and the attention equation of Section II-A with a causal mask).

Nothing here is imported by the CUDA package; only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it.  It shares no code with the CUDA path.

Conventions
-----------
* bf16 tensors are numpy ``uint16`` arrays holding the bit patterns.
* ``seq`` arenas are ``[N, Bl, T, H, D]``, ``head`` arenas ``[N, Bl, S, H/K, D]``.
* ``G = 0`` (or ``G = B``) is BASP, ``G = 1`` is standard Ulysses.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "basp_oracle.c")
_LIB = os.path.join(_HERE, "libbasp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP, strict IEEE: no -ffast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-march=native", "-fopenmp", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        try:
            subprocess.check_call(cmd)
        except subprocess.CalledProcessError:
            cmd.remove("-march=native")
            subprocess.check_call(cmd)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


# ----------------------------------------------------------------------------- plan
@dataclass(frozen=True)
class Plan:
    N: int      # ranks
    B: int      # micro-batch (sequences)
    G: int      # groups
    K: int      # ranks per group
    Bl: int     # sequences per group
    S: int      # tokens per sequence
    T: int      # tokens per rank and sequence
    T_last: int = 0   # tokens of a group's LAST rank when K does not divide S (plan_uneven); 0 = T

    @property
    def uneven(self) -> bool:
        return self.T_last not in (0, self.T)

    def token_range(self, l: int) -> tuple[int, int]:
        """Tokens [begin, end) of local rank l (Algorithm 2's token_start / token_end, clipped to the sequence)."""
        return min(l * self.T, self.S), min((l + 1) * self.T, self.S)

    def group_ranks(self, g: int) -> list[int]:
        out = (ctypes.c_int * self.K)()
        _load().oracle_group_ranks(self.K, g, out)
        return list(out)

    def rank_info(self, r: int, Hq: int, Hkv: int) -> dict:
        out = (ctypes.c_int * 10)()
        _load().oracle_rank_info(self.K, self.Bl, self.T, Hq, Hkv, r, out)
        keys = ("group", "local_rank", "seq_begin", "seq_end", "token_begin", "token_end",
                "q_head_begin", "q_head_end", "kv_head_begin", "kv_head_end")
        return dict(zip(keys, list(out)))


def plan(N: int, B: int, S: int, G: int = 0) -> Plan:
    """Algorithm 1 (+ the explicit group count of Section IV-C).  Raises ValueError
    where the paper asserts or declares the case unsupported."""
    out = (ctypes.c_int * 4)()
    rc = _load().oracle_plan(int(N), int(B), int(G), int(S), out)
    if rc != 0:
        raise ValueError(f"invalid BASP plan N={N} B={B} G={G} S={S}")
    K, G_, Bl, T = list(out)
    return Plan(N=N, B=B, G=G_, K=K, Bl=Bl, S=S, T=T)


def plan_uneven(N: int, B: int, S: int, G: int = 0) -> Plan:
    """The plan for a sequence length that the group size does not divide.  Algorithm 2 writes the chunk as L / K and
    the paper says nothing about a remainder; the reading taken: chunk = ceil(S / K), local rank l holds tokens
    [l chunk, min((l+1) chunk, S)), so only the group's last rank is short, and it must not be empty.  The groups
    themselves (Algorithm 1) do not depend on S."""
    base = plan(N, B, N, G)                      # group structure only (any S that K divides)
    K = base.K
    T = -(-S // K)
    T_last = S - (K - 1) * T
    if S <= 0 or T_last <= 0:
        raise ValueError(f"invalid uneven plan N={N} B={B} G={G} S={S}: the last rank of a group would be empty")
    return Plan(N=N, B=B, G=base.G, K=K, Bl=base.Bl, S=S, T=T, T_last=T_last)


def group_sizes(N: int, B: int) -> list[int]:
    """Ranks per group when B does not divide N.  Algorithm 1 asserts N mod B = 0 and the paper leaves the other case
    to future work; the reading taken keeps its structure (B groups of contiguous ranks, one sequence each) and lets
    the sizes differ by at most one: the first N mod B groups get ceil(N/B) ranks, the others floor(N/B)."""
    if N <= 0 or B <= 0 or B > N:
        raise ValueError(f"invalid group formation N={N} B={B}")
    big = N % B
    return [-(-N // B)] * big + [N // B] * (B - big)


@dataclass(frozen=True)
class PlanPart:
    plan: Plan        # a uniform plan over this part's ranks and sequences
    rank_begin: int   # first global rank of the part
    seq_begin: int    # first sequence of the micro-batch that the part works on


def plan_parts(N: int, B: int, S: int) -> list:
    """The unequal groups of :func:`group_sizes` as at most two uniform plans over disjoint rank and sequence ranges:
    the groups of ceil(N/B) ranks (ranks from 0, sequences from 0) and the groups of floor(N/B) ranks (the rest).
    With B | N this is the one plan of Algorithm 1.  A length that a group size does not divide is cut unevenly
    (plan_uneven)."""
    sizes = group_sizes(N, B)
    parts, r0, b0 = [], 0, 0
    for K in sorted(set(sizes), reverse=True):
        n_groups = sizes.count(K)
        mk = plan if S % K == 0 else plan_uneven
        parts.append(PlanPart(mk(n_groups * K, n_groups, S), r0, b0))
        r0 += n_groups * K
        b0 += n_groups
    assert r0 == N and b0 == B
    return parts


def layer_fwd_parts(Xq: np.ndarray, Xk: np.ndarray, Xv: np.ndarray, parts: list, scale: float | None = None,
                    causal: bool = True) -> dict:
    """The layer over unequal groups: every part runs the layer of its own plan on its own sequences."""
    outs = [layer_fwd(Xq[pt.seq_begin:pt.seq_begin + pt.plan.B], Xk[pt.seq_begin:pt.seq_begin + pt.plan.B],
                      Xv[pt.seq_begin:pt.seq_begin + pt.plan.B], pt.plan, scale, causal) for pt in parts]
    return dict(parts=outs, o_global=np.concatenate([o["o_global"] for o in outs], axis=0))


def layer_bwd_parts(Xq, Xk, Xv, XdO, parts: list, scale: float | None = None, causal: bool = True) -> dict:
    sl = lambda X, pt: X[pt.seq_begin:pt.seq_begin + pt.plan.B]
    outs = [layer_bwd(sl(Xq, pt), sl(Xk, pt), sl(Xv, pt), sl(XdO, pt), pt.plan, scale, causal) for pt in parts]
    res = dict(parts=outs)
    for n in ("dq", "dk", "dv"):
        res[n + "_global"] = np.concatenate([o[n + "_global"] for o in outs], axis=0)
    return res


# ------------------------------------------------------------------ permutations
def _esize(a: np.ndarray) -> int:
    return int(a.dtype.itemsize)


def partition(X: np.ndarray, pl: Plan) -> np.ndarray:
    """Algorithm 2 for every rank: X[B,S,H,D] -> [N,Bl,T,H,D]."""
    X = np.ascontiguousarray(X)
    B, S, H, D = X.shape
    assert B == pl.B and S == pl.S
    out = np.empty((pl.N, pl.Bl, pl.T, H, D), dtype=X.dtype)
    _load().oracle_partition(_p(X), _p(out), pl.N, pl.K, pl.Bl, S, H, D, _esize(X))
    return out


def gather(shards: np.ndarray, pl: Plan) -> np.ndarray:
    """Inverse of :func:`partition`: [N,Bl,T,H,D] -> X[B,S,H,D]."""
    shards = np.ascontiguousarray(shards)
    N, Bl, T, H, D = shards.shape
    out = np.empty((pl.B, pl.S, H, D), dtype=shards.dtype)
    _load().oracle_gather(_p(shards), _p(out), pl.N, pl.K, pl.Bl, pl.S, H, D, _esize(shards))
    return out


# The same four maps when the last rank of a group is short (plan_uneven): the shards differ in length, so they are a
# list of N arrays [Bl, T_r, H, D]; the head-sharded side is unchanged ([N, Bl, S, H/K, D], every rank holds whole
# sequences).  Written as slice assignments of the index maps, one (group, source rank, destination rank) at a time.
def partition_uneven(X: np.ndarray, pl: Plan) -> list:
    """Algorithm 2 for every rank with chunk = ceil(S/K): rank gK+l gets X[g Bl:(g+1) Bl, token_range(l)]."""
    assert X.shape[0] == pl.B and X.shape[1] == pl.S
    out = []
    for r in range(pl.N):
        g, l = divmod(r, pl.K)
        t0, t1 = pl.token_range(l)
        out.append(np.ascontiguousarray(X[g * pl.Bl:(g + 1) * pl.Bl, t0:t1]))
    return out


def gather_uneven(shards: list, pl: Plan) -> np.ndarray:
    """Inverse of :func:`partition_uneven`."""
    H, D = shards[0].shape[2:]
    out = np.empty((pl.B, pl.S, H, D), dtype=shards[0].dtype)
    for r in range(pl.N):
        g, l = divmod(r, pl.K)
        t0, t1 = pl.token_range(l)
        assert shards[r].shape == (pl.Bl, t1 - t0, H, D)
        out[g * pl.Bl:(g + 1) * pl.Bl, t0:t1] = shards[r]
    return out


def s2h_uneven(shards: list, pl: Plan) -> np.ndarray:
    """First all-to-all from uneven shards: head[gK+m][bl][s][h'] = seq[gK+src][bl][s - src T][m H/K + h'] with src
    the rank whose token range holds s.  A tensor with fewer heads than the group has ranks is replicated as in
    :func:`s2h_replicated` (local rank m receives head m // (K/H))."""
    H, D = shards[0].shape[2:]
    K = pl.K
    assert H % K == 0 or K % H == 0
    Hl, rep = (H // K, 1) if H % K == 0 else (1, K // H)
    out = np.empty((pl.N, pl.Bl, pl.S, Hl, D), dtype=shards[0].dtype)
    for g in range(pl.G):
        for m in range(K):
            h0 = m * Hl if rep == 1 else m // rep
            for src in range(K):
                t0, t1 = pl.token_range(src)
                out[g * K + m, :, t0:t1] = shards[g * K + src][:, :, h0:h0 + Hl, :]
    return out


def h2s_uneven(head: np.ndarray, pl: Plan, H: int | None = None) -> list:
    """Reverse all-to-all to uneven shards.  With H given and smaller than K the tensor is the gradient of a replicated
    K/V tensor and the copies are summed as in :func:`h2s_sum_replicated`."""
    N, Bl, S, Hl, D = head.shape
    K = pl.K
    assert (N, Bl, S) == (pl.N, pl.Bl, pl.S)
    if H is None:
        H = Hl * K
    rep = 1 if H % K == 0 else K // H
    out = []
    for r in range(N):
        g, dst = divmod(r, K)
        t0, t1 = pl.token_range(dst)
        o = np.zeros((Bl, t1 - t0, H, D), dtype=head.dtype)
        for m in range(K):
            if rep == 1:
                o[:, :, m * Hl:(m + 1) * Hl, :] = head[g * K + m, :, t0:t1]
            else:
                o[:, :, m // rep, :] += head[g * K + m, :, t0:t1, 0, :]
        out.append(o)
    return out


def s2h(seq: np.ndarray, pl: Plan) -> np.ndarray:
    """Group-local all-to-all, sequence-sharded -> head-sharded (Section IV-C)."""
    seq = np.ascontiguousarray(seq)
    N, Bl, T, H, D = seq.shape
    assert (N, Bl, T) == (pl.N, pl.Bl, pl.T) and H % pl.K == 0
    out = np.empty((N, Bl, pl.S, H // pl.K, D), dtype=seq.dtype)
    _load().oracle_s2h(_p(seq), _p(out), N, pl.K, Bl, pl.S, H, D, _esize(seq))
    return out


def s2h_replicated(seq: np.ndarray, pl: Plan) -> np.ndarray:
    """First all-to-all for a K/V tensor with FEWER heads than the group has ranks (K mod H = 0): local rank m needs
    the KV head that its query heads read, head m // (K/H), over the whole sequence, so each head is delivered to K/H
    consecutive local ranks.  seq [N,Bl,T,H,D] -> [N,Bl,S,1,D].  (The paper does not treat grouped-query attention;
    this is the head mapping h -> h / (Hq/Hkv) applied to the contiguous query-head blocks of Section IV-C.)"""
    seq = np.ascontiguousarray(seq)
    N, Bl, T, H, D = seq.shape
    assert (N, Bl, T) == (pl.N, pl.Bl, pl.T) and pl.K % H == 0 and H < pl.K
    rep = pl.K // H
    out = np.empty((N, Bl, pl.S, 1, D), dtype=seq.dtype)
    for g in range(pl.G):
        for m in range(pl.K):                      # destination local rank
            for src in range(pl.K):                # source local rank = chunk of the sequence
                out[g * pl.K + m, :, src * T:(src + 1) * T, 0, :] = seq[g * pl.K + src, :, :, m // rep, :]
    return out


def h2s_sum_replicated(head: np.ndarray, pl: Plan, H: int) -> np.ndarray:
    """Reverse all-to-all of the GRADIENT of a replicated K/V tensor (see :func:`s2h_replicated`): the K/H local ranks
    that received a copy of KV head h each hold the gradient contribution of their own query heads, so the gradient of
    head h is their sum.  head [N,Bl,S,1,D] (fp64) -> [N,Bl,T,H,D]."""
    head = np.ascontiguousarray(head)
    N, Bl, S, one, D = head.shape
    assert (N, Bl, S, one) == (pl.N, pl.Bl, pl.S, 1) and pl.K % H == 0 and H < pl.K
    rep, T = pl.K // H, pl.T
    out = np.zeros((N, Bl, T, H, D), dtype=head.dtype)
    for g in range(pl.G):
        for dst in range(pl.K):                    # owner of tokens [dst*T, (dst+1)*T)
            for m in range(pl.K):                  # local rank that holds a copy of head m // rep
                out[g * pl.K + dst, :, :, m // rep, :] += head[g * pl.K + m, :, dst * T:(dst + 1) * T, 0, :]
    return out


def h2s(head: np.ndarray, pl: Plan) -> np.ndarray:
    """Group-local all-to-all, head-sharded -> sequence-sharded (the reverse one)."""
    head = np.ascontiguousarray(head)
    N, Bl, S, Hl, D = head.shape
    assert (N, Bl, S) == (pl.N, pl.Bl, pl.S)
    out = np.empty((N, Bl, pl.T, Hl * pl.K, D), dtype=head.dtype)
    _load().oracle_h2s(_p(head), _p(out), N, pl.K, Bl, S, Hl * pl.K, D, _esize(head))
    return out


# --------------------------------------------------------------------- attention
def attn_fwd(Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float | None = None,
             causal: bool = True):
    """Attention from its definition on bf16 bit patterns.

    Q [Bn,S,Hq,D], K,V [Bn,S,Hkv,D] uint16 -> (O [Bn,S,Hq,D] f64, LSE [Bn,Hq,S] f64)."""
    Q, K, V = (np.ascontiguousarray(a, dtype=np.uint16) for a in (Q, K, V))
    Bn, S, Hq, D = Q.shape
    Hkv = K.shape[2]
    assert K.shape == (Bn, S, Hkv, D) and V.shape == K.shape and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    O = np.empty((Bn, S, Hq, D), dtype=np.float64)
    LSE = np.empty((Bn, Hq, S), dtype=np.float64)
    _load().oracle_attn_fwd(_p(Q), _p(K), _p(V), _p(O), _p(LSE), Bn, S, Hq, Hkv, D,
                            ctypes.c_double(scale), int(causal))
    return O, LSE


def attn_fwd_rows(Q: np.ndarray, K: np.ndarray, V: np.ndarray, rows: np.ndarray,
                  scale: float | None = None, causal: bool = True):
    """Selected output rows; ``rows`` is int32 [n,3] of (b, h, i).  Returns
    (O_rows [n,D] f64, lse_rows [n] f64)."""
    Q, K, V = (np.ascontiguousarray(a, dtype=np.uint16) for a in (Q, K, V))
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    Bn, S, Hq, D = Q.shape
    Hkv = K.shape[2]
    assert K.shape == (Bn, S, Hkv, D) and V.shape == K.shape and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    n = rows.shape[0]
    O = np.empty((n, D), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    _load().oracle_attn_fwd_rows(_p(Q), _p(K), _p(V), _p(rows), n, _p(O), _p(lse), S, Hq, Hkv,
                                 D, ctypes.c_double(scale), int(causal))
    return O, lse


def _scale(scale, D):
    return 1.0 / np.sqrt(D) if scale is None else scale


def attn_bwd(Q, K, V, dO, scale: float | None = None, causal: bool = True):
    """Gradients of attention by the chain rule (see basp_oracle.c).  Q, dO [Bn,S,Hq,D]; K, V
    [Bn,S,Hkv,D] uint16.  Returns dict(dQ, dK, dV, LSE, DELTA) in fp64 (LSE/DELTA [Bn,Hq,S])."""
    Q, K, V, dO = (np.ascontiguousarray(a, dtype=np.uint16) for a in (Q, K, V, dO))
    Bn, S, Hq, D = Q.shape
    Hkv = K.shape[2]
    assert dO.shape == Q.shape and K.shape == (Bn, S, Hkv, D) and V.shape == K.shape
    dQ = np.empty(Q.shape, dtype=np.float64)
    dK = np.empty(K.shape, dtype=np.float64)
    dV = np.empty(K.shape, dtype=np.float64)
    LSE = np.empty((Bn, Hq, S), dtype=np.float64)
    DELTA = np.empty((Bn, Hq, S), dtype=np.float64)
    _load().oracle_attn_bwd(_p(Q), _p(K), _p(V), _p(dO), _p(dQ), _p(dK), _p(dV), _p(LSE), _p(DELTA), Bn, S, Hq,
                            Hkv, D, ctypes.c_double(_scale(scale, D)), int(causal))
    return dict(dQ=dQ, dK=dK, dV=dV, LSE=LSE, DELTA=DELTA)


def attn_bwd_dq_rows(Q, K, V, dO, rows, scale: float | None = None, causal: bool = True):
    """dQ of selected rows; ``rows`` int32 [n,3] of (b, h, i) -> [n, D] fp64."""
    Q, K, V, dO = (np.ascontiguousarray(a, dtype=np.uint16) for a in (Q, K, V, dO))
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    Bn, S, Hq, D = Q.shape
    out = np.empty((rows.shape[0], D), dtype=np.float64)
    _load().oracle_attn_bwd_dq_rows(_p(Q), _p(K), _p(V), _p(dO), _p(rows), rows.shape[0], _p(out), S, Hq,
                                    K.shape[2], D, ctypes.c_double(_scale(scale, D)), int(causal))
    return out


def attn_bwd_dkdv_tail(Q, K, V, dO, b: int, kv: int, ncols: int, scale: float | None = None):
    """dK, dV of the last ``ncols`` key positions of (sequence b, KV head kv), causal -> two [ncols, D]."""
    Q, K, V, dO = (np.ascontiguousarray(a, dtype=np.uint16) for a in (Q, K, V, dO))
    Bn, S, Hq, D = Q.shape
    dK = np.empty((ncols, D), dtype=np.float64)
    dV = np.empty((ncols, D), dtype=np.float64)
    _load().oracle_attn_bwd_dkdv_tail(_p(Q), _p(K), _p(V), _p(dO), int(b), int(kv), int(ncols), _p(dK), _p(dV),
                                      S, Hq, K.shape[2], D, ctypes.c_double(_scale(scale, D)))
    return dK, dV


def attn_bwd_dkdv_cols(Q, K, V, dO, b: int, kv: int, cols, scale: float | None = None, causal: bool = True):
    """dK, dV of the key positions ``cols`` (any positions) of (sequence b, KV head kv) -> two [len(cols), D] fp64.
    The row statistics (LSE, Delta) of every row that sees the smallest sampled column are formed once, from each
    row's own definition, and shared by the columns."""
    Q, K, V, dO = (np.ascontiguousarray(a, dtype=np.uint16) for a in (Q, K, V, dO))
    cols = np.ascontiguousarray(cols, dtype=np.int32).reshape(-1)
    Bn, S, Hq, D = Q.shape
    assert 0 <= b < Bn and 0 <= kv < K.shape[2] and ((cols >= 0) & (cols < S)).all()
    dK = np.empty((cols.shape[0], D), dtype=np.float64)
    dV = np.empty((cols.shape[0], D), dtype=np.float64)
    _load().oracle_attn_bwd_dkdv_cols(_p(Q), _p(K), _p(V), _p(dO), int(b), int(kv), _p(cols), int(cols.shape[0]),
                                      _p(dK), _p(dV), S, Hq, K.shape[2], D, ctypes.c_double(_scale(scale, D)),
                                      int(causal))
    return dK, dV


def layer_bwd(Xq, Xk, Xv, XdO, pl: Plan, scale: float | None = None, causal: bool = True):
    """Backward of the sequence-parallel layer, step by step: partition the four global tensors,
    all-to-all each to head-sharded, per-rank attention backward, reverse all-to-all of dQ, dK, dV,
    collect.  Returns dict with head- and sequence-sharded gradients and the global ones."""
    Hkv = Xk.shape[2]
    replicated = Hkv % pl.K != 0                  # more ranks in a group than KV heads
    if pl.uneven:
        qh, doh, kh, vh = (s2h_uneven(partition_uneven(X, pl), pl) for X in (Xq, XdO, Xk, Xv))
    else:
        kv_s2h = s2h_replicated if replicated else s2h
        qh, doh = s2h(partition(Xq, pl), pl), s2h(partition(XdO, pl), pl)
        kh, vh = kv_s2h(partition(Xk, pl), pl), kv_s2h(partition(Xv, pl), pl)
    dqh = np.empty(qh.shape, dtype=np.float64)
    dkh = np.empty(kh.shape, dtype=np.float64)
    dvh = np.empty(kh.shape, dtype=np.float64)
    for r in range(pl.N):
        g = attn_bwd(qh[r], kh[r], vh[r], doh[r], scale, causal)
        dqh[r], dkh[r], dvh[r] = g["dQ"], g["dK"], g["dV"]
    out = dict(dq_head=dqh, dk_head=dkh, dv_head=dvh, do_head=doh)
    for n, a in (("dq", dqh), ("dk", dkh), ("dv", dvh)):
        if pl.uneven:
            out[n + "_seq"] = h2s_uneven(a, pl, None if n == "dq" else Hkv)
            out[n + "_global"] = gather_uneven(out[n + "_seq"], pl)
            continue
        out[n + "_seq"] = h2s_sum_replicated(a, pl, Hkv) if (replicated and n != "dq") else h2s(a, pl)
        out[n + "_global"] = gather(out[n + "_seq"], pl)
    return out


# ------------------------------------------------------------------------- layer
def layer_fwd(Xq: np.ndarray, Xk: np.ndarray, Xv: np.ndarray, pl: Plan,
              scale: float | None = None, causal: bool = True):
    """The whole sequence-parallel layer on global tensors, step by step as the
    paper describes it: partition (Alg. 2) -> all-to-all -> per-rank attention over
    the rank's head slice -> reverse all-to-all -> collect.

    Xq [B,S,Hq,D], Xk,Xv [B,S,Hkv,D] uint16.  Returns a dict with every intermediate
    (seq shards, head shards, per-rank O/LSE in fp64) and the global O [B,S,Hq,D]."""
    if pl.uneven:
        qs, ks, vs = (partition_uneven(X, pl) for X in (Xq, Xk, Xv))
        qh, kh, vh = (s2h_uneven(x, pl) for x in (qs, ks, vs))
    else:
        qs, ks, vs = partition(Xq, pl), partition(Xk, pl), partition(Xv, pl)
        kv_s2h = s2h if Xk.shape[2] % pl.K == 0 else s2h_replicated
        qh, kh, vh = s2h(qs, pl), kv_s2h(ks, pl), kv_s2h(vs, pl)
    N = pl.N
    oh = np.empty(qh.shape, dtype=np.float64)
    lse = np.empty((N, pl.Bl, qh.shape[3], pl.S), dtype=np.float64)
    for r in range(N):
        oh[r], lse[r] = attn_fwd(qh[r], kh[r], vh[r], scale, causal)
    os_ = h2s_uneven(oh, pl) if pl.uneven else h2s(oh, pl)
    return dict(q_seq=qs, k_seq=ks, v_seq=vs, q_head=qh, k_head=kh, v_head=vh,
                o_head=oh, lse_head=lse, o_seq=os_,
                o_global=gather_uneven(os_, pl) if pl.uneven else gather(os_, pl))


# ------------------------------------------------------------------- projections
def linear(X: np.ndarray, W: np.ndarray) -> np.ndarray:
    """The projections of Section II-A (Q = X W_Q, ..., Concat(H_i) W_O) as one product in fp64:
    X [M,K] and W [N,K] are bf16 bit patterns (W holds one output feature per row); returns X . W^T [M,N]."""
    return bf16_bits_to_f64(X) @ bf16_bits_to_f64(W).T


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray, positions: np.ndarray) -> np.ndarray:
    """Rotary position embedding in the rotate-half form, in fp64 (the paper does not treat position encodings; this
    is the convention of the Llama / Qwen models it trains): within a head, feature j < D/2 pairs with feature
    j + D/2 and the pair is turned by the angle of (position, j):
        y_j = x_j cos - x_{j+D/2} sin,    y_{j+D/2} = x_{j+D/2} cos + x_j sin.
    x [tokens, H, D] (fp64), cos / sin [S, D/2] tables (any float type, read as given), positions [tokens]."""
    x = np.asarray(x, dtype=np.float64)
    tokens, H, D = x.shape
    half = D // 2
    c = np.asarray(cos, dtype=np.float64)[np.asarray(positions)][:, None, :]      # [tokens, 1, D/2]
    s_ = np.asarray(sin, dtype=np.float64)[np.asarray(positions)][:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s_, hi * c + lo * s_], axis=-1)


def qkv_proj_rope(X: np.ndarray, W: np.ndarray, Hq: int, Hkv: int, D: int, cos, sin, positions) -> tuple:
    """Q = X W_Q, K = X W_K, V = X W_V (Section II-A) with the rotation applied to Q and K before anything is rounded.
    X [tokens, hidden], W [(Hq + 2 Hkv) D, hidden] as bf16 bits; returns fp64 (Q [tokens,Hq,D], K, V [tokens,Hkv,D])."""
    Y = linear(X, W)
    tokens = Y.shape[0]
    q = Y[:, :Hq * D].reshape(tokens, Hq, D)
    k = Y[:, Hq * D:(Hq + Hkv) * D].reshape(tokens, Hkv, D)
    v = Y[:, (Hq + Hkv) * D:].reshape(tokens, Hkv, D)
    return rope(q, cos, sin, positions), rope(k, cos, sin, positions), v


# ----------------------------------------------------------------- bf16 helpers
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).astype(np.float64)
