"""Pins of the oracle's plan against what the paper fixes (Algorithms 1 and 2, Table I)."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden", "plan_examples.txt")


def _golden():
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        n, b, k, groups = line.split()
        yield int(n), int(b), int(k), [[int(x) for x in g.split(",")] for g in groups.split("|")]


@pytest.mark.parametrize("N,B,K,groups", list(_golden()))
def test_paper_worked_examples(N, B, K, groups):
    pl = oracle.plan(N, B, S=1024)
    assert pl.K == K and pl.G == B and pl.Bl == 1
    assert [pl.group_ranks(g) for g in range(pl.G)] == groups


@pytest.mark.parametrize("N", [1, 2, 4, 6, 8, 12, 16, 64])
def test_table1_closed_forms(N):
    S = 3840  # divisible by every K used here
    for B in [b for b in range(1, N + 1) if N % b == 0]:
        pl = oracle.plan(N, B, S)
        assert pl.K == N // B                    # all-to-all participants = N/B (Table I)
        assert pl.T * 1 == B * S // N            # tokens per GPU = B*S/N (Table I)
        seen = []
        for g in range(pl.G):
            seen += pl.group_ranks(g)
        assert seen == list(range(N))            # disjoint, contiguous, covering
        # Standard Ulysses (one group of N): same tokens per GPU (workload equivalence).
        if S % N == 0:
            ul = oracle.plan(N, B, S, G=1)
            assert ul.K == N and ul.Bl * ul.T == pl.Bl * pl.T == B * S // N


@pytest.mark.parametrize("N,B", [(4, 2), (8, 2), (8, 4), (16, 4), (6, 3)])
def test_table1_ulysses_with_sp_degree_n_over_b(N, B):
    """Table I's middle row: standard Ulysses with sequence-parallel degree N/B.  The N GPUs form B data-parallel
    replicas of N/B GPUs, and each replica works on a whole micro-batch of B sequences: as a plan that is B groups with B
    sequences per group (B*B sequences in flight).  Tokens per GPU B^2 S / N, all-to-all participants N/B, as printed;
    the same groups as BASP (which puts ONE sequence in each), B times the tokens per GPU."""
    S = 3840
    sp = oracle.plan(N, B * B, S, G=B)
    basp_plan = oracle.plan(N, B, S)
    assert sp.K == N // B == basp_plan.K                       # participants: N/B in both
    assert sp.Bl == B and sp.Bl * sp.T == B * B * S // N       # tokens per GPU = B^2 S / N
    assert sp.Bl * sp.T == B * basp_plan.Bl * basp_plan.T      # B times BASP's B S / N
    assert [sp.group_ranks(g) for g in range(B)] == [basp_plan.group_ranks(g) for g in range(B)]
    for r in range(N):
        ri = sp.rank_info(r, Hq=N, Hkv=N)
        assert (ri["seq_begin"], ri["seq_end"]) == (r // sp.K * B, (r // sp.K + 1) * B)   # a replica's own micro-batch


def test_rank_info_matches_algorithm2():
    pl = oracle.plan(8, 2, 32768)
    for r in range(8):
        ri = pl.rank_info(r, Hq=32, Hkv=8)
        assert ri["group"] == r // 4 and ri["local_rank"] == r % 4
        assert (ri["seq_begin"], ri["seq_end"]) == (r // 4, r // 4 + 1)
        assert (ri["token_begin"], ri["token_end"]) == ((r % 4) * 8192, (r % 4 + 1) * 8192)
        assert (ri["q_head_begin"], ri["q_head_end"]) == ((r % 4) * 8, (r % 4 + 1) * 8)
        assert (ri["kv_head_begin"], ri["kv_head_end"]) == ((r % 4) * 2, (r % 4 + 1) * 2)


def test_more_sequences_than_ranks_falls_back_to_data_parallelism():
    """Section IV-B: with B > N there is nothing to shard; every rank takes whole sequences (K = 1, B/N of them)."""
    pl = oracle.plan(4, 8, 1024)
    assert (pl.K, pl.G, pl.Bl, pl.T) == (1, 4, 2, 1024)
    for r in range(4):
        ri = pl.rank_info(r, Hq=8, Hkv=8)
        assert (ri["group"], ri["local_rank"]) == (r, 0)
        assert (ri["seq_begin"], ri["seq_end"]) == (2 * r, 2 * r + 2)
        assert (ri["token_begin"], ri["token_end"]) == (0, 1024) and (ri["q_head_begin"], ri["q_head_end"]) == (0, 8)
    X = np.arange(8 * 1024 * 8 * 2, dtype=np.int32).reshape(8, 1024, 8, 2)
    seq = oracle.partition(X, pl)
    assert np.array_equal(seq.reshape(X.shape), X)                 # rank r holds sequences 2r, 2r+1 whole
    assert np.array_equal(oracle.s2h(seq, pl), seq)                # the exchange of a one-rank group is the identity


@pytest.mark.parametrize("N,B,S,G", [
    (8, 3, 1024, 0),     # N mod B != 0 (Algorithm 1's assertion)
    (4, 6, 1024, 0),     # B > N and N does not divide B: no data-parallel split either
    (8, 2, 1022, 0),     # S not divisible by K
    (8, 4, 1024, 3),     # G does not divide N / B
    (0, 1, 1024, 0),
])
def test_invalid_plans(N, B, S, G):
    with pytest.raises(ValueError):
        oracle.plan(N, B, S, G)
