// Group planner: Algorithm 1 (batch-aware group creation) and Algorithm 2 (batch-aware
// sequence partitioning) as integer arithmetic on the host.  No communicator is built:
// a group is the contiguous rank range [g*K, (g+1)*K).
#include <new>

#include "plan.h"

extern "C" int basp_plan_create(const basp_config *cfg, basp_plan **out) {
    if (!cfg || !out) return BASP_ERR_NULL;
    *out = nullptr;
    const int N = cfg->n_ranks, B = cfg->micro_batch, S = cfg->seq_len;
    const int Hq = cfg->n_q_heads, Hkv = cfg->n_kv_heads, D = cfg->head_dim;
    if (N <= 0 || B <= 0 || S <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || cfg->num_groups < 0)
        return BASP_ERR_INVALID;
    // Algorithm 1: num_groups = B.  With more sequences than ranks the method falls back to plain data parallelism
    // (Section IV-B): every rank is a group of its own (K = 1) holding B/N whole sequences; the exchanges are identities.
    const int G = cfg->num_groups == 0 ? (B > N ? N : B) : cfg->num_groups;
    if (N % G != 0 || B % G != 0) return BASP_ERR_INVALID;      // Algorithm 1: assert N mod B = 0
    const int K = N / G;                                         // Algorithm 1: K = N / B
    // Algorithm 2: chunk = L / K.  Where K does not divide L (the paper is silent) the chunk is rounded up and the
    // group's last rank holds the short remainder, which must not be empty.
    const int T = (S + K - 1) / K, T_last = S - (K - 1) * T;
    if (T_last <= 0) return BASP_ERR_INVALID;
    // Each rank takes Hq/K query heads and their KV heads.  A group with more ranks than KV heads replicates: KV head
    // h goes to the K/Hkv consecutive local ranks whose query heads read it (one KV head per rank).
    if (Hq % Hkv != 0 || Hq % K != 0) return BASP_ERR_INVALID;
    if (Hkv % K != 0 && K % Hkv != 0) return BASP_ERR_INVALID;
    const int kv_rep = Hkv % K == 0 ? 1 : K / Hkv, Hkv_l = Hkv % K == 0 ? Hkv / K : 1;
    if (cfg->dtype != BASP_DTYPE_BF16 || N > BASP_MAX_RANKS) return BASP_ERR_UNSUPPORTED;
    if ((Hkv_l * D * 2) % 16 != 0 || ((Hq / K) * D * 2) % 16 != 0) return BASP_ERR_UNSUPPORTED;
    if (cfg->causal != 0 && cfg->causal != 1) return BASP_ERR_INVALID;

    basp_plan *p = new (std::nothrow) basp_plan;
    if (!p) return BASP_ERR_INVALID;
    p->cfg = *cfg;
    p->N = N; p->B = B; p->G = G; p->K = K; p->Bl = B / G; p->S = S; p->T = T; p->T_last = T_last;
    p->Hq = Hq; p->Hkv = Hkv; p->D = D; p->Hq_l = Hq / K; p->Hkv_l = Hkv_l; p->kv_rep = kv_rep;
    p->causal = cfg->causal;
    *out = p;
    return BASP_OK;
}

// Unequal groups (B does not divide N): the first N mod B groups take ceil(N/B) ranks, the others floor(N/B); each
// size class is a uniform plan of its own over a contiguous range of ranks and sequences.
extern "C" int basp_plan_create_parts(const basp_config *cfg, basp_plan_part parts[2], int *n_parts) {
    if (!cfg || !parts || !n_parts) return BASP_ERR_NULL;
    *n_parts = 0;
    parts[0].plan = parts[1].plan = nullptr;
    const int N = cfg->n_ranks, B = cfg->micro_batch;
    if (N <= 0 || B <= 0) return BASP_ERR_INVALID;
    if (cfg->num_groups != 0 && cfg->num_groups != B) return BASP_ERR_INVALID;
    if (B > N) {                              // the data-parallel fallback is one uniform plan
        basp_config c = *cfg;
        c.num_groups = 0;
        const int rc = basp_plan_create(&c, &parts[0].plan);
        if (rc != BASP_OK) return rc;
        parts[0].rank_begin = 0; parts[0].n_ranks = N; parts[0].seq_begin = 0; parts[0].n_seqs = B; parts[0].group_size = 1;
        *n_parts = 1;
        return BASP_OK;
    }
    const int big = N % B, k_hi = (N + B - 1) / B, k_lo = N / B;
    const int groups[2] = {big == 0 ? B : big, big == 0 ? 0 : B - big};
    const int sizes[2] = {big == 0 ? k_lo : k_hi, k_lo};
    int r0 = 0, b0 = 0;
    for (int i = 0; i < 2 && groups[i] > 0; ++i) {
        basp_config c = *cfg;
        c.n_ranks = groups[i] * sizes[i];
        c.micro_batch = groups[i];
        c.num_groups = 0;
        const int rc = basp_plan_create(&c, &parts[i].plan);
        if (rc != BASP_OK) {
            if (i == 1) { basp_plan_destroy(parts[0].plan); parts[0].plan = nullptr; }
            *n_parts = 0;
            return rc;
        }
        parts[i].rank_begin = r0; parts[i].n_ranks = c.n_ranks;
        parts[i].seq_begin = b0; parts[i].n_seqs = groups[i];
        parts[i].group_size = sizes[i];
        r0 += c.n_ranks; b0 += groups[i];
        *n_parts = i + 1;
    }
    return BASP_OK;
}

extern "C" int basp_plan_destroy(basp_plan *plan) {
    if (!plan) return BASP_ERR_NULL;
    delete plan;
    return BASP_OK;
}

extern "C" int basp_plan_get_info(const basp_plan *p, basp_plan_info *info) {
    if (!p || !info) return BASP_ERR_NULL;
    info->group_size = p->K;
    info->num_groups = p->G;
    info->seqs_per_group = p->Bl;
    info->tokens_per_rank = p->T;
    info->tokens_last_rank = p->T_last;
    info->q_heads_per_rank = p->Hq_l;
    info->kv_heads_per_rank = p->Hkv_l;
    // Workload equivalence (Section IV-C): Bl*T*H*D = (B*S/N)*H*D for every grouping.
    info->q_shard_elems = (size_t)p->Bl * p->T * p->Hq * p->D;
    info->kv_shard_elems = (size_t)p->Bl * p->T * p->Hkv * p->D;
    info->lse_shard_elems = (size_t)p->Bl * p->Hq_l * p->S;
    return BASP_OK;
}

extern "C" int basp_plan_get_rank(const basp_plan *p, int r, basp_rank_info *info) {
    if (!p || !info) return BASP_ERR_NULL;
    if (r < 0 || r >= p->N) return BASP_ERR_INVALID;
    const int g = r / p->K, l = r % p->K;       // Algorithm 2: my_group, my_local_rank
    info->group = g;
    info->local_rank = l;
    info->seq_begin = g * p->Bl;                // Algorithm 2: seq_start = my_group (Bl = 1)
    info->seq_end = (g + 1) * p->Bl;
    info->token_begin = l * p->T;               // Algorithm 2: token_start = local * chunk
    info->token_end = l * p->T + basp_rank_tokens(p, l);
    info->q_head_begin = l * p->Hq_l;
    info->q_head_end = (l + 1) * p->Hq_l;
    info->kv_head_begin = p->kv_rep > 1 ? l / p->kv_rep : l * p->Hkv_l;
    info->kv_head_end = info->kv_head_begin + p->Hkv_l;
    return BASP_OK;
}

extern "C" int basp_plan_group_ranks(const basp_plan *p, int group, int *ranks_out) {
    if (!p || !ranks_out) return BASP_ERR_NULL;
    if (group < 0 || group >= p->G) return BASP_ERR_INVALID;
    for (int j = 0; j < p->K; ++j) ranks_out[j] = group * p->K + j;   // Algorithm 1: [iK .. iK+K-1]
    return BASP_OK;
}
