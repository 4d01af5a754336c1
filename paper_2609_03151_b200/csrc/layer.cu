// Whole-layer entry points: the three-launch path (all-to-all, attention, reverse all-to-all)
// through a caller-provided workspace, and the host-buffer wrapper around the fused kernel.
#include "common.cuh"

int basp_attn_dispatch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                       void *const *o, float *const *lse, float scale, bool fused, void *stream);

namespace {
size_t q_shard_bytes(const basp_plan *p) { return (size_t)p->Bl * p->T * p->Hq * p->D * 2; }
size_t kv_shard_bytes(const basp_plan *p) { return (size_t)p->Bl * p->T * p->Hkv * p->D * 2; }
}  // namespace

extern "C" size_t basp_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    return (size_t)p->N * (2 * q_shard_bytes(p) + 2 * kv_shard_bytes(p));   // head-sharded Q, K, V, O
}

extern "C" size_t basp_host_arena_bytes(const basp_plan *p) { return basp_workspace_bytes(p); }

extern "C" int basp_layer_fwd(const basp_plan *p, const void *const *q_seq, const void *const *k_seq,
                              const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                              void *workspace, size_t workspace_bytes, float softmax_scale, void *stream) {
    if (!p || !workspace) return BASP_ERR_NULL;
    if (!aligned16(workspace)) return BASP_ERR_ALIGN;
    if (workspace_bytes < basp_workspace_bytes(p)) return BASP_ERR_WORKSPACE;
    char *w = (char *)workspace;
    void *qh[BASP_MAX_RANKS], *kh[BASP_MAX_RANKS], *vh[BASP_MAX_RANKS], *oh[BASP_MAX_RANKS];
    const size_t qb = q_shard_bytes(p), kb = kv_shard_bytes(p);
    for (int r = 0; r < p->N; ++r) {
        qh[r] = w + (size_t)r * qb;
        kh[r] = w + (size_t)p->N * qb + (size_t)r * kb;
        vh[r] = w + (size_t)p->N * (qb + kb) + (size_t)r * kb;
        oh[r] = w + (size_t)p->N * (qb + 2 * kb) + (size_t)r * qb;
    }
    int rc = basp_reshard_qkv_s2h(p, q_seq, k_seq, v_seq, qh, kh, vh, stream);
    if (rc != BASP_OK) return rc;
    rc = basp_attn_dispatch(p, qh, kh, vh, oh, lse_shards, softmax_scale, false, stream);
    if (rc != BASP_OK) return rc;
    return basp_reshard_h2s(p, p->Hq, oh, o_seq, stream);
}

extern "C" int basp_layer_workspace_shards(const basp_plan *p, void *workspace, void **q_head, void **k_head,
                                           void **v_head, void **o_head) {
    if (!p || !workspace || !q_head || !k_head || !v_head || !o_head) return BASP_ERR_NULL;
    char *w = (char *)workspace;
    const size_t qb = q_shard_bytes(p), kb = kv_shard_bytes(p);
    for (int r = 0; r < p->N; ++r) {
        q_head[r] = w + (size_t)r * qb;
        k_head[r] = w + (size_t)p->N * qb + (size_t)r * kb;
        v_head[r] = w + (size_t)p->N * (qb + kb) + (size_t)r * kb;
        o_head[r] = w + (size_t)p->N * (qb + 2 * kb) + (size_t)r * qb;
    }
    return BASP_OK;
}

extern "C" size_t basp_layer_bwd_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    // head-sharded dO and dQ (query-sized), dK and dV (key-sized), then the attention-backward workspace
    return (size_t)p->N * (2 * q_shard_bytes(p) + 2 * kv_shard_bytes(p)) + basp_attn_bwd_workspace_bytes(p);
}

extern "C" int basp_layer_bwd(const basp_plan *p, const void *const *q_head, const void *const *k_head,
                              const void *const *v_head, const void *const *o_head, const float *const *lse_shards,
                              const void *const *do_seq, void *const *dq_seq, void *const *dk_seq,
                              void *const *dv_seq, void *workspace, size_t workspace_bytes, float softmax_scale,
                              void *stream) {
    if (!p || !workspace) return BASP_ERR_NULL;
    if (!aligned16(workspace)) return BASP_ERR_ALIGN;
    if (workspace_bytes < basp_layer_bwd_workspace_bytes(p)) return BASP_ERR_WORKSPACE;
    char *w = (char *)workspace;
    void *doh[BASP_MAX_RANKS], *dqh[BASP_MAX_RANKS], *dkh[BASP_MAX_RANKS], *dvh[BASP_MAX_RANKS];
    const size_t qb = q_shard_bytes(p), kb = kv_shard_bytes(p);
    for (int r = 0; r < p->N; ++r) {
        doh[r] = w + (size_t)r * qb;
        dqh[r] = w + (size_t)p->N * qb + (size_t)r * qb;
        dkh[r] = w + (size_t)p->N * 2 * qb + (size_t)r * kb;
        dvh[r] = w + (size_t)p->N * (2 * qb + kb) + (size_t)r * kb;
    }
    char *bwd_ws = w + (size_t)p->N * (2 * qb + 2 * kb);
    int rc = basp_reshard_s2h(p, p->Hq, do_seq, doh, stream);
    if (rc != BASP_OK) return rc;
    rc = basp_attn_bwd(p, q_head, k_head, v_head, o_head, doh, lse_shards, dqh, dkh, dvh, bwd_ws,
                       workspace_bytes - (size_t)(bwd_ws - w), softmax_scale, stream);
    if (rc != BASP_OK) return rc;
    return basp_reshard_grads_h2s(p, dqh, dkh, dvh, dq_seq, dk_seq, dv_seq, stream);
}

extern "C" int basp_layer_fwd_host(const basp_plan *p, const void *const *q_seq_host, const void *const *k_seq_host,
                                   const void *const *v_seq_host, void *const *o_seq_host, void *device_arena,
                                   size_t arena_bytes, float softmax_scale, void *stream) {
    if (!p || !q_seq_host || !k_seq_host || !v_seq_host || !o_seq_host || !device_arena) return BASP_ERR_NULL;
    if (!aligned16(device_arena)) return BASP_ERR_ALIGN;
    if (arena_bytes < basp_host_arena_bytes(p)) return BASP_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char *w = (char *)device_arena;
    void *qd[BASP_MAX_RANKS], *kd[BASP_MAX_RANKS], *vd[BASP_MAX_RANKS], *od[BASP_MAX_RANKS];
    const size_t qb = q_shard_bytes(p), kb = kv_shard_bytes(p);
    for (int r = 0; r < p->N; ++r) {
        if (!q_seq_host[r] || !k_seq_host[r] || !v_seq_host[r] || !o_seq_host[r]) return BASP_ERR_NULL;
        qd[r] = w + (size_t)r * qb;
        kd[r] = w + (size_t)p->N * qb + (size_t)r * kb;
        vd[r] = w + (size_t)p->N * (qb + kb) + (size_t)r * kb;
        od[r] = w + (size_t)p->N * (qb + 2 * kb) + (size_t)r * qb;
        BASP_CUDA_TRY(cudaMemcpyAsync(qd[r], q_seq_host[r], qb, cudaMemcpyHostToDevice, st));
        BASP_CUDA_TRY(cudaMemcpyAsync(kd[r], k_seq_host[r], kb, cudaMemcpyHostToDevice, st));
        BASP_CUDA_TRY(cudaMemcpyAsync(vd[r], v_seq_host[r], kb, cudaMemcpyHostToDevice, st));
    }
    int rc = basp_attn_dispatch(p, qd, kd, vd, od, nullptr, softmax_scale, true, stream);
    if (rc != BASP_OK) return rc;
    for (int r = 0; r < p->N; ++r)
        BASP_CUDA_TRY(cudaMemcpyAsync(o_seq_host[r], od[r], qb, cudaMemcpyDeviceToHost, st));
    BASP_CUDA_TRY(cudaStreamSynchronize(st));
    return BASP_OK;
}
