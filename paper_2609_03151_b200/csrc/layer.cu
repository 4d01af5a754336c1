// Whole-layer entry points: the three-launch path (all-to-all, attention, reverse all-to-all)
// through a caller-provided workspace, and the host-buffer wrapper around the fused kernel.
#include "common.cuh"

#include <mutex>

int basp_attn_dispatch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                       void *const *o, float *const *lse, float scale, bool fused, void *stream);
int basp_attn_dispatch_range(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                             void *const *o, float *const *lse, float scale, bool fused, const int *range,
                             void *stream);

namespace {
size_t q_shard_bytes(const basp_plan *p) { return (size_t)p->Bl * p->T * p->Hq * p->D * 2; }
size_t kv_shard_bytes(const basp_plan *p) { return (size_t)p->Bl * p->T * p->Hkv * p->D * 2; }
// head-sharded Q (or O) of one rank: the same bytes as a sequence-sharded shard when K divides S
size_t q_head_bytes(const basp_plan *p) { return (size_t)p->Bl * p->S * p->Hq_l * p->D * 2; }
// head-sharded K or V of one rank: the same bytes unless KV heads are replicated inside the group
size_t kv_head_bytes(const basp_plan *p) { return (size_t)p->Bl * p->S * p->Hkv_l * p->D * 2; }
}  // namespace

extern "C" size_t basp_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    return (size_t)p->N * (2 * q_head_bytes(p) + 2 * kv_head_bytes(p));   // head-sharded Q, K, V, O
}

extern "C" size_t basp_host_arena_bytes(const basp_plan *p) {
    if (!p) return 0;
    return (size_t)p->N * (2 * q_shard_bytes(p) + 2 * kv_shard_bytes(p));  // sequence-sharded Q, K, V, O
}

extern "C" int basp_layer_fwd(const basp_plan *p, const void *const *q_seq, const void *const *k_seq,
                              const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                              void *workspace, size_t workspace_bytes, float softmax_scale, void *stream) {
    if (!p || !workspace) return BASP_ERR_NULL;
    if (!aligned16(workspace)) return BASP_ERR_ALIGN;
    if (workspace_bytes < basp_workspace_bytes(p)) return BASP_ERR_WORKSPACE;
    char *w = (char *)workspace;
    void *qh[BASP_MAX_RANKS], *kh[BASP_MAX_RANKS], *vh[BASP_MAX_RANKS], *oh[BASP_MAX_RANKS];
    const size_t qb = q_head_bytes(p), kb = kv_head_bytes(p);
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
    const size_t qb = q_head_bytes(p), kb = kv_head_bytes(p);
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
    return (size_t)p->N * (2 * q_head_bytes(p) + 2 * kv_head_bytes(p)) + basp_attn_bwd_workspace_bytes(p);
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
    const size_t qb = q_head_bytes(p), kb = kv_head_bytes(p);
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

extern "C" size_t basp_layer_bwd_seq_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    // head-sharded Q, O, dO, dQ (query-sized), K, V, dK, dV (key-sized), then the attention-backward workspace
    return (size_t)p->N * (4 * q_head_bytes(p) + 4 * kv_head_bytes(p)) + basp_attn_bwd_workspace_bytes(p);
}

extern "C" int basp_layer_bwd_seq(const basp_plan *p, const void *const *q_seq, const void *const *k_seq,
                                  const void *const *v_seq, const void *const *o_seq, const float *const *lse_shards,
                                  const void *const *do_seq, void *const *dq_seq, void *const *dk_seq,
                                  void *const *dv_seq, void *workspace, size_t workspace_bytes, float softmax_scale,
                                  void *stream) {
    if (!p || !workspace) return BASP_ERR_NULL;
    if (!aligned16(workspace)) return BASP_ERR_ALIGN;
    if (workspace_bytes < basp_layer_bwd_seq_workspace_bytes(p)) return BASP_ERR_WORKSPACE;
    char *w = (char *)workspace;
    void *qh[BASP_MAX_RANKS], *kh[BASP_MAX_RANKS], *vh[BASP_MAX_RANKS], *oh[BASP_MAX_RANKS], *doh[BASP_MAX_RANKS],
        *dqh[BASP_MAX_RANKS], *dkh[BASP_MAX_RANKS], *dvh[BASP_MAX_RANKS];
    const size_t qb = q_head_bytes(p), kb = kv_head_bytes(p);
    const size_t n = (size_t)p->N;
    for (int r = 0; r < p->N; ++r) {
        qh[r] = w + (size_t)r * qb;
        oh[r] = w + n * qb + (size_t)r * qb;
        doh[r] = w + n * 2 * qb + (size_t)r * qb;
        dqh[r] = w + n * 3 * qb + (size_t)r * qb;
        kh[r] = w + n * 4 * qb + (size_t)r * kb;
        vh[r] = w + n * (4 * qb + kb) + (size_t)r * kb;
        dkh[r] = w + n * (4 * qb + 2 * kb) + (size_t)r * kb;
        dvh[r] = w + n * (4 * qb + 3 * kb) + (size_t)r * kb;
    }
    char *bwd_ws = w + n * (4 * qb + 4 * kb);
    int rc = basp_reshard_qkv_s2h(p, q_seq, k_seq, v_seq, qh, kh, vh, stream);
    if (rc != BASP_OK) return rc;
    rc = basp_reshard_s2h(p, p->Hq, o_seq, oh, stream);
    if (rc != BASP_OK) return rc;
    rc = basp_reshard_s2h(p, p->Hq, do_seq, doh, stream);
    if (rc != BASP_OK) return rc;
    rc = basp_attn_bwd(p, qh, kh, vh, oh, doh, lse_shards, dqh, dkh, dvh, bwd_ws, workspace_bytes - (size_t)(bwd_ws - w),
                       softmax_scale, stream);
    if (rc != BASP_OK) return rc;
    return basp_reshard_grads_h2s(p, dqh, dkh, dvh, dq_seq, dk_seq, dv_seq, stream);
}

namespace {
// Copy streams and events of the host-buffer entry, created once per device (no device memory).
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, arrived[BASP_MAX_RANKS] = {}, computed[BASP_MAX_RANKS] = {};
    cudaEvent_t kv_arrived[BASP_MAX_RANKS] = {};   // per group
};
std::mutex g_pipe_mu;
HostPipe g_pipes[64];

int get_pipe(HostPipe **out) {
    int dev = -1;
    BASP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return BASP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_pipe_mu);
    HostPipe &p = g_pipes[dev];
    if (!p.in) {
        BASP_CUDA_TRY(cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking));
        BASP_CUDA_TRY(cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking));
        BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
        BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming));
        for (int i = 0; i < BASP_MAX_RANKS; ++i) {
            BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.arrived[i], cudaEventDisableTiming));
            BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.computed[i], cudaEventDisableTiming));
            BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.kv_arrived[i], cudaEventDisableTiming));
        }
    }
    *out = &p;
    return BASP_OK;
}
}  // namespace

// Copies, kernels and read-backs are pipelined (three streams: copies in, the caller's stream for the kernels,
// copies out).  The bus is the slow part, so the order of the copies is chosen to give the GPU its longest work
// first: a group's K and V shards (a quarter of the bytes under GQA) go ahead of its first Q shard, and the Q shards go
// from the LAST local rank down, the groups taking turns.  Under the causal mask the rows of local rank l cost
// (2l+1)/K^2 of the group's arithmetic, so the longest launches start first and the short ones follow while the
// rest is still on the bus; O shard l is read back as soon as its launch is done.
// Calls that overlap in time on one device share the internal streams and events: serialise them.
extern "C" int basp_layer_fwd_host(const basp_plan *p, const void *const *q_seq_host, const void *const *k_seq_host,
                                   const void *const *v_seq_host, void *const *o_seq_host, void *device_arena,
                                   size_t arena_bytes, float softmax_scale, void *stream) {
    if (!p || !q_seq_host || !k_seq_host || !v_seq_host || !o_seq_host || !device_arena) return BASP_ERR_NULL;
    if (!aligned16(device_arena)) return BASP_ERR_ALIGN;
    if (arena_bytes < basp_host_arena_bytes(p)) return BASP_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    HostPipe *pipe = nullptr;
    int rc = get_pipe(&pipe);
    if (rc != BASP_OK) return rc;
    char *w = (char *)device_arena;
    void *qd[BASP_MAX_RANKS], *kd[BASP_MAX_RANKS], *vd[BASP_MAX_RANKS], *od[BASP_MAX_RANKS];
    const size_t qb = q_shard_bytes(p), kb = kv_shard_bytes(p);
    for (int r = 0; r < p->N; ++r) {
        if (!q_seq_host[r] || !k_seq_host[r] || !v_seq_host[r] || !o_seq_host[r]) return BASP_ERR_NULL;
        qd[r] = w + (size_t)r * qb;
        kd[r] = w + (size_t)p->N * qb + (size_t)r * kb;
        vd[r] = w + (size_t)p->N * (qb + kb) + (size_t)r * kb;
        od[r] = w + (size_t)p->N * (qb + 2 * kb) + (size_t)r * qb;
    }
    const bool by_chunk = p->causal && p->T % 256 == 0;     // a launch per local rank's rows, else per group
    // bytes of rank r's shards (the last rank of a group is short when K does not divide S)
    auto qbytes = [&](int r) { return qb / p->T * basp_rank_tokens(p, r % p->K); };
    auto kbytes = [&](int r) { return kb / p->T * basp_rank_tokens(p, r % p->K); };
    BASP_CUDA_TRY(cudaEventRecord(pipe->start, st));
    BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->in, pipe->start, 0));
    BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->out, pipe->start, 0));
    if (by_chunk) {
        // Units (group, local rank) in the order: every group's LAST local rank first (after that group's K and V), then
        // the next-to-last of every group, and so on.  The longest launches are fed first and the groups alternate, so
        // the GPU is not left waiting for the second group's shards while the first group's short launches finish.
        for (int l = p->K - 1; l >= 0; --l)
            for (int g = 0; g < p->G; ++g) {
                const int r0 = g * p->K;
                if (l == p->K - 1) {
                    for (int j = 0; j < p->K; ++j) {
                        BASP_CUDA_TRY(cudaMemcpyAsync(kd[r0 + j], k_seq_host[r0 + j], kbytes(r0 + j), cudaMemcpyHostToDevice, pipe->in));
                        BASP_CUDA_TRY(cudaMemcpyAsync(vd[r0 + j], v_seq_host[r0 + j], kbytes(r0 + j), cudaMemcpyHostToDevice, pipe->in));
                    }
                }
                BASP_CUDA_TRY(cudaMemcpyAsync(qd[r0 + l], q_seq_host[r0 + l], qbytes(r0 + l), cudaMemcpyHostToDevice, pipe->in));
                BASP_CUDA_TRY(cudaEventRecord(pipe->arrived[r0 + l], pipe->in));
            }
        for (int l = p->K - 1; l >= 0; --l)
            for (int g = 0; g < p->G; ++g) {
                const int r0 = g * p->K;
                BASP_CUDA_TRY(cudaStreamWaitEvent(st, pipe->arrived[r0 + l], 0));   // implies the group's K and V
                const int range[4] = {r0, p->K, l * (p->T / 256), (basp_rank_tokens(p, l) + 255) / 256};
                rc = basp_attn_dispatch_range(p, qd, kd, vd, od, nullptr, softmax_scale, true, range, stream);
                if (rc != BASP_OK) return rc;
                BASP_CUDA_TRY(cudaEventRecord(pipe->computed[r0 + l], st));
                BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->out, pipe->computed[r0 + l], 0));
                BASP_CUDA_TRY(cudaMemcpyAsync(o_seq_host[r0 + l], od[r0 + l], qbytes(r0 + l), cudaMemcpyDeviceToHost, pipe->out));
            }
    } else {
        for (int g = 0; g < p->G; ++g) {
            const int r0 = g * p->K;
            for (int l = 0; l < p->K; ++l) {
                BASP_CUDA_TRY(cudaMemcpyAsync(kd[r0 + l], k_seq_host[r0 + l], kbytes(r0 + l), cudaMemcpyHostToDevice, pipe->in));
                BASP_CUDA_TRY(cudaMemcpyAsync(vd[r0 + l], v_seq_host[r0 + l], kbytes(r0 + l), cudaMemcpyHostToDevice, pipe->in));
                BASP_CUDA_TRY(cudaMemcpyAsync(qd[r0 + l], q_seq_host[r0 + l], qbytes(r0 + l), cudaMemcpyHostToDevice, pipe->in));
            }
            BASP_CUDA_TRY(cudaEventRecord(pipe->arrived[r0], pipe->in));
        }
        for (int g = 0; g < p->G; ++g) {
            const int r0 = g * p->K;
            BASP_CUDA_TRY(cudaStreamWaitEvent(st, pipe->arrived[r0], 0));
            const int range[4] = {r0, p->K, 0, ((p->S + 127) / 128 + 1) / 2};
            rc = basp_attn_dispatch_range(p, qd, kd, vd, od, nullptr, softmax_scale, true, range, stream);
            if (rc != BASP_OK) return rc;
            BASP_CUDA_TRY(cudaEventRecord(pipe->computed[r0], st));
            BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->out, pipe->computed[r0], 0));
            for (int l = 0; l < p->K; ++l)
                BASP_CUDA_TRY(cudaMemcpyAsync(o_seq_host[r0 + l], od[r0 + l], qbytes(r0 + l), cudaMemcpyDeviceToHost, pipe->out));
        }
    }
    BASP_CUDA_TRY(cudaEventRecord(pipe->done, pipe->out));
    BASP_CUDA_TRY(cudaStreamWaitEvent(st, pipe->done, 0));
    BASP_CUDA_TRY(cudaStreamSynchronize(st));
    return BASP_OK;
}
