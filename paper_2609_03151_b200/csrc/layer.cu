// Whole-layer entry points: the three-launch path (all-to-all, attention, reverse all-to-all)
// through a caller-provided workspace, and the host-buffer wrapper around the fused kernel.
#include "common.cuh"

#include <mutex>
#include <vector>

int basp_attn_dispatch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                       void *const *o, float *const *lse, float scale, bool fused, void *stream);
int basp_attn_dispatch_range(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                             void *const *o, float *const *lse, float scale, bool fused, const int *range,
                             void *stream, bool cta_per_item);

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
    if (!scale_ok(softmax_scale)) return BASP_ERR_INVALID;
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
    if (!scale_ok(softmax_scale)) return BASP_ERR_INVALID;
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
    if (!scale_ok(softmax_scale)) return BASP_ERR_INVALID;
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
constexpr int kHostCompStreams = 3;
// Copy streams and events of the host-buffer entry, created once per device (no device memory).
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr, comp[kHostCompStreams] = {};
    cudaEvent_t start = nullptr, done = nullptr, arrived[BASP_MAX_RANKS] = {}, computed[BASP_MAX_RANKS] = {};
    std::vector<cudaEvent_t> events;               // per piece: arrived, computed (grown on demand, kept)
    int reserve_events(size_t n) {
        while (events.size() < n) {
            cudaEvent_t e;
            BASP_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
            events.push_back(e);
        }
        return BASP_OK;
    }
};
constexpr int kHostPieceWaves = 2;
constexpr int kHostUpperEighths = 5;   // share of a group's pieces (from the end of the sequence) sent right behind its K and V
// Sustained attention rate over host-link rate of the machine this was tuned on (about 1.3 PFLOP/s over 50 GB/s).
constexpr double kHostBalanceFlopPerByte = 26e3;
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
        for (int i = 0; i < kHostCompStreams; ++i) BASP_CUDA_TRY(cudaStreamCreateWithFlags(&p.comp[i], cudaStreamNonBlocking));
        BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
        BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming));
        for (int i = 0; i < BASP_MAX_RANKS; ++i) {
            BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.arrived[i], cudaEventDisableTiming));
            BASP_CUDA_TRY(cudaEventCreateWithFlags(&p.computed[i], cudaEventDisableTiming));
        }
    }
    *out = &p;
    return BASP_OK;
}
}  // namespace

// Copies, kernels and read-backs are pipelined (copies in on one stream, kernels on a few internal streams, copies out
// on another; the caller's stream is joined before and after).  Bus and GPU need about the same time on the
// long-sequence shapes, so the order on the bus is chosen to start the GPU early and never let it run dry.  A group's
// K and V shards go first (a quarter of the bytes under GQA; every query row needs a prefix of them), then its Q rows
// in PIECES of a few 256-row query blocks from the END of the sequence down: under the causal mask a piece's arithmetic
// grows with its position, so the first pieces carry the most work per byte.  After the UPPER 5/8 of a group's pieces
// (most of its arithmetic) the next group's K and V and upper pieces follow, the backlog on the GPU covering the K/V
// transfer; the cheap lower pieces of a group travel between the next group's upper pieces (their O rows leave early
// instead of queueing behind the last byte), the last group's lower pieces come last: a short tail.
// One launch per piece (all ranks and heads of the group, the piece's query blocks, one CTA per work item so that
// consecutive launches fill each other's last wave) starts as soon as the piece is there, and its O rows are read back
// while later pieces run.
// Calls that overlap in time on one device share the internal streams and events: serialise them.
extern "C" int basp_layer_fwd_host(const basp_plan *p, const void *const *q_seq_host, const void *const *k_seq_host,
                                   const void *const *v_seq_host, void *const *o_seq_host, void *device_arena,
                                   size_t arena_bytes, float softmax_scale, void *stream) {
    if (!p || !q_seq_host || !k_seq_host || !v_seq_host || !o_seq_host || !device_arena) return BASP_ERR_NULL;
    if (!scale_ok(softmax_scale)) return BASP_ERR_INVALID;
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
    const bool by_piece = p->T % 256 == 0;     // a launch per piece of query blocks, else one per group
    // bytes of rank r's shards (the last rank of a group is short when K does not divide S)
    auto qbytes = [&](int r) { return qb / p->T * basp_rank_tokens(p, r % p->K); };
    auto kbytes = [&](int r) { return kb / p->T * basp_rank_tokens(p, r % p->K); };
    BASP_CUDA_TRY(cudaEventRecord(pipe->start, st));
    BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->in, pipe->start, 0));
    BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->out, pipe->start, 0));
    for (int i = 0; i < kHostCompStreams; ++i) BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->comp[i], pipe->start, 0));
    if (by_piece) {
        int dev = 0, sms = 0;
        BASP_CUDA_TRY(cudaGetDevice(&dev));
        BASP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        // Piece size: about kHostPieceWaves waves of work items (one item = two query tiles of one head), the shard cut evenly.
        const int qb_shard = p->T / 256, items_per_qb = p->K * p->Bl * p->Hq_l;
        int want = (kHostPieceWaves * sms + items_per_qb - 1) / items_per_qb;
        if (want < 1) want = 1;
        const int n_pc = (qb_shard + want - 1) / want, piece_qb = (qb_shard + n_pc - 1) / n_pc;
        const size_t row_bytes = (size_t)p->Hq * p->D * 2;
        // kv_upto: the group's K and V shards of local ranks <= kv_upto go on the bus ahead of this piece (those not yet sent)
        struct Piece { int g, r, qb_begin, qb_count; size_t row0, rows; int kv_upto; };
        // Which side is the longer one decides the order.  The estimate needs the machine's balance (sustained
        // attention rate over host-link rate, FLOP per byte); it only chooses between two correct orders.
        const double flop = 4.0 * p->D * ((double)p->S * (p->S + 1) / (p->causal ? 2 : 1)) * p->Hq * p->B;
        const double bytes_in = (double)p->B * p->S * (p->Hq + 2.0 * p->Hkv) * p->D * 2;
        const bool gpu_bound = p->causal && flop > 1.25 * kHostBalanceFlopPerByte * bytes_in;
        std::vector<Piece> pieces, lower;
        for (int g = 0; g < p->G; ++g) {
            std::vector<Piece> mine;
            for (int l = p->K - 1; l >= 0; --l) {
                const int Tr = basp_rank_tokens(p, l), n_qb = (Tr + 255) / 256;
                for (int pc = (n_qb + piece_qb - 1) / piece_qb - 1; pc >= 0; --pc) {
                    Piece x;
                    x.g = g; x.r = g * p->K + l;
                    x.qb_begin = l * qb_shard + pc * piece_qb;
                    x.qb_count = n_qb - pc * piece_qb < piece_qb ? n_qb - pc * piece_qb : piece_qb;
                    x.row0 = (size_t)pc * piece_qb * 256;
                    x.rows = x.row0 + (size_t)x.qb_count * 256 > (size_t)Tr ? (size_t)Tr - x.row0 : (size_t)x.qb_count * 256;
                    x.kv_upto = gpu_bound ? l : p->K - 1;
                    mine.push_back(x);
                }
            }
            if (gpu_bound) {
                // The GPU is the longer side: get it going as early as possible and keep the bus ahead of it.  Shard by shard
                // from the START of the sequence (rows of local rank l need the K and V shards of ranks 0..l only), so the
                // first launch waits for one shard of K, V and a piece of Q; the cheap early rows overlap with the transfer
                // of the rest, and the backlog that builds up keeps the GPU busy to the end.
                for (int l = 0; l < p->K; ++l)
                    for (const Piece &x : mine)
                        if (x.r == g * p->K + l) pieces.push_back(x);
                continue;
            }
            // The bus is the longer side (or they balance): every group's pieces from the end of its sequences down; the
            // upper 5/8 of a group's pieces right behind its K and V, its lower pieces woven into the next group's upper
            // ones, the last group's lower pieces at the end.
            const size_t upper = p->causal ? (mine.size() * kHostUpperEighths + 7) / 8 : mine.size();
            // the previous group's cheap lower pieces travel between this group's upper pieces, one for one: their O rows
            // leave early instead of queueing on the way out behind the last byte
            size_t li = 0;
            for (size_t i = 0; i < upper; ++i) {
                pieces.push_back(mine[i]);
                if (li < lower.size()) pieces.push_back(lower[li++]);
            }
            pieces.insert(pieces.end(), lower.begin() + li, lower.end());
            lower.clear();
            lower.insert(lower.end(), mine.begin() + upper, mine.end());
        }
        pieces.insert(pieces.end(), lower.begin(), lower.end());
        rc = pipe->reserve_events(2 * pieces.size());
        if (rc != BASP_OK) return rc;
        // Rows [row0, row0 + rows) of every sequence of a shard: one contiguous slab per sequence.
        auto copy_rows = [&](void *dst, const void *src, const Piece &x, cudaMemcpyKind kind, cudaStream_t cs) -> int {
            const size_t pitch = (size_t)basp_rank_tokens(p, x.r % p->K) * row_bytes;
            for (int bl = 0; bl < p->Bl; ++bl) {
                const size_t off = (size_t)bl * pitch + x.row0 * row_bytes;
                BASP_CUDA_TRY(cudaMemcpyAsync((char *)dst + off, (const char *)src + off, x.rows * row_bytes, kind, cs));
            }
            return BASP_OK;
        };
        int kv_sent[BASP_MAX_RANKS];             // per group: local ranks whose K and V are on the bus already
        for (int g = 0; g < p->G; ++g) kv_sent[g] = 0;
        for (size_t i = 0; i < pieces.size(); ++i) {
            const Piece &x = pieces[i];
            for (; kv_sent[x.g] <= x.kv_upto; ++kv_sent[x.g]) {
                const int j = x.g * p->K + kv_sent[x.g];
                BASP_CUDA_TRY(cudaMemcpyAsync(kd[j], k_seq_host[j], kbytes(j), cudaMemcpyHostToDevice, pipe->in));
                BASP_CUDA_TRY(cudaMemcpyAsync(vd[j], v_seq_host[j], kbytes(j), cudaMemcpyHostToDevice, pipe->in));
            }
            rc = copy_rows(qd[x.r], q_seq_host[x.r], x, cudaMemcpyHostToDevice, pipe->in);
            if (rc != BASP_OK) return rc;
            BASP_CUDA_TRY(cudaEventRecord(pipe->events[2 * i], pipe->in));
        }
        for (size_t i = 0; i < pieces.size(); ++i) {
            const Piece &x = pieces[i];
            // The launches take turns on a few internal streams, so that the next piece's CTAs fill the SMs the
            // previous piece's last wave leaves idle.
            cudaStream_t cs = pipe->comp[i % kHostCompStreams];
            BASP_CUDA_TRY(cudaStreamWaitEvent(cs, pipe->events[2 * i], 0));      // implies the K and V shards it needs
            const int range[4] = {x.g * p->K, p->K, x.qb_begin, x.qb_count};
            rc = basp_attn_dispatch_range(p, qd, kd, vd, od, nullptr, softmax_scale, true, range, cs, true);
            if (rc != BASP_OK) return rc;
            BASP_CUDA_TRY(cudaEventRecord(pipe->events[2 * i + 1], cs));
            BASP_CUDA_TRY(cudaStreamWaitEvent(pipe->out, pipe->events[2 * i + 1], 0));
            rc = copy_rows(o_seq_host[x.r], od[x.r], x, cudaMemcpyDeviceToHost, pipe->out);
            if (rc != BASP_OK) return rc;
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
            rc = basp_attn_dispatch_range(p, qd, kd, vd, od, nullptr, softmax_scale, true, range, stream, false);
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
