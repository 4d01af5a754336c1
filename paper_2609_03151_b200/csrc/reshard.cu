// Group-local all-to-alls of the Ulysses layer (Section II-C, Section IV-C) as in-HBM
// permutations between N virtual ranks.
//
//   s2h: head[gK+m][bl][s][h'][d] = seq[gK + s/T][bl][s mod T][m*H/K + h'][d]
//   h2s: the inverse map.
// (T = ceil(S/K); where K does not divide S the last rank of a group holds the short remainder, a compact shard.)
//
// The unit moved is a 16-byte vector.  Walking the SEQUENCE-sharded side in memory order, a
// token row of H*D elements is K consecutive runs of (H/K)*D elements, run m belonging to
// local rank m of the group; on the head-sharded side each run is contiguous too.  So both
// sides are touched in runs of >= 256 bytes and every 128-byte line is moved whole.  One
// launch covers up to three tensors (Q, K, V) of all ranks.
//
// HBM-bound: 2 bytes of traffic per byte of tensor, no arithmetic.  Each thread keeps U
// independent 16-byte streaming loads in flight before its stores.
#include <cuda_bf16.h>

#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 8;                       // vectors per thread and chunk
constexpr uint32_t kChunkV = kThreads * kUnroll; // 32 KiB per CTA

struct ReshardTensor {
    const char *seq[BASP_MAX_RANKS];
    const char *head[BASP_MAX_RANKS];
    uint32_t row_v;            // vectors per token row on the sequence-sharded side (K runs)
    uint32_t run_v;            // vectors per run = (H/K)*D*2/16 (one head when replicated)
    uint32_t rep;              // head-side ranks that receive each run (1; K/H when a group has more ranks than heads)
    uint32_t shard_v;          // vectors per rank shard (of T tokens; a short last rank has fewer)
    uint32_t chunks_per_shard;
    uint32_t chunk_begin;      // first CTA index of this tensor
    FastDiv div_row, div_run;
};

struct ReshardParams {
    int n_tensors;
    uint32_t r_begin, r_count; // sequence-side ranks this launch walks
    uint32_t K, T, S, Bl;
    uint32_t T_last;           // tokens per sequence of a group's last rank (= T when K divides S)
    FastDiv div_T, div_T_last;
    ReshardTensor t[3];
};

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// kToHead = true: s2h (read the sequence side in order, scatter runs to the head side);
// false: h2s (gather runs from the head side, write the sequence side in order).
template <bool kToHead>
__global__ void __launch_bounds__(kThreads) reshard_kernel(const __grid_constant__ ReshardParams p) {
    uint32_t c = blockIdx.x;
    int ti = 0;
    while (ti + 1 < p.n_tensors && c >= p.t[ti + 1].chunk_begin) ++ti;
    const ReshardTensor &t = p.t[ti];
    c -= t.chunk_begin;
    const uint32_t ri = c / t.chunks_per_shard;
    const uint32_t chunk = c - ri * t.chunks_per_shard;
    const uint32_t r = p.r_begin + ri;
    const uint32_t g = r / p.K, l = r - g * p.K;
    const uint32_t v0 = chunk * kChunkV + threadIdx.x;
    const bool last = l == p.K - 1;
    const uint32_t Tr = last ? p.T_last : p.T;                       // this rank's tokens per sequence
    const FastDiv div_Tr = last ? p.div_T_last : p.div_T;
    const uint32_t shard_v = last ? p.Bl * Tr * t.row_v : t.shard_v;

    const uint4 *seq = reinterpret_cast<const uint4 *>(t.seq[r]);
    const uint4 *hp[kUnroll];   // address on the head-sharded side of each vector (of its first copy when replicated)
    uint32_t hrank[kUnroll], hoff[kUnroll];
#pragma unroll
    for (int i = 0; i < kUnroll; ++i) {
        const uint32_t v = v0 + i * kThreads;
        const uint32_t vv = v < shard_v ? v : 0;
        const uint32_t tok = fdiv(vv, t.div_row);          // (bl, t) flattened
        const uint32_t col = vv - tok * t.row_v;
        const uint32_t m = fdiv(col, t.div_run);           // destination local rank
        const uint32_t j = col - m * t.run_v;
        const uint32_t bl = fdiv(tok, div_Tr);
        const uint32_t tt = tok - bl * Tr;
        const uint32_t hv = (bl * p.S + l * p.T + tt) * t.run_v + j;
        hrank[i] = g * p.K + m * t.rep;
        hoff[i] = hv;
        hp[i] = reinterpret_cast<const uint4 *>(t.head[hrank[i]]) + hv;
    }
    uint4 data[kUnroll];
#pragma unroll
    for (int i = 0; i < kUnroll; ++i) {
        const uint32_t v = v0 + i * kThreads;
        if (v < shard_v) data[i] = ld_stream(kToHead ? seq + v : hp[i]);
    }
    if (!kToHead && t.rep > 1) {
        // The way back of a replicated tensor carries gradients: every copy holds the contribution of its own rank's
        // query heads, the owner gets their sum (added in fp32, rounded to bf16 once).
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const uint32_t v = v0 + i * kThreads;
            if (v >= shard_v) continue;
            float acc[8];
            const uint32_t w0[4] = {data[i].x, data[i].y, data[i].z, data[i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) { acc[2 * e] = __uint_as_float(w0[e] << 16); acc[2 * e + 1] = __uint_as_float(w0[e] & 0xffff0000u); }
            for (uint32_t c = 1; c < t.rep; ++c) {
                const uint4 d = ld_stream(reinterpret_cast<const uint4 *>(t.head[hrank[i] + c]) + hoff[i]);
                const uint32_t wc[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) { acc[2 * e] += __uint_as_float(wc[e] << 16); acc[2 * e + 1] += __uint_as_float(wc[e] & 0xffff0000u); }
            }
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[2 * e], acc[2 * e + 1]);
                o[e] = *reinterpret_cast<const uint32_t *>(&b2);
            }
            data[i] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
#pragma unroll
    for (int i = 0; i < kUnroll; ++i) {
        const uint32_t v = v0 + i * kThreads;
        if (v < shard_v) st_stream(const_cast<uint4 *>(kToHead ? hp[i] : seq + v), data[i]);
    }
    if (kToHead && t.rep > 1) {         // the other local ranks that read this KV head get the same run
        for (uint32_t c = 1; c < t.rep; ++c)
#pragma unroll
            for (int i = 0; i < kUnroll; ++i) {
                const uint32_t v = v0 + i * kThreads;
                if (v < shard_v)
                    st_stream(const_cast<uint4 *>(reinterpret_cast<const uint4 *>(t.head[hrank[i] + c]) + hoff[i]), data[i]);
            }
    }
}

struct TensorArg {
    int n_heads;
    const void *const *seq;
    const void *const *head;
};

int fill_tensor(const basp_plan *p, const TensorArg &a, bool to_head, int r_begin, int r_count, ReshardTensor *t,
                uint32_t *chunk_cursor) {
    if (!a.seq || !a.head) return BASP_ERR_NULL;
    if (a.n_heads <= 0) return BASP_ERR_INVALID;
    // fewer heads than ranks in a group (KV heads under GQA): every head goes to K/H consecutive local ranks
    const int rep = a.n_heads % p->K == 0 ? 1 : (p->K % a.n_heads == 0 ? p->K / a.n_heads : 0);
    if (rep == 0) return BASP_ERR_INVALID;
    const size_t run_bytes = (rep > 1 ? (size_t)1 : (size_t)(a.n_heads / p->K)) * p->D * 2;
    if (run_bytes % 16 != 0) return BASP_ERR_UNSUPPORTED;
    const size_t shard_bytes = (size_t)p->Bl * p->T * a.n_heads * p->D * 2;                 // sequence side
    const size_t head_bytes = rep > 1 ? (size_t)p->Bl * p->S * p->D * 2 : shard_bytes;          // head side
    if (head_bytes / 16 >= (1ull << 31)) return BASP_ERR_UNSUPPORTED;
    // The launch walks the sequence-side shards of ranks [r_begin, r_begin + r_count) and touches the head-side
    // shards of every member of their groups; the other entries are not read (they may be NULL).
    const int g_begin = r_begin / p->K * p->K, g_end = (r_begin + r_count + p->K - 1) / p->K * p->K;
    for (int r = 0; r < p->N; ++r) {
        const bool need_seq = r >= r_begin && r < r_begin + r_count, need_head = r >= g_begin && r < g_end;
        t->seq[r] = need_seq ? (const char *)a.seq[r] : nullptr;
        t->head[r] = need_head ? (const char *)a.head[r] : nullptr;
        if ((need_seq && !a.seq[r]) || (need_head && !a.head[r])) return BASP_ERR_NULL;
        if ((need_seq && !aligned16(a.seq[r])) || (need_head && !aligned16(a.head[r]))) return BASP_ERR_ALIGN;
    }
    // out-of-place only: no destination shard may overlap a source shard.  The head side's extent is exact (whole
    // sequences of S tokens: smaller than Bl*T*H*D where the group size does not divide S), so a buffer that starts
    // right behind the last head shard is not taken for an overlap.
    const size_t head_extent = (size_t)p->Bl * p->S * (rep > 1 ? (size_t)1 : (size_t)(a.n_heads / p->K)) * p->D * 2;
    for (int i = r_begin; i < r_begin + r_count; ++i)
        for (int j = g_begin; j < g_end; ++j) {
            const char *s = t->seq[i], *d = t->head[j];
            const size_t seq_bytes = shard_bytes / p->T * basp_rank_tokens(p, i % p->K);
            if (s < d + head_extent && d < s + seq_bytes) return BASP_ERR_ALIAS;
        }
    t->rep = (uint32_t)rep;
    t->run_v = (uint32_t)(run_bytes / 16);
    t->row_v = t->run_v * (rep > 1 ? (uint32_t)a.n_heads : (uint32_t)p->K);
    t->shard_v = (uint32_t)(shard_bytes / 16);
    t->chunks_per_shard = (t->shard_v + kChunkV - 1) / kChunkV;
    t->chunk_begin = *chunk_cursor;
    t->div_row = make_fastdiv(t->row_v);
    t->div_run = make_fastdiv(t->run_v);
    *chunk_cursor += t->chunks_per_shard * (uint32_t)r_count;
    return BASP_OK;
}

int launch(const basp_plan *p, const TensorArg *args, int n, bool to_head, int r_begin, int r_count, void *stream) {
    if (!p) return BASP_ERR_NULL;
    if (r_count < 0) { r_begin = 0; r_count = p->N; }          // every rank
    if (r_begin < 0 || r_begin + r_count > p->N) return BASP_ERR_INVALID;
    if (r_count == 0) return BASP_OK;
    ReshardParams prm;
    prm.n_tensors = n;
    prm.r_begin = (uint32_t)r_begin; prm.r_count = (uint32_t)r_count;
    prm.K = p->K; prm.T = p->T; prm.S = p->S; prm.Bl = p->Bl; prm.T_last = p->T_last;
    prm.div_T = make_fastdiv((uint32_t)p->T);
    prm.div_T_last = make_fastdiv((uint32_t)p->T_last);
    uint32_t chunks = 0;
    for (int i = 0; i < n; ++i) {
        int rc = fill_tensor(p, args[i], to_head, r_begin, r_count, &prm.t[i], &chunks);
        if (rc != BASP_OK) return rc;
    }
    if (chunks == 0) return BASP_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (to_head) reshard_kernel<true><<<chunks, kThreads, 0, st>>>(prm);
    else         reshard_kernel<false><<<chunks, kThreads, 0, st>>>(prm);
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(1);
    return BASP_OK;
}

}  // namespace

extern "C" int basp_reshard_s2h(const basp_plan *plan, int n_heads, const void *const *seq_shards,
                                void *const *head_shards, void *stream) {
    TensorArg a{n_heads, seq_shards, (const void *const *)head_shards};
    return launch(plan, &a, 1, true, 0, -1, stream);
}

extern "C" int basp_reshard_h2s(const basp_plan *plan, int n_heads, const void *const *head_shards,
                                void *const *seq_shards, void *stream) {
    TensorArg a{n_heads, (const void *const *)seq_shards, head_shards};
    return launch(plan, &a, 1, false, 0, -1, stream);
}

extern "C" int basp_reshard_qkv_s2h(const basp_plan *plan, const void *const *q_seq,
                                    const void *const *k_seq, const void *const *v_seq,
                                    void *const *q_head, void *const *k_head, void *const *v_head,
                                    void *stream) {
    if (!plan) return BASP_ERR_NULL;
    TensorArg a[3] = {{plan->Hq, q_seq, (const void *const *)q_head},
                      {plan->Hkv, k_seq, (const void *const *)k_head},
                      {plan->Hkv, v_seq, (const void *const *)v_head}};
    return launch(plan, a, 3, true, 0, -1, stream);
}

extern "C" int basp_reshard_grads_h2s(const basp_plan *plan, const void *const *dq_head, const void *const *dk_head,
                                      const void *const *dv_head, void *const *dq_seq, void *const *dk_seq,
                                      void *const *dv_seq, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    TensorArg a[3] = {{plan->Hq, (const void *const *)dq_seq, dq_head},
                      {plan->Hkv, (const void *const *)dk_seq, dk_head},
                      {plan->Hkv, (const void *const *)dv_seq, dv_head}};
    return launch(plan, a, 3, false, 0, -1, stream);
}

// The same exchanges restricted to the sequence-side shards of ranks [rank_begin, rank_begin + rank_count): what ONE
// physical GPU launches when a group spans several GPUs and the other ranks' shards are peer memory.  s2h pushes
// this GPU's sequence shards into every group member's head shard; h2s pulls this GPU's sequence shards together.
extern "C" int basp_reshard_qkv_s2h_ranks(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                                          const void *const *v_seq, void *const *q_head, void *const *k_head,
                                          void *const *v_head, int rank_begin, int rank_count, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    if (rank_count < 0) return BASP_ERR_INVALID;
    TensorArg a[3] = {{plan->Hq, q_seq, (const void *const *)q_head},
                      {plan->Hkv, k_seq, (const void *const *)k_head},
                      {plan->Hkv, v_seq, (const void *const *)v_head}};
    return launch(plan, a, 3, true, rank_begin, rank_count, stream);
}

extern "C" int basp_reshard_h2s_ranks(const basp_plan *plan, int n_heads, const void *const *head_shards,
                                      void *const *seq_shards, int rank_begin, int rank_count, void *stream) {
    if (rank_count < 0) return BASP_ERR_INVALID;
    TensorArg a{n_heads, (const void *const *)seq_shards, head_shards};
    return launch(plan, &a, 1, false, rank_begin, rank_count, stream);
}
