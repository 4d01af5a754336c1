// Causal attention over each virtual rank's head slice (Section II-A equation, evaluated
// tile by tile with an online softmax as in the FlashAttention technique the paper cites),
// on tcgen05 tensor cores with TMEM accumulators and TMA-fed shared memory.
//
// The same kernel serves two addressings of its operands:
//   head-sharded  rank r holds [Bl][S][H/K][D]; tile (bl, s0, h) is rows bl*S+s0.. of rank r
//   fused         operands stay SEQUENCE-sharded [Bl][T][H][D] (T a multiple of the tile; the last rank of a group may
//                 hold fewer tokens); the tile at sequence position
//                 s0 of local head h lives on rank gK + s0/T, rows bl*T + s0 mod T, head l*H/K+h
//                 (the all-to-all of Section IV-C folded into the tile fetch / the O store).
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tmap.cuh"
#include "attn_common.cuh"
#include "attn_fwd_ws.cuh"

int *basp_status_device_ptr();

constexpr int kBandTarget = 32;   // CTAs that share one KV stream at a time (query blocks per band x query heads per KV head)

namespace {

template <int R>
int fill_and_launch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                    void *const *o, float *const *lse, float scale, bool fused, const int range[4], bool cta_per_item,
                    cudaStream_t st) {
    AttnParams<R> prm;
    const int hq = fused ? pl->Hq : pl->Hq_l, hkv = fused ? pl->Hkv : pl->Hkv_l;
    // Operands of ranks outside the launch's range are not touched: with head-sharded operands only the ranks of the
    // range, with sequence-sharded (fused) operands every member of their groups.
    const int need_lo = fused ? range[0] / pl->K * pl->K : range[0];
    const int need_hi = fused ? (range[0] + range[1] + pl->K - 1) / pl->K * pl->K : range[0] + range[1];
    for (int r = need_lo; r < need_hi; ++r) {
        const uint64_t rows = (uint64_t)pl->Bl * (fused ? basp_rank_tokens(pl, r % pl->K) : pl->S);
        int rc = tmap::encode_rows_heads_d(&prm.q[r], q[r], rows, hq, pl->D, kTile);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.k[r], k[r], rows, hkv, pl->D, kTile);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.v[r], v[r], rows, hkv, pl->D, kTile);
        if (rc != BASP_OK) return rc;
        prm.o[r] = (__nv_bfloat16 *)o[r];
        prm.lse[r] = lse ? lse[r] : nullptr;
    }
    prm.n_ranks = pl->N; prm.K = pl->K; prm.Bl = pl->Bl; prm.S = pl->S; prm.T = pl->T;
    prm.Hq_l = pl->Hq_l; prm.Hkv_l = pl->Hkv_l; prm.q_per_kv = pl->Hq_l / pl->Hkv_l;
    prm.kv_rep = pl->kv_rep;
    prm.o_heads = hq;
    prm.Dg = pl->D;
    {
        const int q_per_kv = pl->Hq_l / pl->Hkv_l;
        prm.r_begin = range[0]; prm.r_count = range[1]; prm.qb_begin = range[2]; prm.qb_count = range[3];
        int band = kBandTarget / q_per_kv < 1 ? 1 : (kBandTarget / q_per_kv > 16 ? 16 : kBandTarget / q_per_kv);
        while (prm.qb_count % band != 0) --band;
        prm.qb_band = band;
        prm.div_per_band = make_fastdiv((uint32_t)(range[1] * pl->Bl * pl->Hq_l * band));
        prm.div_per_stream = make_fastdiv((uint32_t)(band * q_per_kv));
        prm.div_q_per_kv = make_fastdiv((uint32_t)q_per_kv);
        prm.div_hkv_l = make_fastdiv((uint32_t)pl->Hkv_l);
        prm.div_bl = make_fastdiv((uint32_t)pl->Bl);
        prm.div_T = make_fastdiv((uint32_t)pl->T);
        prm.div_K = make_fastdiv((uint32_t)pl->K);
    }
    prm.fused = fused; prm.causal = pl->causal; prm.has_lse = lse != nullptr;
    prm.scale_log2 = (scale == 0.f ? 1.f / sqrtf((float)pl->D) : scale) * 1.4426950408889634f;
    prm.status = basp_status_device_ptr();
    if (!prm.status) return BASP_ERR_CUDA;

    {
        int dev = 0, sms = 0;
        BASP_CUDA_TRY(cudaGetDevice(&dev));
        BASP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        const long long items = (long long)range[3] * range[1] * pl->Bl * pl->Hq_l;
        // One persistent CTA per SM; a launch that shares the GPU with other launches (the pieces of the host-buffer
        // entry) takes one CTA per item instead and leaves the balancing to the hardware's block scheduler.
        const int grid = (int)(items < sms || (cta_per_item && items < (1 << 20)) ? items : sms);
        if (pl->D > 64) {        // 80 .. 128: the 128-wide kernel
            const int smem = (2 + kStages) * kTile * 128 * 2 + 1024;
            BASP_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_ws_kernel<128, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attn_fwd_ws_kernel<128, R><<<grid, kWsThreads, smem, st>>>(prm);
        } else {
            // every CTA holds all 512 TMEM columns: with more CTAs than SMs in flight, ask for enough shared memory that no
            // two share an SM (the second would only sit in its TMEM allocation until the first has left)
            const int smem = cta_per_item ? 120 * 1024 : (2 + kStages) * kTile * 64 * 2 + 1024;
            BASP_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_ws_kernel<64, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attn_fwd_ws_kernel<64, R><<<grid, kWsThreads, smem, st>>>(prm);
        }
    }
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(1);
    return BASP_OK;
}

}  // namespace

// Shared by basp_attn_fwd (head-sharded operands) and basp_layer_fwd_fused (sequence-sharded).
// `range` = {first rank, ranks, first 256-row query block, blocks} restricts the launch to a part of
// the work (NULL = everything); the host-buffer entry uses it to start on what has already arrived.
int basp_attn_dispatch_range(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                             void *const *o, float *const *lse, float scale, bool fused, const int *range,
                             void *stream, bool cta_per_item) {
    if (!pl || !q || !k || !v || !o) return BASP_ERR_NULL;
    // the kernel takes the row maximum of the raw scores and masks with -inf before it scales: a negative scale would pick
    // the wrong reference and turn masked keys into +inf
    if (!scale_ok(scale)) return BASP_ERR_INVALID;
    if (pl->D < 16 || pl->D > 128 || pl->D % 16 != 0) return BASP_ERR_UNSUPPORTED;
    if (fused && pl->T % kTile != 0) return BASP_ERR_UNSUPPORTED;
    // A short last shard (K does not divide S) holds its sequences T_last rows apart, the others T: the kernel's tile
    // addressing knows one distance only (this kernel's speed depends on its code layout; the extra select cost 5 % on
    // one of the benchmark shapes), so that case is served when a shard holds one sequence, as in BASP grouping.
    if (fused && pl->T_last != pl->T && pl->Bl > 1) return BASP_ERR_UNSUPPORTED;
    const int full[4] = {0, pl->N, 0, ((pl->S + kTile - 1) / kTile + 1) / 2};
    if (!range) range = full;
    if (range[0] < 0 || range[1] < 0 || range[0] + range[1] > pl->N) return BASP_ERR_INVALID;
    if (range[1] <= 0 || range[3] <= 0) return BASP_OK;
    const int need_lo = fused ? range[0] / pl->K * pl->K : range[0];
    const int need_hi = fused ? (range[0] + range[1] + pl->K - 1) / pl->K * pl->K : range[0] + range[1];
    for (int r = need_lo; r < need_hi; ++r) {
        const bool own = r >= range[0] && r < range[0] + range[1];       // LSE is written by the ranks of the range only
        if (!q[r] || !k[r] || !v[r] || !o[r] || (lse && own && !lse[r])) return BASP_ERR_NULL;
        if (!aligned16(q[r]) || !aligned16(k[r]) || !aligned16(v[r]) || !aligned16(o[r]) ||
            (lse && own && ((uintptr_t)lse[r] & 3)))
            return BASP_ERR_ALIGN;
        for (int r2 = need_lo; r2 < need_hi; ++r2)
            if (o[r] == q[r2] || o[r] == k[r2] || o[r] == v[r2]) return BASP_ERR_ALIAS;
    }
    if (pl->N <= 8) return fill_and_launch<8>(pl, q, k, v, o, lse, scale, fused, range, cta_per_item, (cudaStream_t)stream);
    return fill_and_launch<BASP_MAX_RANKS>(pl, q, k, v, o, lse, scale, fused, range, cta_per_item, (cudaStream_t)stream);
}

int basp_attn_dispatch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                       void *const *o, float *const *lse, float scale, bool fused, void *stream) {
    return basp_attn_dispatch_range(pl, q, k, v, o, lse, scale, fused, nullptr, stream, false);
}

extern "C" int basp_attn_fwd(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                             const void *const *v_head, void *const *o_head, float *const *lse_shards,
                             float softmax_scale, void *stream) {
    return basp_attn_dispatch(plan, q_head, k_head, v_head, o_head, lse_shards, softmax_scale, false, stream);
}

extern "C" int basp_layer_fwd_fused(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                                    const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                                    float softmax_scale, void *stream) {
    return basp_attn_dispatch(plan, q_seq, k_seq, v_seq, o_seq, lse_shards, softmax_scale, true, stream);
}

// One physical GPU's share when the N ranks are spread over several GPUs: only ranks [rank_begin, rank_begin +
// rank_count) compute.  Head-sharded operands of other ranks are not touched.  With sequence-sharded operands (fused)
// the tiles of the other members of the range's groups are fetched from wherever their pointers lead - peer memory
// mapped into this process included (plain TMA tile loads, every CTA fetching its own tile) - and O tiles are stored there with plain
// stores: the all-to-alls of Section IV-C and the attention in one kernel over NVLink.
extern "C" int basp_attn_fwd_ranks(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                                   const void *const *v_head, void *const *o_head, float *const *lse_shards,
                                   float softmax_scale, int rank_begin, int rank_count, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    const int range[4] = {rank_begin, rank_count, 0, ((plan->S + kTile - 1) / kTile + 1) / 2};
    return basp_attn_dispatch_range(plan, q_head, k_head, v_head, o_head, lse_shards, softmax_scale, false, range, stream, false);
}

extern "C" int basp_layer_fwd_fused_ranks(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                                          const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                                          float softmax_scale, int rank_begin, int rank_count, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    const int range[4] = {rank_begin, rank_count, 0, ((plan->S + kTile - 1) / kTile + 1) / 2};
    return basp_attn_dispatch_range(plan, q_seq, k_seq, v_seq, o_seq, lse_shards, softmax_scale, true, range, stream, false);
}
