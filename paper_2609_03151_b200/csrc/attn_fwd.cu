// Causal attention over each virtual rank's head slice (Section II-A equation, evaluated
// tile by tile with an online softmax as in the FlashAttention technique the paper cites),
// on tcgen05 tensor cores with TMEM accumulators and TMA-fed shared memory.
//
// The same kernel serves two addressings of its operands:
//   head-sharded  rank r holds [Bl][S][H/K][D]; tile (bl, s0, h) is rows bl*S+s0.. of rank r
//   fused         operands stay SEQUENCE-sharded [Bl][T][H][D]; the tile at sequence position
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

static int g_attn_variant = 0;
extern "C" void basp_debug_set_attn_variant(int v) { g_attn_variant = v; }
#ifdef BASP_PHASE_TIMING
extern "C" int basp_debug_trace(long long *out) {
    return cudaMemcpyFromSymbol(out, g_trace, sizeof(long long) * 4 * 256) == cudaSuccess ? 0 : -1;
}
extern "C" int basp_debug_phases(long long *out, int reset) {
    if (out && cudaMemcpyFromSymbol(out, g_phase_cycles, sizeof(long long) * 64) != cudaSuccess) return -1;
    if (reset) { long long z[64] = {0}; if (cudaMemcpyToSymbol(g_phase_cycles, z, sizeof(z)) != cudaSuccess) return -1; }
    return 0;
}
#endif

namespace {

// ---------------------------------------------------------------------------------------
// Baseline kernel: one CTA of 128 threads per (q tile, head, sequence); every step in order.
template <int D, int R>
__global__ void __launch_bounds__(128) attn_fwd_simple_kernel(const __grid_constant__ AttnParams<R> p) {
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kTile * D * 2;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem, *sK = smem + kTileBytes, *sV = smem + 2 * kTileBytes;
    __shared__ uint64_t bar_q, bar_kv, bar_s, bar_o;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int n_qt = p.S / kTile;
    const int qt = n_qt - 1 - (int)blockIdx.x;          // longest tiles first
    const int h = blockIdx.y;
    const int r = blockIdx.z / p.Bl, bl = blockIdx.z - r * p.Bl;
    const int hkv = h / p.q_per_kv;
    const int n_kv = p.causal ? qt + 1 : n_qt;

    if (tid == 0) {
        mbar_init(&bar_q, 1); mbar_init(&bar_kv, 1); mbar_init(&bar_s, 1); mbar_init(&bar_o, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_base_s, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    const uint32_t S_t = tmem, O_t = tmem + 128, P_t = tmem;   // P (bf16) overlays S columns 0..63
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;

    if (tid == 0) {
        const TileCoord c = locate(p, r, bl, qt * kTile, h, p.Hq_l);
        mbar_arrive_expect_tx(&bar_q, kTileBytes);
        for (int s = 0; s < kSlabs; ++s) tma_load_3d(sQ + s * 16384, &p.q[c.rank], &bar_q, s * 64, c.head, c.row);
    }

    float m_run = -INFINITY, l_run = 0.f;
    const int row_in_tile = tid;
    bool ok = true;

    for (int j = 0; j < n_kv && ok; ++j) {
        const uint32_t ph = j & 1;
        if (tid == 0) {
            const TileCoord c = locate(p, r, bl, j * kTile, hkv, p.Hkv_l);
            mbar_arrive_expect_tx(&bar_kv, 2 * kTileBytes);
            for (int s = 0; s < kSlabs; ++s) {
                tma_load_3d(sK + s * 16384, &p.k[c.rank], &bar_kv, s * 64, c.head, c.row);
                tma_load_3d(sV + s * 16384, &p.v[c.rank], &bar_kv, s * 64, c.head, c.row);
            }
            ok = (j > 0 || mbar_wait(&bar_q, 0, &abort_flag)) && mbar_wait(&bar_kv, ph, &abort_flag);
            if (ok) {
                tc_fence_after();
                const uint32_t idesc = make_idesc_bf16(kTile, kTile, false, false);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * 16384 + (kk % 4) * 32;
                    mma_ss(S_t, make_smem_desc_sw128(smem_u32(sQ) + off, 16, 1024),
                           make_smem_desc_sw128(smem_u32(sK) + off, 16, 1024), idesc, kk > 0);
                }
                tc_commit(&bar_s);
            } else {
                abort_flag = 1;
                report(p.status, 1, 0, j);
            }
        }
        ok = mbar_wait(&bar_s, ph, &abort_flag);
        if (!ok) { abort_flag = 1; report(p.status, 1, 1, j); }
        if (__syncthreads_or(!ok)) { ok = false; break; }
        tc_fence_after();

        // ---- online softmax of this thread's row
        float s[kTile];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t rr[32];
            tmem_ld_x32(S_t + lane_addr + c * 32, rr);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(rr[i]) * p.scale_log2;
        }
        if (p.causal && j == qt) {
#pragma unroll
            for (int i = 0; i < kTile; ++i)
                if (i > row_in_tile) s[i] = -INFINITY;
        }
        float m_new = m_run;
#pragma unroll
        for (int i = 0; i < kTile; ++i) m_new = fmaxf(m_new, s[i]);
        const float alpha = exp2_approx(m_run - m_new);
        float rs = 0.f;
#pragma unroll
        for (int i = 0; i < kTile; ++i) { s[i] = exp2_approx(s[i] - m_new); rs += s[i]; }
        l_run = l_run * alpha + rs;
        m_run = m_new;
        // rescale the accumulator (skipped while no row of the warp moved its maximum)
        if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t rr[32];
                tmem_ld_x32(O_t + lane_addr + c * 32, rr);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) rr[i] = __float_as_uint(__uint_as_float(rr[i]) * alpha);
                tmem_st_x32(O_t + lane_addr + c * 32, rr);
            }
        }
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t rr[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) rr[i] = pack_bf16x2(s[c * 64 + 2 * i], s[c * 64 + 2 * i + 1]);
            tmem_st_x32(P_t + lane_addr + c * 32, rr);
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const uint32_t idesc = make_idesc_bf16(kTile, D, false, true);
#pragma unroll
            for (int kk = 0; kk < kTile / 16; ++kk)
                mma_ts(O_t, P_t + kk * 8, make_smem_desc_sw128(smem_u32(sV) + kk * 2048, 16384, 1024), idesc,
                       (j > 0) || (kk > 0));
            tc_commit(&bar_o);
        }
        ok = mbar_wait(&bar_o, ph, &abort_flag);
        if (!ok) { abort_flag = 1; report(p.status, 1, 2, j); }
        if (__syncthreads_or(!ok)) { ok = false; break; }
        tc_fence_after();
    }

    if (ok) {
        const TileCoord c = locate(p, r, bl, qt * kTile, h, p.Hq_l);
        const float inv_l = 1.f / l_run;
        __nv_bfloat16 *dst = p.o[c.rank] + ((size_t)(c.row + row_in_tile) * p.o_heads + c.head) * D;
#pragma unroll
        for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t rr[32];
            tmem_ld_x32(O_t + lane_addr + cc * 32, rr);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 o4;
                o4.x = pack_bf16x2(__uint_as_float(rr[8 * i + 0]) * inv_l, __uint_as_float(rr[8 * i + 1]) * inv_l);
                o4.y = pack_bf16x2(__uint_as_float(rr[8 * i + 2]) * inv_l, __uint_as_float(rr[8 * i + 3]) * inv_l);
                o4.z = pack_bf16x2(__uint_as_float(rr[8 * i + 4]) * inv_l, __uint_as_float(rr[8 * i + 5]) * inv_l);
                o4.w = pack_bf16x2(__uint_as_float(rr[8 * i + 6]) * inv_l, __uint_as_float(rr[8 * i + 7]) * inv_l);
                *reinterpret_cast<uint4 *>(dst + cc * 32 + i * 8) = o4;
            }
        }
        if (p.has_lse)
            p.lse[r][((size_t)bl * p.Hq_l + h) * p.S + qt * kTile + row_in_tile] =
                m_run * 0.6931471805599453f + logf(l_run);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

template <int R>
int fill_and_launch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                    void *const *o, float *const *lse, float scale, bool fused, cudaStream_t st) {
    AttnParams<R> prm;
    const uint64_t rows = (uint64_t)pl->Bl * (fused ? pl->T : pl->S);
    const int hq = fused ? pl->Hq : pl->Hq_l, hkv = fused ? pl->Hkv : pl->Hkv_l;
    for (int r = 0; r < pl->N; ++r) {
        int rc = tmap::encode_rows_heads_d(&prm.q[r], q[r], rows, hq, pl->D, kTile);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.k[r], k[r], rows, hkv, pl->D, kTile);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.v[r], v[r], rows, hkv, pl->D, kTile);
        if (rc != BASP_OK) return rc;
        prm.o[r] = (__nv_bfloat16 *)o[r];
        prm.lse[r] = lse ? lse[r] : nullptr;
    }
    prm.n_ranks = pl->N; prm.K = pl->K; prm.Bl = pl->Bl; prm.S = pl->S; prm.T = pl->T;
    prm.Hq_l = pl->Hq_l; prm.Hkv_l = pl->Hkv_l; prm.q_per_kv = pl->Hq / pl->Hkv;
    prm.o_heads = hq;
    {
        const int n_qb = (pl->S / kTile + 1) / 2, q_per_kv = pl->Hq / pl->Hkv;
        int band = 16 / q_per_kv < 1 ? 1 : (16 / q_per_kv > 8 ? 8 : 16 / q_per_kv);
        while (n_qb % band != 0) --band;
        prm.qb_band = band;
    }
    prm.fused = fused; prm.causal = pl->causal; prm.has_lse = lse != nullptr;
    prm.scale_log2 = (scale == 0.f ? 1.f / sqrtf((float)pl->D) : scale) * 1.4426950408889634f;
    prm.status = basp_status_device_ptr();
    if (!prm.status) return BASP_ERR_CUDA;

    if (g_attn_variant == 1) {      // baseline kernel (development comparison only)
        dim3 grid(pl->S / kTile, pl->Hq_l, pl->N * pl->Bl);
        if (pl->D == 128) {
            const int smem = 3 * kTile * 128 * 2 + 1024;
            BASP_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_simple_kernel<128, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attn_fwd_simple_kernel<128, R><<<grid, 128, smem, st>>>(prm);
        } else {
            const int smem = 3 * kTile * 64 * 2 + 1024;
            BASP_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_simple_kernel<64, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attn_fwd_simple_kernel<64, R><<<grid, 128, smem, st>>>(prm);
        }
    } else {
        int dev = 0, sms = 0;
        BASP_CUDA_TRY(cudaGetDevice(&dev));
        BASP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        const long long items = (long long)((pl->S / kTile + 1) / 2) * pl->N * pl->Bl * pl->Hq_l;
        const int grid = (int)(items < sms ? items : sms);
        if (pl->D == 128) {
            const int smem = (2 + kStages) * kTile * 128 * 2 + 1024;
            BASP_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_ws_kernel<128, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attn_fwd_ws_kernel<128, R><<<grid, kWsThreads, smem, st>>>(prm);
        } else {
            const int smem = (2 + kStages) * kTile * 64 * 2 + 1024;
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
int basp_attn_dispatch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
                       void *const *o, float *const *lse, float scale, bool fused, void *stream) {
    if (!pl || !q || !k || !v || !o) return BASP_ERR_NULL;
    if ((pl->D != 64 && pl->D != 128) || pl->S % kTile != 0) return BASP_ERR_UNSUPPORTED;
    if (fused && pl->T % kTile != 0) return BASP_ERR_UNSUPPORTED;
    if ((size_t)pl->N * pl->Bl > 65535 || pl->Hq_l > 65535) return BASP_ERR_UNSUPPORTED;
    for (int r = 0; r < pl->N; ++r) {
        if (!q[r] || !k[r] || !v[r] || !o[r] || (lse && !lse[r])) return BASP_ERR_NULL;
        if (!aligned16(q[r]) || !aligned16(k[r]) || !aligned16(v[r]) || !aligned16(o[r]) || (lse && ((uintptr_t)lse[r] & 3)))
            return BASP_ERR_ALIGN;
        for (int r2 = 0; r2 < pl->N; ++r2)
            if (o[r] == q[r2] || o[r] == k[r2] || o[r] == v[r2]) return BASP_ERR_ALIAS;
    }
    if (pl->N <= 8) return fill_and_launch<8>(pl, q, k, v, o, lse, scale, fused, (cudaStream_t)stream);
    return fill_and_launch<BASP_MAX_RANKS>(pl, q, k, v, o, lse, scale, fused, (cudaStream_t)stream);
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
