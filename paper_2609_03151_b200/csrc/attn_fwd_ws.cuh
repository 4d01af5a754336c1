// Warp-specialised persistent attention kernel (one CTA of 512 threads per SM).
//
// A work item is one block of 256 query rows of one (rank, sequence, local head): two 128-row
// query tiles that share one stream of K/V tiles.  Roles:
//   warps  0-3   softmax of query tile 0      (one thread per score row)
//   warps  4-7   softmax of query tile 1
//   warps  8-11  correction: rescales the O accumulators in TMEM when a row's reference maximum
//                moved, and writes the normalised O tile at the end of the item
//   warp  12     TMA producer (Q tiles, then K_0 V_0 K_1 V_1 ... through a shared-memory ring)
//   warp  13     tcgen05.mma issuer for S = Q_t K_j^T (one thread)
//   warp  14     tcgen05.mma issuer for O_t += P_t V_j (one thread)
// TMEM: S | P_0 P_1 | O_0 | O_1.  There is ONE score buffer: a softmax warp moves its row of S into
// registers and hands the buffer back at once, so the next product (the other tile's, then this
// tile's next key block) is computed while the exponentials run; P_t has columns of its own.  The two
// issuers only follow their own barriers (scores read out / K tile landed; P_t written / O_t
// rescaled / V tile landed), so the tensor pipe takes whichever product is ready and neither issuer's
// waits sit in front of the other's work.  With one issuer and S_t overlaid by P_t the chain
// softmax(j) -> P.V(j) -> Q.K(j+1) -> softmax(j+1) of a tile was serial and set the period.
// All hand-offs are mbarriers; every wait is bounded.
//
// Online softmax with a lazily updated reference: the running reference m of a row only moves
// when the tile maximum exceeds it by more than 8 (log2 units), so most iterations need no
// rescale of O (exp2(s - m) <= 256 stays well inside bf16/fp32 range; the result is the same
// softmax, the final division by the row sum absorbs the reference).
#pragma once
#include <type_traits>

#include "attn_common.cuh"

namespace {

constexpr int kWsThreads = 512;
constexpr int kStages = 4;            // K/V ring slots (one 128 x D tile each)
constexpr float kRescaleThreshold = 8.f;

struct WsItem {
    int r, bl, h, hkv, qb;
    int n[2];                         // KV tiles of query tile 0 / 1 (0 = tile absent)
    int n_max;
};

template <int R>
__device__ __forceinline__ bool ws_get_item(const AttnParams<R> &p, int round, WsItem &it) {
    const int n_qt = (p.S + kTile - 1) / kTile;       // the last tile may be ragged
    const int per_qb = p.r_count * p.Bl * p.Hq_l;
    const int total = p.qb_count * per_qb;
    const int pos = (round & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;   // boustrophedon
    const int i = round * (int)gridDim.x + pos;
    if (i >= total) return false;
    // Order: bands of `qb_band` consecutive query blocks, longest first; inside a band the items of
    // one KV stream (rank, sequence, KV head) are adjacent -- qb_band blocks x q_per_kv query heads --
    // so that the CTAs running side by side read the same K/V tiles through L2.
    const int band = (int)fdiv((uint32_t)i, p.div_per_band);
    int rem = i - band * (int)p.div_per_band.d;
    const int stream = (int)fdiv((uint32_t)rem, p.div_per_stream);
    rem -= stream * (int)p.div_per_stream.d;
    const int qb_in_band = (int)fdiv((uint32_t)rem, p.div_q_per_kv);
    it.qb = p.qb_begin + p.qb_count - 1 - (band * p.qb_band + qb_in_band);
    const int sb = (int)fdiv((uint32_t)stream, p.div_hkv_l);
    it.hkv = stream - sb * p.Hkv_l;
    it.h = it.hkv * p.q_per_kv + (rem - qb_in_band * p.q_per_kv);
    const int rr = (int)fdiv((uint32_t)sb, p.div_bl);
    it.bl = sb - rr * p.Bl;
    it.r = p.r_begin + rr;
    const int qt0 = 2 * it.qb, qt1 = qt0 + 1;
    const bool has1 = qt1 < n_qt;
    it.n[0] = p.causal ? qt0 + 1 : n_qt;
    it.n[1] = has1 ? (p.causal ? qt1 + 1 : n_qt) : 0;
    it.n_max = it.n[1] > it.n[0] ? it.n[1] : it.n[0];
    return true;
}

struct WsShared {
    uint64_t q_full, q_empty;
    uint64_t kv_full[kStages], kv_empty[kStages];
    uint64_t s_free, pv_done[2];
    uint64_t alpha_full[2][2];       // [tile][step parity]
    uint64_t s_full[2], p_full[2], o_rescaled[2], o_final[2], o_free[2];
    uint64_t l_full[2][2];           // [tile][item parity]: a one-step item can end before the epilogue of the one before
    float alpha[2][2][kTile];        // [tile][step parity][row]
    float l[2][2][kTile];            // [item parity][tile][row]
    uint32_t tmem_base;
    int abort_flag;
};

constexpr uint32_t kSleepNs = 32;     // back-off of the correction and producer warps while they wait

#define WS_WAIT(bar, parity, role, detail)                                     \
    do {                                                                        \
        if (!mbar_wait((bar), (parity), &sh.abort_flag, ((role) >= 20 && (role) < 40) ? kSleepNs : 0)) { \
            sh.abort_flag = 1;                                                  \
            report(p.status, 1, (role), (detail));                              \
            goto ws_done;                                                       \
        }                                                                       \
    } while (0)

template <int D, int R>
__global__ void __launch_bounds__(kWsThreads, 1) attn_fwd_ws_kernel(const __grid_constant__ AttnParams<R> p) {
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kTile * D * 2;
    constexpr int kOCols = D;                          // fp32 accumulator columns per O tile
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = smem;                                // 2 tiles
    uint8_t *sKV = smem + 2 * kTileBytes;              // kStages tiles
    __shared__ WsShared sh;

    // the warp index is broadcast from lane 0 so that the compiler knows it is warp-uniform
    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;

    if (tid == 0) {
        mbar_init(&sh.q_full, 1);
        mbar_init(&sh.q_empty, 1);
        for (int i = 0; i < kStages; ++i) { mbar_init(&sh.kv_full[i], 1); mbar_init(&sh.kv_empty[i], 1); }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sh.s_full[t], 1);
            mbar_init(&sh.alpha_full[t][0], 4);
            mbar_init(&sh.alpha_full[t][1], 4);
            mbar_init(&sh.p_full[t], 4);
            mbar_init(&sh.o_rescaled[t], 4);
            mbar_init(&sh.o_final[t], 1);
            mbar_init(&sh.l_full[t][0], 4);
            mbar_init(&sh.l_full[t][1], 4);
            mbar_init(&sh.o_free[t], 4);
        }
        mbar_init(&sh.s_free, 4);
        mbar_init(&sh.pv_done[0], 1);
        mbar_init(&sh.pv_done[1], 1);
        sh.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 12) { tmem_alloc(&sh.tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    // One score tile S at columns 0..127 (the two query tiles take turns), P_t at 128 + 64 t, O_t at 256 + 128 t.

    if (warp < 8) {
        // =============================================================== softmax of query tile t
        reg_inc<192>();
        const int t = warp >> 2;
        const int row = tid & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t S_a = tmem + lane_addr;                   // the shared score tile
        const uint32_t P_t = tmem + 128 + 64 * t + lane_addr;
        uint32_t it_cnt = 0, ep_cnt = 0;
        WsItem item;
        for (int round = 0; ws_get_item(p, round, item); ++round) {
            const int n_t = item.n[t];
            if (n_t == 0) continue;
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_t; ++j, ++it_cnt) {
                WS_WAIT(&sh.s_full[t], it_cnt & 1, 10 + t, j);
                tc_fence_after();
                uint32_t s[kTile];
                tmem_ld_x32(S_a + 0, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
                tmem_ld_x32(S_a + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
                tmem_ld_x32(S_a + 64, *reinterpret_cast<uint32_t(*)[32]>(&s[64]));
                tmem_ld_x32(S_a + 96, *reinterpret_cast<uint32_t(*)[32]>(&s[96]));
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.s_free);       // the scores are in registers: the other tile's Q.K^T may overwrite S
                // Key column i of this tile is visible iff i <= lim: the causal diagonal (i <= row) and, in a
                // ragged last tile, the end of the sequence (i < S - 128 j; what lies beyond belongs to the next
                // sequence of the shard or is TMA zero fill).
                int lim = kTile - 1;
                if (p.causal && j == n_t - 1) lim = row;
                if (p.S - j * kTile - 1 < lim) lim = p.S - j * kTile - 1;
                const bool masked = __any_sync(0xffffffffu, lim < kTile - 1);
                if (masked) {
#pragma unroll
                    for (int i = 0; i < kTile; ++i)
                        if (i > lim) s[i] = 0xff800000u;   // -inf
                }
                float mxs[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) mxs[i] = max3(__uint_as_float(s[i]), __uint_as_float(s[8 + i]), __uint_as_float(s[16 + i]));
#pragma unroll
                for (int i = 24; i + 15 < kTile; i += 16)
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        mxs[k] = max3(mxs[k], __uint_as_float(s[i + k]), __uint_as_float(s[i + 8 + k]));
#pragma unroll
                for (int k = 0; k < 8; ++k) mxs[k] = fmaxf(mxs[k], __uint_as_float(s[120 + k]));
                float mx = fmaxf(fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])),
                                 fmaxf(fmaxf(mxs[4], mxs[5]), fmaxf(mxs[6], mxs[7])));
                mx *= p.scale_log2;
                float m_new, alpha;
                if (j == 0) { m_new = mx; alpha = 1.f; }
                else if (mx > m_ref + kRescaleThreshold) { m_new = mx; alpha = exp2_approx(m_ref - m_new); }
                else { m_new = m_ref; alpha = 1.f; }
                sh.alpha[t][it_cnt & 1][row] = alpha;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.alpha_full[t][it_cnt & 1]);
                m_ref = m_new;
                const uint64_t sc2 = pack_f2(p.scale_log2, p.scale_log2), nm2 = pack_f2(-m_new, -m_new);
                uint64_t rs2[2] = {0ull, 0ull};
                auto exp_row = [&](auto diag_tag) {
                    constexpr bool kDiag = decltype(diag_tag)::value;
#pragma unroll
                    for (int i = 0; i < kTile; i += 2) {
                        const uint64_t x2 = fma2(pack_f2(__uint_as_float(s[i]), __uint_as_float(s[i + 1])), sc2, nm2);
                        float x0, x1;
                        unpack_f2(x2, x0, x1);
                        float e0 = exp2_approx(x0), e1 = exp2_approx(x1);
                        if (kDiag) {                  // masked keys contribute exactly nothing
                            if (i > lim) e0 = 0.f;
                            if (i + 1 > lim) e1 = 0.f;
                        }
                        rs2[(i >> 1) & 1] = add2(rs2[(i >> 1) & 1], pack_f2(e0, e1));
                        s[i >> 1] = pack_bf16x2(e0, e1);
                    }
                };
                // masked scores are -inf already, and exp2(-inf - m) is exactly 0 (m is finite: key 0 is always visible),
                // so one copy of the loop serves both cases: the hot code stays small
                exp_row(std::false_type{});
                float ra, rb;
                unpack_f2(add2(rs2[0], rs2[1]), ra, rb);
                l_run = l_run * alpha + (ra + rb);
                // The previous P_t V (of this item or, at j = 0, the last one of the item before) is issued by a warp
                // of its own: make sure it has read P_t before this step's P_t replaces it.  Waiting at every step
                // also means that no phase of the barrier is ever skipped.
                if (it_cnt > 0) { WS_WAIT(&sh.pv_done[t], (it_cnt - 1) & 1, 14 + t, j); tc_fence_after(); }
                tmem_st_x32(P_t + 0, *reinterpret_cast<const uint32_t(*)[32]>(&s[0]));
                tmem_st_x32(P_t + 32, *reinterpret_cast<const uint32_t(*)[32]>(&s[32]));
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.p_full[t]);
            }
            sh.l[ep_cnt & 1][t][row] = l_run;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.l_full[t][ep_cnt & 1]);
            ++ep_cnt;
            const int s_pos = (2 * item.qb + t) * kTile + row;
            if (p.has_lse && s_pos < p.S) {
                p.lse[item.r][((size_t)item.bl * p.Hq_l + item.h) * p.S + s_pos] =
                    m_ref * 0.6931471805599453f + __logf(l_run);
            }
        }
    } else if (warp < 12) {
        // =============================================================== correction + epilogue
        reg_dec<64>();
        const int row = tid & 127;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t it_cnt[2] = {0, 0}, ep_cnt[2] = {0, 0};
        WsItem item;
        for (int round = 0; ws_get_item(p, round, item); ++round) {
            for (int j = 0; j < item.n_max; ++j) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (j >= item.n[t]) continue;
                    // two barriers per tile, used in turn: the softmax warps can be a step ahead of this one
                    WS_WAIT(&sh.alpha_full[t][it_cnt[t] & 1], (it_cnt[t] >> 1) & 1, 20 + t, j);
                    const float alpha = sh.alpha[t][it_cnt[t] & 1][row];
                    ++it_cnt[t];
                    // O_t is only ours once P_t V(j-1) has completed (it is issued behind Q_t K(j)); waiting for it
                    // every step also keeps o_rescaled at most one phase ahead of the MMA warp
                    if (j > 0) WS_WAIT(&sh.pv_done[t], (it_cnt[t] - 2) & 1, 22 + t, j);
                    if (j > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {
                        tc_fence_after();
                        const uint32_t O_t = tmem + 256 + 128 * t + lane_addr;
#pragma unroll 1                 // rare and not time-critical: kept small
                        for (int c = 0; c < kOCols / 32; ++c) {
                            uint32_t rr[32];
                            tmem_ld_x32(O_t + c * 32, rr);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) rr[i] = __float_as_uint(__uint_as_float(rr[i]) * alpha);
                            tmem_st_x32(O_t + c * 32, rr);
                        }
                        tmem_wait_st();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.o_rescaled[t]);
                }
            }
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (item.n[t] == 0) continue;
                WS_WAIT(&sh.l_full[t][ep_cnt[t] & 1], (ep_cnt[t] >> 1) & 1, 24 + t, 0);
                WS_WAIT(&sh.o_final[t], ep_cnt[t] & 1, 26 + t, 0);
                const float inv_l = 1.f / sh.l[ep_cnt[t] & 1][t][row];
                ++ep_cnt[t];
                tc_fence_after();
                const TileCoord c = locate(p, item.r, item.bl, (2 * item.qb + t) * kTile, item.h, p.Hq_l);
                __nv_bfloat16 *dst = p.o[c.rank] + ((size_t)(c.row + row) * p.o_heads + c.head) * p.Dg;
                const uint32_t O_t = tmem + 256 + 128 * t + lane_addr;
                const bool in_seq = (2 * item.qb + t) * kTile + row < p.S;   // rows past a ragged end are not stored
#pragma unroll
                for (int cc = 0; cc < kOCols / 32; ++cc) {
                    if (cc * 32 >= p.Dg) break;          // columns past the real head dimension are zero padding
                    uint32_t rr[32];
                    tmem_ld_x32(O_t + cc * 32, rr);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 o4;
                        o4.x = pack_bf16x2(__uint_as_float(rr[8 * i + 0]) * inv_l, __uint_as_float(rr[8 * i + 1]) * inv_l);
                        o4.y = pack_bf16x2(__uint_as_float(rr[8 * i + 2]) * inv_l, __uint_as_float(rr[8 * i + 3]) * inv_l);
                        o4.z = pack_bf16x2(__uint_as_float(rr[8 * i + 4]) * inv_l, __uint_as_float(rr[8 * i + 5]) * inv_l);
                        o4.w = pack_bf16x2(__uint_as_float(rr[8 * i + 6]) * inv_l, __uint_as_float(rr[8 * i + 7]) * inv_l);
                        if (in_seq && cc * 32 + i * 8 < p.Dg) *reinterpret_cast<uint4 *>(dst + cc * 32 + i * 8) = o4;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.o_free[t]);
            }
        }
    } else {
        reg_dec<64>();
        if (warp == 12) {
            // =========================================================== TMA producer (lane 0 issues)
            uint32_t kv_it = 0, item_n = 0;
            WsItem item;
            for (int round = 0; ws_get_item(p, round, item); ++round, ++item_n) {
                WS_WAIT(&sh.q_empty, (item_n & 1) ^ 1, 30, round);
                const int n_tiles = item.n[1] > 0 ? 2 : 1;
                if (lane == 0) mbar_arrive_expect_tx(&sh.q_full, n_tiles * kTileBytes);
                for (int t = 0; t < n_tiles; ++t) {
                    const TileCoord c = locate(p, item.r, item.bl, (2 * item.qb + t) * kTile, item.h, p.Hq_l);
                    if (lane == 0)
                        for (int s = 0; s < kSlabs; ++s)
                            tma_load_3d(sQ + t * kTileBytes + s * 16384, &p.q[c.rank], &sh.q_full, s * 64, c.head, c.row);
                }
                for (int j = 0; j < item.n_max; ++j) {
                    const TileCoord c = locate(p, item.r, item.bl, j * kTile, item.hkv, p.Hkv_l, p.kv_rep);
#pragma unroll
                    for (int x = 0; x < 2; ++x, ++kv_it) {
                        const uint32_t slot = kv_it % kStages, ph = (kv_it / kStages) & 1;
                        WS_WAIT(&sh.kv_empty[slot], ph ^ 1, 31, j);
                        const CUtensorMap *tm = x == 0 ? &p.k[c.rank] : &p.v[c.rank];
                        if (lane == 0) {
                            mbar_arrive_expect_tx(&sh.kv_full[slot], kTileBytes);
                            for (int s = 0; s < kSlabs; ++s)
                                tma_load_3d(sKV + slot * kTileBytes + s * 16384, tm, &sh.kv_full[slot], s * 64, c.head, c.row);
                        }
                    }
                }
            }
        } else if (warp == 13) {
            // =========================================================== MMA issuer 1: S = Q_t K_j^T (lane 0 issues)
            // The two issuers run on their own barriers, so the tensor pipe takes whichever product is ready:
            // Q_t.K(j+1) goes ahead as soon as the previous scores have been read out of the single S buffer,
            // while P_t.V(j) waits for the softmax of step j.
            const uint32_t idesc_qk = make_idesc_bf16(kTile, kTile, false, false);
            uint32_t item_n = 0, qk_cnt = 0, kv_base = 0;     // K_j of the item at ring index kv_base + 2j
            WsItem item;
            // Descriptors differ only in the 14-bit start-address field, so a step along K is an add.
            const uint64_t desc_k = make_smem_desc_sw128(0, 16, 1024);        // K-major operands (Q, K)
            const uint32_t q_addr16 = smem_u32(sQ) >> 4, kv_addr16 = smem_u32(sKV) >> 4;
            for (int round = 0; ws_get_item(p, round, item); ++round, ++item_n) {
                WS_WAIT(&sh.q_full, item_n & 1, 40, round);
                for (int j = 0; j < item.n_max; ++j) {
                    const uint32_t idx = kv_base + 2 * j, slot = idx % kStages;
                    WS_WAIT(&sh.kv_full[slot], (idx / kStages) & 1, 41, j);
                    tc_fence_after();
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (j >= item.n[t]) continue;
                        // score tile number q may only follow the hand-over of q - 1 to its softmax warps
                        if (qk_cnt > 0) { WS_WAIT(&sh.s_free, (qk_cnt - 1) & 1, 48, j); tc_fence_after(); }
                        ++qk_cnt;
                        const uint64_t a = desc_k | (uint64_t)(q_addr16 + t * (kTileBytes >> 4));
                        const uint64_t b = desc_k | (uint64_t)(kv_addr16 + slot * (kTileBytes >> 4));
                        if (lane == 0) {
                            // all D/16 steps even when the head dimension is smaller: the padding columns are zero, and a
                            // per-MMA test in this loop costs more (12 % of the kernel) than the two or three extra MMAs
#pragma unroll
                            for (int kk = 0; kk < D / 16; ++kk) {
                                const uint32_t off16 = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                                mma_ss(tmem, a + off16, b + off16, idesc_qk, kk > 0);
                            }
                            tc_commit(&sh.s_full[t]);
                        }
                    }
                    if (lane == 0) {
                        tc_commit(&sh.kv_empty[slot]);                            // K_j has no reader left
                        if (j == item.n_max - 1) tc_commit(&sh.q_empty);          // that was the item's last Q.K^T
                    }
                }
                kv_base += 2 * item.n_max;
            }
        } else if (warp == 14) {
            // =========================================================== MMA issuer 2: O_t += P_t V_j (lane 0 issues)
            const uint32_t idesc_pv = make_idesc_bf16(kTile, D, false, true);
            uint32_t it_cnt[2] = {0, 0}, ep_cnt[2] = {0, 0}, kv_base = 0;     // V_j at ring index kv_base + 2j + 1
            WsItem item;
            const uint64_t desc_v = make_smem_desc_sw128(0, 16384, 1024);     // MN-major operand (V)
            const uint32_t kv_addr16 = smem_u32(sKV) >> 4;
            for (int round = 0; ws_get_item(p, round, item); ++round) {
                for (int j = 0; j < item.n_max; ++j) {
                    const uint32_t idx = kv_base + 2 * j + 1, slot = idx % kStages;
                    WS_WAIT(&sh.kv_full[slot], (idx / kStages) & 1, 42, j);
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (j >= item.n[t]) continue;
                        if (j == 0) WS_WAIT(&sh.o_free[t], (ep_cnt[t] & 1) ^ 1, 43 + t, round);
                        WS_WAIT(&sh.p_full[t], it_cnt[t] & 1, 45 + t, j);
                        WS_WAIT(&sh.o_rescaled[t], it_cnt[t] & 1, 47 + t, j);
                        ++it_cnt[t];
                        tc_fence_after();
                        const uint64_t b = desc_v | (uint64_t)(kv_addr16 + slot * (kTileBytes >> 4));
                        if (lane == 0) {
#pragma unroll
                            for (int kk = 0; kk < kTile / 16; ++kk)
                                mma_ts(tmem + 256 + 128 * t, tmem + 128 + 64 * t + kk * 8, b + kk * (2048 >> 4), idesc_pv,
                                       (j > 0) || (kk > 0));
                            tc_commit(&sh.pv_done[t]);
                            if (j == item.n[t] - 1) tc_commit(&sh.o_final[t]);
                        }
                        if (j == item.n[t] - 1) ++ep_cnt[t];
                    }
                    if (lane == 0) tc_commit(&sh.kv_empty[slot]);                 // V_j has no reader left
                }
                kv_base += 2 * item.n_max;
            }
        }
    }

ws_done:
    tc_fence_before();
    __syncthreads();
    if (sh.abort_flag) {
        // let copies that are still in flight land before the shared memory is given back
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == 12) tmem_dealloc(tmem, 512);
}

#undef WS_WAIT

}  // namespace
