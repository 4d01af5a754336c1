// Backward for head dimensions 80..128 as TWO passes without any reduction through global memory.
//
// The one-pass kernel (attn_bwd_kernel<128>) keeps dK_n, dV_n in TMEM and adds every dQ partial (64 KiB of fp32 per tile
// pair) into an accumulator in global memory: the L2's reduction rate bounds it, and neither TMEM nor shared memory has
// room left to take the five products off the compute warps' critical path.  Here every output is accumulated where it
// is produced, at the price of forming S, dP and the element-wise part twice (7 products per tile pair instead of 5):
//
//   pass KV  one item = key tile n of one (rank, sequence, KV head); streams Q_m, dO_m for the query heads of the GQA group
//            and m >= n:   S^T = K Q^T,  dP^T = V dO^T,  dV += P^T dO,  dK += dS^T Q        (dK_n, dV_n in TMEM)
//   pass Q   one item = query tile m of one (rank, sequence, query head); streams K_n, V_n for n <= m:
//                          S = Q K^T,    dP = dO V^T,                    dQ += dS K          (dQ_m in TMEM)
//
// Both are one kernel template: "stationary" tiles X0, X1 (K, V or Q, dO) stay in shared memory for the item, "stream"
// tiles Y0, Y1 (Q, dO or K, V) pass through a 2-stage ring, (1) ST = X0 Y0^T, (2) DP = X1 Y1^T, (4) ACC0 += dS Y0 and, in
// pass KV only, (3) ACC1 += P Y1 with P read from TMEM.  With no dQ in the dP columns and no staging buffer aliasing the
// ring, the products of step i+1 are issued while step i is computed on:
//   compute warps   wait ST -> load scores -> P = exp2(..) -> [pass KV: P as bf16 over its own score columns] -> p_ready
//                   wait DP -> dS = P (dP scale - Delta scale) -> dS as bf16 into shared memory -> pds_ready
//   issuing warp    p_ready(i): (3)(i), (1)(i+1)        pds_ready(i): (4)(i), (2)(i+1)
// so the tensor core always has the other half of a step to work on, and results are deterministic (no atomics).
// Row statistics: LSE and Delta belong to the query index, which is the score COLUMN in pass KV (staged per step by the
// producer warp) and the score ROW in pass Q (two registers per thread for the whole item).
// TMEM columns: ST 0, DP 128, ACC0 256 (dK or dQ), ACC1 384 (dV).
#pragma once

template <int kPass, int R>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_pass_kernel(const __grid_constant__ BwdParams<R> p) {
    constexpr bool kKV = kPass == 0;
    constexpr int D = 128;
    constexpr int kTileBytes = kT * D * 2;             // 32 KiB: two slabs of [128 rows][64 columns]
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *sX0 = smem, *sX1 = smem + kTileBytes;     // stationary tiles
    uint8_t *sY0 = smem + 2 * kTileBytes;              // stream tiles, 2 stages each
    uint8_t *sY1 = smem + 4 * kTileBytes;
    uint8_t *sdS = smem + 6 * kTileBytes;              // dS [score rows][score cols] as bf16, two 64-column slabs (32 KiB)
    float *s_lse = reinterpret_cast<float *>(sdS + 2 * 16384);         // pass KV: [2][128], already times log2(e)
    float *s_delta = s_lse + 2 * kT;                                   //          [2][128], already times -scale
    BwdBars *bars = reinterpret_cast<BwdBars *>(s_delta + 2 * kT);

    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
    const int n_t = (p.S + kT - 1) / kT;               // tiles per sequence (the last one may be ragged)

    // Work items, longest first.  Pass KV: low key tiles are seen by the most query tiles; pass Q: high query tiles see
    // the most key tiles.
    struct Item { int r, bl, h, hkv, t, steps; };
    auto get_item = [&](int round, Item &it) -> bool {
        const int streams = p.n_ranks * p.Bl * (kKV ? p.Hkv_l : p.Hq_l);
        const int total = n_t * streams;
        const int pos = (round & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
        const int i = round * (int)gridDim.x + pos;
        if (i >= total) return false;
        const int ti = i / streams;
        int rem = i - ti * streams;
        const int heads = kKV ? p.Hkv_l : p.Hq_l;
        const int hh = rem % heads;
        rem /= heads;
        it.bl = rem % p.Bl;
        it.r = rem / p.Bl;
        if (kKV) {
            it.t = ti; it.hkv = hh; it.h = hh * p.q_per_kv;
            it.steps = p.q_per_kv * (n_t - (p.causal ? ti : 0));
        } else {
            it.t = p.causal ? n_t - 1 - ti : ti; it.h = hh; it.hkv = hh / p.q_per_kv;
            it.steps = p.causal ? it.t + 1 : n_t;
        }
        return true;
    };
    // Step j of an item: which stream tile (head and tile index).
    auto step_of = [&](const Item &it, int j, int &head, int &tile) {
        if (kKV) {
            const int cnt = n_t - (p.causal ? it.t : 0);
            const int hq = j / cnt;
            head = it.h + hq;
            tile = (p.causal ? it.t : 0) + (j - hq * cnt);
        } else {
            head = it.hkv;
            tile = j;
        }
    };

    if (tid == 0) {
        mbar_init(&bars->kv_full, 1); mbar_init(&bars->kv_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->qdo_full[s], 1);
            mbar_init(&bars->qdo_mma_done[s], 1);
            mbar_init(&bars->stats_full[s], 1);
        }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->p_ready, kBwdComputeWarps);
        mbar_init(&bars->pds_ready, kBwdComputeWarps);
        mbar_init(&bars->dkdv_full, 1);
        mbar_init(&bars->dkdv_read, kBwdComputeWarps);
        bars->abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        if (bars->abort_flag) bwd_report(p.status, 4, 0, (int)(smem_u32(smem) & 1023u));
        fence_mbar_init();
    }
    if (warp == kBwdTmaWarp) { tmem_alloc(&bars->tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    constexpr uint32_t kColST = 0, kColDP = 128, kColA0 = 256, kColA1 = 384;
    if (bars->abort_flag) goto bwd_done;

    if (warp < kBwdComputeWarps) {
        // ======================================================================= compute warps
        const int g = warp >> 2;                        // which 32-column quarter of the score tile
        const int row = tid & 127;                      // TMEM lane: score row (key in pass KV, query in pass Q)
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t it_g = 0, item_n = 0;
        Item item;
        for (int round = 0; get_item(round, item); ++round, ++item_n) {
            float lse_row = 0.f, del_row = 0.f;         // pass Q: this thread's query row, for the whole item
            if (!kKV) {
                const int s_pos = item.t * kT + row;
                if (s_pos < p.S) {
                    const size_t off = ((size_t)item.bl * p.Hq_l + item.h) * p.S + s_pos;
                    lse_row = p.lse[item.r][off] * 1.4426950408889634f;
                    del_row = -p.scale * p.delta[item.r][off];
                }
            }
            for (int j = 0; j < item.steps; ++j, ++it_g) {
                int head, tile;
                step_of(item, j, head, tile);
                const int buf = it_g & 1;
                if (kKV) BWD_WAIT(&bars->stats_full[buf], (it_g >> 1) & 1, 10, j);
                BWD_WAIT(&bars->s_full, it_g & 1, 11, j);
                tc_fence_after();
                uint32_t st[32], dp[32];
                tmem_ld_x32(tmem + kColST + 32 * g + lane_addr, st);
                tmem_wait_ld();
                if (!kKV) {                 // the scores are in registers and nothing is written back: (1) of the next step may go
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->p_ready);
                }
                // Which of this thread's 32 columns count: [c_lo, c_hi).  Only edge steps (the diagonal tile, a ragged last
                // tile) restrict it; the loop is instantiated twice so that the common step has no masking code.
                const int kv_t = kKV ? item.t : tile, q_t = kKV ? tile : item.t;
                const bool diag = p.causal && kv_t == q_t;
                const bool edge = diag || (kv_t + 1) * kT > p.S || (q_t + 1) * kT > p.S;
                int c_lo = 0, c_hi = 32;
                if (edge) {
                    if (kKV) {              // row = key, columns = queries: a query counts iff it is not before the key
                        if (diag) c_lo = row - 32 * g;
                        if (kv_t * kT + row >= p.S) c_lo = 32;
                        if (p.S - q_t * kT - 32 * g < c_hi) c_hi = p.S - q_t * kT - 32 * g;
                    } else {                // row = query, columns = keys: a key counts iff it is not after the query
                        if (diag) c_hi = row - 32 * g + 1;
                        if (p.S - kv_t * kT - 32 * g < c_hi) c_hi = p.S - kv_t * kT - 32 * g;
                        if (q_t * kT + row >= p.S) c_lo = 32;
                    }
                }
                const float *lse_b = s_lse + buf * kT + 32 * g;
                const float *del_b = s_delta + buf * kT + 32 * g;
                auto p_phase = [&](auto edge_tag) {
                    constexpr bool kEdge = decltype(edge_tag)::value;
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        float lv[4] = {lse_row, lse_row, lse_row, lse_row};
                        if (kKV) {
                            const float4 l4 = *reinterpret_cast<const float4 *>(lse_b + c);
                            lv[0] = l4.x; lv[1] = l4.y; lv[2] = l4.z; lv[3] = l4.w;
                        }
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float pv = exp2_approx(fmaf(__uint_as_float(st[c + e]), p.scale_log2, -lv[e]));
                            if (kEdge && (c + e < c_lo || c + e >= c_hi)) pv = 0.f;
                            st[c + e] = __float_as_uint(pv);
                        }
                    }
                };
                if (edge) p_phase(std::true_type{});
                else p_phase(std::false_type{});
                if (kKV) {
                    // P^T (bf16) over this quarter's own score columns, stored BEFORE the wait for dP^T: the store needs the
                    // values, so the compiler cannot schedule the exponentials behind that wait; product (3) starts on it.
                    uint32_t pk[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        pk[c] = pack_bf16x2(__uint_as_float(st[2 * c]), __uint_as_float(st[2 * c + 1]));
                    tmem_st_x16(tmem + kColST + 32 * g + lane_addr, pk);
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->p_ready);
                }
                BWD_WAIT(&bars->dp_full, it_g & 1, 12, j);
                tc_fence_after();
                tmem_ld_x32(tmem + kColDP + 32 * g + lane_addr, dp);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; c += 4) {
                    float dl[4] = {del_row, del_row, del_row, del_row};
                    if (kKV) {
                        const float4 d4 = *reinterpret_cast<const float4 *>(del_b + c);
                        dl[0] = d4.x; dl[1] = d4.y; dl[2] = d4.z; dl[3] = d4.w;
                    }
                    float dsv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        dsv[e] = __uint_as_float(st[c + e]) * fmaf(__uint_as_float(dp[c + e]), p.scale, dl[e]);   // dl = -Delta scale
                    dp[c >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                    dp[(c >> 1) + 1] = pack_bf16x2(dsv[2], dsv[3]);
                }
                // dS row `row`, columns 32g..32g+31 = half a 128-byte line of slab g/2 (128-byte swizzle).  The buffer's last
                // readers, product (4) of the step before, were complete before (2) of this step was.
                {
                    uint8_t *line = sdS + (g >> 1) * 16384 + row * 128;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch)
                        *reinterpret_cast<uint4 *>(line + (((4 * (g & 1) + ch) ^ (row & 7)) << 4)) =
                            make_uint4(dp[4 * ch], dp[4 * ch + 1], dp[4 * ch + 2], dp[4 * ch + 3]);
                }
                fence_proxy_async_smem();
                tc_fence_before();          // the dP^T columns have been read: (2) of the next step may overwrite them
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->pds_ready);
            }
            // ---- item done: the accumulators to global memory as bf16
            BWD_WAIT(&bars->dkdv_full, item_n & 1, 13, item.t);
            tc_fence_after();
            if (kKV) {
                // quarters 0,1 write the two 64-column halves of dK, quarters 2,3 those of dV
                __nv_bfloat16 *base = (g < 2 ? p.dk[item.r] : p.dv[item.r]) +
                                      (((size_t)item.bl * p.S + (size_t)item.t * kT + row) * p.Hkv_l + item.hkv) * p.Dg +
                                      64 * (g & 1);
                const uint32_t col0 = (g < 2 ? kColA0 : kColA1) + 64 * (g & 1);
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t rr[32];
                    tmem_ld_x32(tmem + col0 + cc * 32 + lane_addr, rr);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 o4;
                        o4.x = pack_bf16x2(__uint_as_float(rr[8 * i + 0]), __uint_as_float(rr[8 * i + 1]));
                        o4.y = pack_bf16x2(__uint_as_float(rr[8 * i + 2]), __uint_as_float(rr[8 * i + 3]));
                        o4.z = pack_bf16x2(__uint_as_float(rr[8 * i + 4]), __uint_as_float(rr[8 * i + 5]));
                        o4.w = pack_bf16x2(__uint_as_float(rr[8 * i + 6]), __uint_as_float(rr[8 * i + 7]));
                        if (64 * (g & 1) + cc * 32 + i * 8 < p.Dg && item.t * kT + row < p.S)
                            *reinterpret_cast<uint4 *>(base + cc * 32 + i * 8) = o4;
                    }
                }
            } else {
                // quarter g writes columns 32g .. 32g+31 of dQ
                __nv_bfloat16 *base = p.dq[item.r] +
                                      (((size_t)item.bl * p.S + (size_t)item.t * kT + row) * p.Hq_l + item.h) * p.Dg + 32 * g;
                uint32_t rr[32];
                tmem_ld_x32(tmem + kColA0 + 32 * g + lane_addr, rr);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 o4;
                    o4.x = pack_bf16x2(__uint_as_float(rr[8 * i + 0]), __uint_as_float(rr[8 * i + 1]));
                    o4.y = pack_bf16x2(__uint_as_float(rr[8 * i + 2]), __uint_as_float(rr[8 * i + 3]));
                    o4.z = pack_bf16x2(__uint_as_float(rr[8 * i + 4]), __uint_as_float(rr[8 * i + 5]));
                    o4.w = pack_bf16x2(__uint_as_float(rr[8 * i + 6]), __uint_as_float(rr[8 * i + 7]));
                    if (32 * g + i * 8 < p.Dg && item.t * kT + row < p.S)
                        *reinterpret_cast<uint4 *>(base + i * 8) = o4;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->dkdv_read);
        }
    } else if (warp < kBwdTmaWarp) {
        // (the fifth warpgroup has no work in this kernel)
    } else {
      reg_dec<56>();
      if (warp == kBwdTmaWarp) {
        // ======================================================================= TMA producer
        uint32_t it_g = 0, item_n = 0;
        Item item;
        for (int round = 0; get_item(round, item); ++round, ++item_n) {
            BWD_WAIT(&bars->kv_empty, (item_n & 1) ^ 1, 20, item.t);
            if (lane == 0) {
                mbar_arrive_expect_tx(&bars->kv_full, 2 * kTileBytes);
                const int row0 = item.bl * p.S + item.t * kT;
                for (int s = 0; s < 2; ++s) {
                    tma_load_3d(sX0 + s * 16384, kKV ? &p.k[item.r] : &p.q[item.r], &bars->kv_full, s * 64, kKV ? item.hkv : item.h, row0);
                    tma_load_3d(sX1 + s * 16384, kKV ? &p.v[item.r] : &p.dout[item.r], &bars->kv_full, s * 64, kKV ? item.hkv : item.h, row0);
                }
            }
            for (int j = 0; j < item.steps; ++j, ++it_g) {
                int head, tile;
                step_of(item, j, head, tile);
                const uint32_t stage = it_g & 1, ph = (it_g >> 1) & 1;
                BWD_WAIT(&bars->qdo_mma_done[stage], ph ^ 1, 21, j);   // products (3), (4) of two steps ago are done with the stage
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bars->qdo_full[stage], 2 * kTileBytes);
                    const int row0 = item.bl * p.S + tile * kT;
                    for (int s = 0; s < 2; ++s) {
                        tma_load_3d(sY0 + stage * kTileBytes + s * 16384, kKV ? &p.q[item.r] : &p.k[item.r], &bars->qdo_full[stage], s * 64, head, row0);
                        tma_load_3d(sY1 + stage * kTileBytes + s * 16384, kKV ? &p.dout[item.r] : &p.v[item.r], &bars->qdo_full[stage], s * 64, head, row0);
                    }
                }
                if (kKV) {  // row statistics of the query tile: LSE (to log2 units) and Delta (times -scale), four rows per lane
                    const size_t off = ((size_t)item.bl * p.Hq_l + head) * p.S + (size_t)tile * kT + 4 * lane;
                    float4 l4, d4;
                    if ((p.S & 3) == 0 && (tile + 1) * kT <= p.S) {
                        l4 = *reinterpret_cast<const float4 *>(p.lse[item.r] + off);
                        d4 = *reinterpret_cast<const float4 *>(p.delta[item.r] + off);
                    } else {                       // ragged: rows of (bl, h) are not 16-byte aligned, or the tile runs past S
                        float lv[4], dv4[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const bool in_seq = tile * kT + 4 * lane + e < p.S;
                            lv[e] = in_seq ? p.lse[item.r][off + e] : 0.f;
                            dv4[e] = in_seq ? p.delta[item.r][off + e] : 0.f;
                        }
                        l4 = make_float4(lv[0], lv[1], lv[2], lv[3]);
                        d4 = make_float4(dv4[0], dv4[1], dv4[2], dv4[3]);
                    }
                    l4.x *= 1.4426950408889634f; l4.y *= 1.4426950408889634f;
                    l4.z *= 1.4426950408889634f; l4.w *= 1.4426950408889634f;
                    d4.x *= -p.scale; d4.y *= -p.scale; d4.z *= -p.scale; d4.w *= -p.scale;
                    *reinterpret_cast<float4 *>(s_lse + stage * kT + 4 * lane) = l4;
                    *reinterpret_cast<float4 *>(s_delta + stage * kT + 4 * lane) = d4;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->stats_full[stage]);
                }
            }
        }
      } else if (warp == kBwdMmaWarp) {
        // ======================================================================= MMA issuer
        const uint32_t idesc_kk = make_idesc_bf16(kT, kT, false, false);     // (1) (2): both operands K-major
        const uint32_t idesc_kn = make_idesc_bf16(kT, D, false, true);       // (3) (4): B is MN-major
        const uint64_t desc_k = make_smem_desc_sw128(0, 16, 1024);
        const uint64_t desc_mn = make_smem_desc_sw128(0, 16384, 1024);
        const uint32_t aX0 = smem_u32(sX0) >> 4, aX1 = smem_u32(sX1) >> 4, aY0 = smem_u32(sY0) >> 4,
                       aY1 = smem_u32(sY1) >> 4, adS = smem_u32(sdS) >> 4;
        uint32_t it_g = 0, item_n = 0;
        Item item;
        for (int round = 0; get_item(round, item); ++round, ++item_n) {
            const uint32_t steps = (uint32_t)item.steps;
            BWD_WAIT(&bars->kv_full, item_n & 1, 30, item.t);
            // (1) ST = X0 Y0^T of step `it` (the score columns are free: their last content, the scores or P^T of the step
            //     before, has been read by the compute warps / by product (3) issued before)
            auto issue_s = [&](uint32_t it) -> bool {
                const uint32_t stage = it & 1;
                if (!mbar_wait(&bars->qdo_full[stage], (it >> 1) & 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColST, desc_k | (uint64_t)(aX0 + off),
                               desc_k | (uint64_t)(aY0 + stage * (kTileBytes >> 4) + off), idesc_kk, kk > 0);
                    }
                    tc_commit(&bars->s_full);
                }
                return true;
            };
            // (2) DP = X1 Y1^T of step `it` (its stage was waited for by (1); the dP columns were read before pds_ready)
            auto issue_dp = [&](uint32_t it) {
                const uint32_t stage = it & 1;
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColDP, desc_k | (uint64_t)(aX1 + off),
                               desc_k | (uint64_t)(aY1 + stage * (kTileBytes >> 4) + off), idesc_kk, kk > 0);
                    }
                    tc_commit(&bars->dp_full);
                }
            };
            if (!issue_s(it_g)) { bars->abort_flag = 1; bwd_report(p.status, 3, 31, item.t); goto bwd_done; }
            issue_dp(it_g);
            for (uint32_t j = 0; j < steps; ++j) {
                const uint32_t it = it_g + j, stage = it & 1;
                const uint32_t y0 = aY0 + stage * (kTileBytes >> 4), y1 = aY1 + stage * (kTileBytes >> 4);
                const uint32_t acc0 = j == 0 ? 0u : 1u;
                BWD_WAIT(&bars->p_ready, it & 1, 32, (int)j);
                if (j == 0) BWD_WAIT(&bars->dkdv_read, (item_n & 1) ^ 1, 34, item.t);   // the accumulators of the item before are stored
                tc_fence_after();
                if (kKV && lane == 0) {
                    // (3) ACC1 += P Y1 : A = P (bf16) in the score columns (8 columns per 16 of the K index, each quarter
                    //     of 32 at its own column 32g), B = Y1 read MN-major
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk)
                        mma_ts(tmem + kColA1, tmem + kColST + (kk / 2) * 32 + (kk % 2) * 8,
                               desc_mn | (uint64_t)(y1 + kk * 128), idesc_kn, kk > 0 ? 1u : acc0);
                }
                if (j + 1 < steps && !issue_s(it + 1)) { bars->abort_flag = 1; bwd_report(p.status, 3, 35, (int)j); goto bwd_done; }
                BWD_WAIT(&bars->pds_ready, it & 1, 33, (int)j);
                tc_fence_after();
                if (lane == 0) {
                    // (4) ACC0 += dS Y0 : A = dS from shared memory (K-major), B = Y0 read MN-major
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColA0, desc_k | (uint64_t)(adS + off), desc_mn | (uint64_t)(y0 + kk * 128),
                               idesc_kn, kk > 0 ? 1u : acc0);
                    }
                    tc_commit(&bars->qdo_mma_done[stage]);        // (3) and (4) are done with the stage
                }
                if (j + 1 < steps) issue_dp(it + 1);
            }
            it_g += steps;
            if (lane == 0) {
                tc_commit(&bars->dkdv_full);
                tc_commit(&bars->kv_empty);
            }
        }
      }
    }

bwd_done:
    tc_fence_before();
    __syncthreads();
    if (bars->abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == kBwdTmaWarp) tmem_dealloc(tmem, 512);
}
