// Backward kernel for head dimensions 80 .. 128 (128 columns wide): the five products of attn_bwd.cu's header comment,
// software-pipelined inside the 512 TMEM columns and 227 KiB of shared memory that a 128-wide tile pair leaves.
//
// TMEM: X = S^T, then P^T (bf16, over its own columns) at 0 | Y = dP^T, then dQ^T at 128 | dK at 256 | dV at 384.
// Shared memory: K, V (resident per item) | Q x 2 stages | dO x 2 stages | dS^T | row statistics.
//
// Order on the tensor pipe in the steady state (step j of an item):
//     (3)_j  dV += P^T_j dO_j          as soon as the exponentials of step j are in TMEM   -> dO stage free
//     (1)_j+1  S^T = K Q_j+1^T         into X right behind (3)_j (the pipe finishes in issue order)
//     (5)_j  dQ_j^T = K^T dS_j^T -> Y,  (4)_j  dK += dS_j^T Q_j    once dS^T_j is in shared memory   -> Q stage free
//     (2)_j+1  dP^T = V dO_j+1^T       into Y once the drain warps have taken dQ_j out
// so the compute warps find the scores of step j+1 waiting when they finish dS of step j, and its dP^T shortly after
// the exponentials.  Every stage is released by the completion of the products that read it, never by the reduction.
//
// dQ leaves without touching shared memory.  Product (5) is issued with its operands swapped, which leaves the tile
// TRANSPOSED in Y (lane = feature, column = query row); a drain warp's 32 lanes then hold 32 consecutive features of
// one query row in each register, and one red.global.add.f32 per register adds a complete 128-byte line of the fp32
// accumulator.  Measured on the access pattern of this kernel (148 CTAs, four warps each): 6.1 TB/s of fp32 payload,
// the same as 512 bytes per instruction, against 2.3 / 4.1 TB/s for bulk reductions of 128 / 256 bytes per operation
// out of shared memory and 2.5 TB/s for a row per thread; and generic loads and stores of shared memory crawl while
// the tensor pipe streams its operands out of it (a staged variant of this kernel spent 3000 clk per half tile there).
// What bounds the kernel now is the L2: per step 64 KiB of Q / dO tiles in and 64 KiB of reductions (which the L2 counts
// twice), close to 10 TB/s in total.
#pragma once

template <int R>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_d128_kernel(const __grid_constant__ BwdParams<R> p) {
    constexpr int D = 128;
    constexpr int kTileBytes = kT * D * 2;             // 32 KiB: two slabs of [128 rows][64 columns]
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *sK = smem, *sV = smem + kTileBytes;
    uint8_t *sQ = smem + 2 * kTileBytes;               // 2 stages
    constexpr int kDoStages = 2;
    uint8_t *sdO = smem + 4 * kTileBytes;
    uint8_t *sdS = smem + (4 + kDoStages) * kTileBytes;   // dS^T [key rows][query cols], two 64-column slabs
    float *s_lse = reinterpret_cast<float *>(smem + 7 * kTileBytes);   // [2][128], already times log2(e)
    float *s_delta = s_lse + 2 * kT;                                   // [2][128], already times -scale
    BwdBars *bars = reinterpret_cast<BwdBars *>(s_delta + 2 * kT);

    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
    auto get_item = [&](int round, BwdItem &it) { return p.gang ? bwd_get_item_gang(p, round, it) : bwd_get_item(p, round, it); };

    if (tid == 0) {
        mbar_init(&bars->kv_full, 1); mbar_init(&bars->kv_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->qdo_full[s], 1);          // Q stage loaded
            mbar_init(&bars->qdo_mma_done[s], 1);      // Q stage free: products (1) and (4) of its step are done
            mbar_init(&bars->stats_full[s], 1);
            mbar_init(&bars->do_full[s], 1);           // dO stage loaded
            mbar_init(&bars->do_free[s], 1);           // dO stage free: products (2) and (3) of its step are done
        }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->p_ready, kBwdComputeWarps);
        mbar_init(&bars->pds_ready, kBwdComputeWarps);
        mbar_init(&bars->dq_full, 1);
        mbar_init(&bars->dq_read, 4);
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
    constexpr uint32_t kColST = 0, kColDP = 128, kColDK = 256, kColDV = 384;
    if (bars->abort_flag) goto bwd_done;

    if (warp < kBwdComputeWarps) {
        // ======================================================================= compute warps
        const int g = warp >> 2;                        // which 32-column quarter of the score tile
        const int row = tid & 127;                      // TMEM lane: key row
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t st_col = tmem + kColST + 32 * g + lane_addr;
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; get_item(round, item); ++round, ++item_n) {
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const uint32_t stage = it_g & 1, sph = (it_g >> 1) & 1;     // Q stage of the step (row statistics with it)
                    BWD_WAIT(&bars->stats_full[stage], sph, 10, m);             // LSE and Delta of the query tile
                    BWD_WAIT(&bars->s_full, it_g & 1, 11, m);
                    tc_fence_after();
                    uint32_t st[32], dp[32];
                    tmem_ld_x32(st_col, st);
                    tmem_wait_ld();
                    // the column window of an edge step (the diagonal, a ragged last tile): this thread's columns c (query
                    // 32g + c) count iff c_lo <= c < c_hi; the common step is instantiated without the test
                    const bool diag = p.causal && m == item.n;
                    const bool edge = diag || (m + 1) * kT > p.S || (item.n + 1) * kT > p.S;
                    int c_lo = 0, c_hi = 32;
                    if (edge) {
                        if (diag) c_lo = row - 32 * g;                              // queries earlier than key `row`
                        if (item.n * kT + row >= p.S) c_lo = 32;                    // this thread's key row does not exist
                        if (p.S - m * kT - 32 * g < c_hi) c_hi = p.S - m * kT - 32 * g;   // queries past the end
                    }
                    const float *lse_b = s_lse + stage * kT + 32 * g;
                    const float *del_b = s_delta + stage * kT + 32 * g;
                    // P^T = exp2(S^T scale log2e - LSE): needs the scores only
                    auto p_phase = [&](auto edge_tag) {
                        constexpr bool kEdge = decltype(edge_tag)::value;
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 l4 = *reinterpret_cast<const float4 *>(lse_b + c);
                            const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
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
                    // P^T (bf16) over this quarter's own score columns, stored before the wait for dP^T: the store needs
                    // the values, so the compiler cannot move the exponentials behind that wait
                    {
                        uint32_t pk[16];
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            pk[c] = pack_bf16x2(__uint_as_float(st[2 * c]), __uint_as_float(st[2 * c + 1]));
                        tmem_st_x16(st_col, pk);
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->p_ready);          // product (3) of this step may start
                    // dS^T = P^T (dP^T scale - Delta scale)
                    BWD_WAIT(&bars->dp_full, it_g & 1, 12, m);
                    tc_fence_after();
                    tmem_ld_x32(tmem + kColDP + 32 * g + lane_addr, dp);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 d4 = *reinterpret_cast<const float4 *>(del_b + c);
                        const float dl[4] = {d4.x, d4.y, d4.z, d4.w};
                        float dsv[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            dsv[e] = __uint_as_float(st[c + e]) * fmaf(__uint_as_float(dp[c + e]), p.scale, dl[e]);
                        dp[c >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                        dp[(c >> 1) + 1] = pack_bf16x2(dsv[2], dsv[3]);
                    }
                    // dS^T row `row`, query columns 32g..32g+31 = half a 128-byte line of slab g/2 (128-byte swizzle).  The
                    // buffer's last readers, products (5) and (4) of the step before, were complete before dP^T of this
                    // step was (the tensor pipe finishes in issue order).
                    {
                        uint8_t *line = sdS + (g >> 1) * 16384 + row * 128;
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch)
                            *reinterpret_cast<uint4 *>(line + (((4 * (g & 1) + ch) ^ (row & 7)) << 4)) =
                                make_uint4(dp[4 * ch], dp[4 * ch + 1], dp[4 * ch + 2], dp[4 * ch + 3]);
                    }
                    fence_proxy_async_smem();
                    tc_fence_before();                  // the load of dP^T is complete: Y may take dQ
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->pds_ready);
                }
            }
            // ---- item done: dK_n (quarters 0, 1) / dV_n (quarters 2, 3) to global as bf16, 64 columns per quarter
            BWD_WAIT(&bars->dkdv_full, item_n & 1, 13, item.n);
            tc_fence_after();
            {
                constexpr int kHalf = D / 2;
                __nv_bfloat16 *base = (g < 2 ? p.dk[item.r] : p.dv[item.r]) +
                                      (((size_t)item.bl * p.S + (size_t)item.n * kT + row) * p.Hkv_l + item.hkv) * p.Dg +
                                      kHalf * (g & 1);
                const uint32_t col0 = (g < 2 ? kColDK : kColDV) + kHalf * (g & 1);
#pragma unroll
                for (int cc = 0; cc < kHalf / 32; ++cc) {
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
                        if (kHalf * (g & 1) + cc * 32 + i * 8 < p.Dg && item.n * kT + row < p.S)
                            *reinterpret_cast<uint4 *>(base + cc * 32 + i * 8) = o4;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->dkdv_read);
        }
    } else if (warp < kBwdTmaWarp) {
        // ======================================================================= dQ drain warps
        // Product (5) leaves dQ_m TRANSPOSED in Y (lane = feature d, column = query row), so a warp's 32 lanes hold 32
        // consecutive features of one query row per register: one red.global.add.f32 per register adds a complete
        // 128-byte line of the fp32 accumulator.  No shared memory, no staging; Y is handed back once its last columns
        // are in registers.
        reg_inc<120>();
        const int wq = warp & 3;
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        const int d = wq * 32 + lane;                   // this thread's feature
        uint32_t it_g = 0;
        BwdItem item;
        for (int round = 0; get_item(round, item); ++round) {
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                const int h = item.hkv * p.q_per_kv + hq;
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    BWD_WAIT(&bars->dq_full, it_g & 1, 14, m);
                    tc_fence_after();
                    // accumulator element (query row m*128 + c, head h, feature d); a row past the end of the sequence
                    // (ragged last tile) and a feature past the head dimension have none
                    const size_t acc_row = (size_t)p.Hq_l * p.Dg;
                    float *acc = p.dq_accp[item.r] + (((size_t)item.bl * p.S + (size_t)m * kT) * p.Hq_l + h) * p.Dg + d;
                    const int rows_left = d < p.Dg ? p.S - m * kT : 0;          // columns c < rows_left are added
                    auto add_cols = [&](const uint32_t *v, int c0, int n) {
                        if (c0 + n <= rows_left) {
#pragma unroll
                            for (int c = 0; c < n; ++c)
                                asm volatile("red.global.add.f32 [%0], %1;" ::"l"(acc + (size_t)(c0 + c) * acc_row),
                                             "f"(__uint_as_float(v[c])) : "memory");
                        } else {
#pragma unroll
                            for (int c = 0; c < n; ++c)
                                if (c0 + c < rows_left)
                                    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(acc + (size_t)(c0 + c) * acc_row),
                                                 "f"(__uint_as_float(v[c])) : "memory");
                        }
                    };
                    uint32_t v[96], w[32];
                    tmem_ld_x32(tmem + kColDP + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                    tmem_ld_x32(tmem + kColDP + 32 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                    tmem_ld_x32(tmem + kColDP + 64 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[64]));
                    tmem_wait_ld();
                    add_cols(&v[0], 0, 32);
                    tmem_ld_x32(tmem + kColDP + 96 + lane_addr, w);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->dq_read);          // Y is free for the next dP^T
                    add_cols(&v[32], 32, 64);
                    add_cols(w, 96, 32);
                }
            }
        }
    } else {
      reg_dec<40>();       // 16 x 80 (compute) + 4 x 120 (drain) + 4 x 40 = the 24 x 80 registers per lane the CTA was launched with
      if (warp == kBwdTmaWarp) {
        // ======================================================================= TMA producer
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; get_item(round, item); ++round, ++item_n) {
            BWD_WAIT(&bars->kv_empty, (item_n & 1) ^ 1, 20, item.n);
            if (lane == 0) {
                mbar_arrive_expect_tx(&bars->kv_full, 2 * kTileBytes);
                const int row0 = item.bl * p.S + item.n * kT;
                for (int s = 0; s < 2; ++s) {
                    tma_load_3d(sK + s * 16384, &p.k[item.r], &bars->kv_full, s * 64, item.hkv, row0);
                    tma_load_3d(sV + s * 16384, &p.v[item.r], &bars->kv_full, s * 64, item.hkv, row0);
                }
            }
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                const int h = item.hkv * p.q_per_kv + hq;
                if (p.gang) {               // the gang's members start this sweep together (see bwd_get_item_gang)
                    int ok = 1;
                    if (lane == 0) ok = bwd_gang_barrier(p, round, hq) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { bars->abort_flag = 1; bwd_report(p.status, 3, 23, hq); goto bwd_done; }
                }
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const uint32_t stage = it_g & 1, ph = (it_g >> 1) & 1;
                    const int row0 = item.bl * p.S + m * kT;
                    // Q stage (tile and row statistics): free once products (1) and (4) of two steps ago are done, which also
                    // means that the compute warps have finished that step
                    BWD_WAIT(&bars->qdo_mma_done[stage], ph ^ 1, 21, m);
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&bars->qdo_full[stage], kTileBytes);
                        for (int s = 0; s < 2; ++s)
                            tma_load_3d(sQ + stage * kTileBytes + s * 16384, &p.q[item.r], &bars->qdo_full[stage], s * 64, h, row0);
                    }
                    {
                        const size_t off = ((size_t)item.bl * p.Hq_l + h) * p.S + (size_t)m * kT + 4 * lane;
                        float4 l4, d4;
                        if ((p.S & 3) == 0 && (m + 1) * kT <= p.S) {
                            l4 = *reinterpret_cast<const float4 *>(p.lse[item.r] + off);
                            d4 = *reinterpret_cast<const float4 *>(p.delta[item.r] + off);
                        } else {                       // ragged: rows of (bl, h) are not 16-byte aligned, or the tile runs past S
                            float lv[4], dv4[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const bool in_seq = m * kT + 4 * lane + e < p.S;
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
                    // dO stage: free once product (3) of its previous step is done
                    const uint32_t dstage = it_g % kDoStages, dph = (it_g / kDoStages) & 1;
                    BWD_WAIT(&bars->do_free[dstage], dph ^ 1, 22, m);
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&bars->do_full[dstage], kTileBytes);
                        for (int s = 0; s < 2; ++s)
                            tma_load_3d(sdO + dstage * kTileBytes + s * 16384, &p.dout[item.r], &bars->do_full[dstage], s * 64, h, row0);
                    }
                }
            }
        }
      } else if (warp == kBwdMmaWarp) {
        // ======================================================================= MMA issuer
        const uint32_t idesc_kk = make_idesc_bf16(kT, kT, false, false);     // (1) (2): both operands K-major
        const uint32_t idesc_kn = make_idesc_bf16(kT, D, false, true);       // (3) (4): B is MN-major
        const uint32_t idesc_nn = make_idesc_bf16(kT, D, true, true);        // (5): A and B MN-major
        const uint64_t desc_k = make_smem_desc_sw128(0, 16, 1024);
        const uint64_t desc_mn = make_smem_desc_sw128(0, 16384, 1024);
        const uint32_t aK = smem_u32(sK) >> 4, aV = smem_u32(sV) >> 4, aQ = smem_u32(sQ) >> 4,
                       adO = smem_u32(sdO) >> 4, adS = smem_u32(sdS) >> 4;
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; get_item(round, item); ++round, ++item_n) {
            const uint32_t steps = (uint32_t)p.q_per_kv * (uint32_t)(item.n_qt - item.m0);
            BWD_WAIT(&bars->kv_full, item_n & 1, 30, item.n);
            // (1) S^T = K Q^T of step `it` into X (its last reader, product (3) of step it-1, was issued before)
            auto issue_s = [&](uint32_t it) -> bool {
                const uint32_t stage = it & 1;
                if (!mbar_wait(&bars->qdo_full[stage], (it >> 1) & 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t q16 = aQ + stage * (kTileBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColST, desc_k | (uint64_t)(aK + off), desc_k | (uint64_t)(q16 + off), idesc_kk, kk > 0);
                    }
                    tc_commit(&bars->s_full);
                }
                return true;
            };
            // (2) dP^T = V dO^T of step `it` into Y, once dQ of step it-1 has left it
            auto issue_dp = [&](uint32_t it) -> bool {
                if (!mbar_wait(&bars->dq_read, (it & 1) ^ 1, &bars->abort_flag)) return false;
                if (!mbar_wait(&bars->do_full[it % kDoStages], (it / kDoStages) & 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t do16 = adO + (it % kDoStages) * (kTileBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColDP, desc_k | (uint64_t)(aV + off), desc_k | (uint64_t)(do16 + off), idesc_kk, kk > 0);
                    }
                    tc_commit(&bars->dp_full);
                }
                return true;
            };
            // (3) dV += P^T dO of step `it`: A = P^T in X (query index along K: 8 columns per 16 queries, each quarter of
            //     32 queries starts at its own column 32g), B = dO read MN-major.  The first one of an item also waits
            //     until dK / dV of the item before have been stored.  When it is done the dO stage is free.
            auto issue_dv = [&](uint32_t it, bool first) -> bool {
                if (!mbar_wait(&bars->p_ready, it & 1, &bars->abort_flag)) return false;
                if (first && !mbar_wait(&bars->dkdv_read, (item_n & 1) ^ 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t do16 = adO + (it % kDoStages) * (kTileBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk)
                        mma_ts(tmem + kColDV, tmem + kColST + (kk / 2) * 32 + (kk % 2) * 8,
                               desc_mn | (uint64_t)(do16 + kk * 128), idesc_kn, kk > 0 ? 1u : (first ? 0u : 1u));
                    tc_commit(&bars->do_free[it % kDoStages]);
                }
                return true;
            };
            bool ok = issue_s(it_g) && issue_dp(it_g);
            if (!ok) { bars->abort_flag = 1; bwd_report(p.status, 3, 31, item.n); goto bwd_done; }
            for (uint32_t j = 0; j < steps; ++j) {
                const uint32_t it = it_g + j, stage = it & 1;
                const uint32_t q16 = aQ + stage * (kTileBytes >> 4);
                ok = issue_dv(it, j == 0);
                if (ok && j + 1 < steps) ok = issue_s(it + 1);
                if (!ok) { bars->abort_flag = 1; bwd_report(p.status, 3, 32, (int)j); goto bwd_done; }
                BWD_WAIT(&bars->pds_ready, it & 1, 33, (int)j);
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t acc0 = j == 0 ? 0u : 1u;
                    // (5) dQ_m^T = K^T dS^T : A = K read MN-major (rows of the result = features), B = the dS^T buffer read
                    //     MN-major (columns = query rows); transposed so that the drain warps add whole lines
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk)
                        mma_ss(tmem + kColDP, desc_mn | (uint64_t)(aK + kk * 128), desc_mn | (uint64_t)(adS + kk * 128),
                               idesc_nn, kk > 0);
                    tc_commit(&bars->dq_full);
                    // (4) dK += dS^T Q : A = dS^T from shared memory (K-major: query columns), B = Q MN-major
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColDK, desc_k | (uint64_t)(adS + off), desc_mn | (uint64_t)(q16 + kk * 128),
                               idesc_kn, kk > 0 ? 1u : acc0);
                    }
                    tc_commit(&bars->qdo_mma_done[stage]);        // (1) and (4) of the step are done: its Q stage may be loaded again
                }
                if (j + 1 < steps && !issue_dp(it + 1)) { bars->abort_flag = 1; bwd_report(p.status, 3, 35, (int)j); goto bwd_done; }
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
