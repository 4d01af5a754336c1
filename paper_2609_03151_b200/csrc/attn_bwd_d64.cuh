// Backward kernel for head dimensions up to 64: the same products, roles and tile layouts as attn_bwd_kernel<64>, but
// software-pipelined.  At this width half of the tensor memory and a third of the shared memory of the 128-wide kernel
// are free, which buys what that kernel cannot have:
//   - a second S^T buffer in TMEM, so S^T of step i+2 is produced while step i+1 is still being computed on, and the
//     compute warps start the exponentials of a step the moment they have finished the step before;
//   - dP^T as a hand-off of its own (it can only be produced once dQ of the step before has left TMEM), awaited between
//     the exponentials and the dS arithmetic;
//   - a dQ staging buffer of its own, so a Q / dO stage is free for the next load as soon as the products that read it
//     are done instead of after the reduce-add.
//   - P^T as a hand-off of its own too: product (3) dV += P^T dO of a step is issued as soon as its P^T is in TMEM.
// Per step the chain is then: dS^T ready -> dQ, dK -> dP^T of the next step -> its dS arithmetic; the next step's
// exponentials, its dV product and the load and S^T product of the step after run underneath.
// TMEM columns: S^T buffers at 0 and 128, dP^T / dQ at 256, dK at 384, dV at 448.
#pragma once

template <int R>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_d64_kernel(const __grid_constant__ BwdParams<R> p) {
    constexpr int D = 64;
    constexpr int kTileBytes = kT * D * 2;             // 16 KiB: one slab of [128 rows][64 columns]
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *sK = smem, *sV = smem + kTileBytes;
    constexpr int kQS = 3;                             // Q / dO stages: the load of step i+2 starts when step i-1 is done with
                                                       // its stage, a whole step before S^T of step i+2 is issued
    uint8_t *sQ = smem + 2 * kTileBytes;
    uint8_t *sdO = sQ + kQS * kTileBytes;
    uint8_t *sdS = sdO + kQS * kTileBytes;             // dS^T [key rows][query cols], two 64-column slabs (32 KiB)
    uint8_t *sStage = sdS + 2 * 16384;                 // dQ staging: two chunks of [128 rows][32 floats] (32 KiB)
    float *s_lse = reinterpret_cast<float *>(sStage + 2 * 16384);      // [kQS][128], already times log2(e)
    float *s_delta = s_lse + kQS * kT;                                 // [kQS][128], already times -scale
    BwdBars *bars = reinterpret_cast<BwdBars *>(s_delta + kQS * kT);

    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;

    if (tid == 0) {
        mbar_init(&bars->kv_full, 1); mbar_init(&bars->kv_empty, 1);
        for (int s = 0; s < kQS; ++s) {
            mbar_init(&bars->qdo_full[s], 1);
            mbar_init(&bars->qdo_mma_done[s], 1);
            mbar_init(&bars->stats_full[s], 1);
        }
        mbar_init(&bars->s_full_b[0], 1);
        mbar_init(&bars->s_full_b[1], 1);
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
    constexpr uint32_t kColST = 0 /* + 128 * buffer */, kColDP = 256, kColDK = 384, kColDV = 448;
    if (bars->abort_flag) goto bwd_done;

    if (warp < kBwdComputeWarps) {
        // ======================================================================= compute warps
        const int g = warp >> 2;                        // which 32-column quarter of the score tile
        const int row = tid & 127;                      // TMEM lane: key row
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; bwd_get_item(p, round, item); ++round, ++item_n) {
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const int buf = it_g & 1;                                   // S^T buffer of the step
                    const uint32_t stage = it_g % kQS, sph = (it_g / kQS) & 1;  // its Q / dO stage (row statistics with it)
                    const uint32_t st_col = tmem + kColST + 128 * buf + 32 * g + lane_addr;
                    BWD_WAIT(&bars->stats_full[stage], sph, 10, m);             // LSE and Delta of the query tile
                    BWD_WAIT(&bars->s_full_b[buf], (it_g >> 1) & 1, 11, m);
                    tc_fence_after();
                    uint32_t st[32], dp[32];
                    tmem_ld_x32(st_col, st);
                    tmem_wait_ld();
                    // the column window of an edge step (the diagonal, a ragged last tile), as in the 128-wide kernel
                    const bool diag = p.causal && m == item.n;
                    const bool edge = diag || (m + 1) * kT > p.S || (item.n + 1) * kT > p.S;
                    int c_lo = 0, c_hi = 32;
                    if (edge) {
                        if (diag) c_lo = row - 32 * g;
                        if (item.n * kT + row >= p.S) c_lo = 32;
                        if (p.S - m * kT - 32 * g < c_hi) c_hi = p.S - m * kT - 32 * g;
                    }
                    const float *lse_b = s_lse + stage * kT + 32 * g;
                    const float *del_b = s_delta + stage * kT + 32 * g;
                    // P^T = exp2(S^T scale log2e - LSE): needs the scores only (two instantiations: the common step carries
                    // no masking code)
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
                    // P^T (bf16) over this quarter's own score columns of the step's S^T buffer, stored before the wait for
                    // dP^T: the store needs the values, so the exponentials cannot be scheduled behind that wait
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
                    // dS^T = P^T (dP^T scale - Delta scale): dP^T arrives after dQ of the step before has left TMEM
                    BWD_WAIT(&bars->dp_full, it_g & 1, 12, m);
                    tc_fence_after();
                    tmem_ld_x32(tmem + kColDP + 32 * g + lane_addr, dp);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        const float4 d4 = *reinterpret_cast<const float4 *>(del_b + c);
                        const float dl[4] = {d4.x, d4.y, d4.z, d4.w};
                        float pv[4], dsv[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            pv[e] = __uint_as_float(st[c + e]);
                            dsv[e] = pv[e] * fmaf(__uint_as_float(dp[c + e]), p.scale, dl[e]);
                        }
                        dp[c >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                        dp[(c >> 1) + 1] = pack_bf16x2(dsv[2], dsv[3]);
                    }
                    // dS^T into the one shared buffer: its last readers, products (5) and (4) of the step before, were
                    // complete before dP^T of this step was (the tensor core finishes in issue order).
                    {
                        uint8_t *line = sdS + (g >> 1) * 16384 + row * 128;
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch)
                            *reinterpret_cast<uint4 *>(line + (((4 * (g & 1) + ch) ^ (row & 7)) << 4)) =
                                make_uint4(dp[4 * ch], dp[4 * ch + 1], dp[4 * ch + 2], dp[4 * ch + 3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->pds_ready);
                }
            }
            // ---- item done: dK_n (quarters 0, 1) / dV_n (quarters 2, 3) to global as bf16, 32 columns per quarter
            BWD_WAIT(&bars->dkdv_full, item_n & 1, 13, item.n);
            tc_fence_after();
            {
                __nv_bfloat16 *base = (g < 2 ? p.dk[item.r] : p.dv[item.r]) +
                                      (((size_t)item.bl * p.S + (size_t)item.n * kT + row) * p.Hkv_l + item.hkv) * p.Dg +
                                      32 * (g & 1);
                uint32_t rr[32];
                tmem_ld_x32(tmem + (g < 2 ? kColDK : kColDV) + 32 * (g & 1) + lane_addr, rr);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 o4;
                    o4.x = pack_bf16x2(__uint_as_float(rr[8 * i + 0]), __uint_as_float(rr[8 * i + 1]));
                    o4.y = pack_bf16x2(__uint_as_float(rr[8 * i + 2]), __uint_as_float(rr[8 * i + 3]));
                    o4.z = pack_bf16x2(__uint_as_float(rr[8 * i + 4]), __uint_as_float(rr[8 * i + 5]));
                    o4.w = pack_bf16x2(__uint_as_float(rr[8 * i + 6]), __uint_as_float(rr[8 * i + 7]));
                    if (32 * (g & 1) + i * 8 < p.Dg && item.n * kT + row < p.S)
                        *reinterpret_cast<uint4 *>(base + i * 8) = o4;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->dkdv_read);
        }
    } else if (warp < kBwdTmaWarp) {
        // ======================================================================= dQ drain warps
        // dQ_m (lane = query row, 64 fp32 columns) leaves TMEM into the staging buffer (two chunks of [128 rows][32 floats],
        // 128-byte swizzle); each warp adds its 32 rows of a chunk to the accumulator with one TMA reduce-add.
        reg_inc<104>();
        const int wq = warp & 3;
        const int row = tid & 127;
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        uint32_t it_g = 0;
        BwdItem item;
        for (int round = 0; bwd_get_item(p, round, item); ++round) {
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                const int h = item.hkv * p.q_per_kv + hq;
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    BWD_WAIT(&bars->dq_full, it_g & 1, 14, m);
                    tc_fence_after();
                    uint32_t v[64];
                    tmem_ld_x32(tmem + kColDP + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
                    tmem_ld_x32(tmem + kColDP + 32 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->dq_read);          // TMEM is free for the next dP^T
                    // this warp's rows of the staging buffer are free: lane 0 waited for the previous reduce-add's reads
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint8_t *line = sStage + c * 16384 + row * 128;
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch)
                            *reinterpret_cast<uint4 *>(line + ((ch ^ (row & 7)) << 4)) =
                                make_uint4(v[32 * c + 4 * ch], v[32 * c + 4 * ch + 1], v[32 * c + 4 * ch + 2], v[32 * c + 4 * ch + 3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        const int row0 = item.bl * p.S + m * kT + wq * 32;
#pragma unroll
                        for (int c = 0; c < 2; ++c)
                            if (32 * c < p.Dg)          // a chunk wholly past the head dimension is padding
                                tma_reduce_add_3d(&p.dq_acc[item.r], sStage + c * 16384 + wq * 4096, 32 * c, h, row0);
                        tma_store_commit();
                        tma_store_wait_read<0>();
                    }
                    __syncwarp();
                }
            }
        }
    } else {
      reg_dec<56>();
      if (warp == kBwdTmaWarp) {
        // ======================================================================= TMA producer
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; bwd_get_item(p, round, item); ++round, ++item_n) {
            BWD_WAIT(&bars->kv_empty, (item_n & 1) ^ 1, 20, item.n);
            if (lane == 0) {
                mbar_arrive_expect_tx(&bars->kv_full, 2 * kTileBytes);
                const int row0 = item.bl * p.S + item.n * kT;
                tma_load_3d(sK, &p.k[item.r], &bars->kv_full, 0, item.hkv, row0);
                tma_load_3d(sV, &p.v[item.r], &bars->kv_full, 0, item.hkv, row0);
            }
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                const int h = item.hkv * p.q_per_kv + hq;
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const uint32_t stage = it_g % kQS, ph = (it_g / kQS) & 1;
                    // the stage (tiles and row statistics) is free once products (3) and (4) of three steps ago are done
                    BWD_WAIT(&bars->qdo_mma_done[stage], ph ^ 1, 21, m);
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&bars->qdo_full[stage], 2 * kTileBytes);
                        const int row0 = item.bl * p.S + m * kT;
                        tma_load_3d(sQ + stage * kTileBytes, &p.q[item.r], &bars->qdo_full[stage], 0, h, row0);
                        tma_load_3d(sdO + stage * kTileBytes, &p.dout[item.r], &bars->qdo_full[stage], 0, h, row0);
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
        for (int round = 0; bwd_get_item(p, round, item); ++round, ++item_n) {
            const uint32_t steps = (uint32_t)p.q_per_kv * (uint32_t)(item.n_qt - item.m0);
            BWD_WAIT(&bars->kv_full, item_n & 1, 30, item.n);
            // (1) S^T = K Q^T of step `it` into its S^T buffer (the P^T that lived there was read by product (3) of step
            //     it-2, issued before)
            auto issue_s = [&](uint32_t it) -> bool {
                const uint32_t stage = it % kQS, buf = it & 1;
                if (!mbar_wait(&bars->qdo_full[stage], (it / kQS) & 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ss(tmem + kColST + 128 * buf, desc_k | (uint64_t)(aK + kk * 2),
                               desc_k | (uint64_t)(aQ + stage * (kTileBytes >> 4) + kk * 2), idesc_kk, kk > 0);
                    tc_commit(&bars->s_full_b[buf]);
                }
                return true;
            };
            // (2) dP^T = V dO^T of step `it`, once dQ of step it-1 has left its columns
            auto issue_dp = [&](uint32_t it) -> bool {
                const uint32_t stage = it % kQS;
                if (!mbar_wait(&bars->dq_read, (it & 1) ^ 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ss(tmem + kColDP, desc_k | (uint64_t)(aV + kk * 2),
                               desc_k | (uint64_t)(adO + stage * (kTileBytes >> 4) + kk * 2), idesc_kk, kk > 0);
                    tc_commit(&bars->dp_full);
                }
                return true;
            };
            // (3) dV += P^T dO of step `it`, as soon as its P^T is in TMEM: A = P^T in the step's S^T buffer, B = dO read
            //     MN-major.  The first one of an item also waits until dK / dV of the item before have been stored.
            auto issue_dv = [&](uint32_t it, bool first) -> bool {
                const uint32_t stage = it % kQS, buf = it & 1;
                if (!mbar_wait(&bars->p_ready, it & 1, &bars->abort_flag)) return false;
                if (first && !mbar_wait(&bars->dkdv_read, (item_n & 1) ^ 1, &bars->abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t do16 = adO + stage * (kTileBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk)
                        mma_ts(tmem + kColDV, tmem + kColST + 128 * buf + (kk / 2) * 32 + (kk % 2) * 8,
                               desc_mn | (uint64_t)(do16 + kk * 128), idesc_kn, kk > 0 ? 1u : (first ? 0u : 1u));
                }
                return true;
            };
            bool ok = issue_s(it_g) && issue_dp(it_g);
            if (ok && steps > 1) ok = issue_s(it_g + 1);
            if (ok) ok = issue_dv(it_g, true);
            if (!ok) { bars->abort_flag = 1; bwd_report(p.status, 3, 31, item.n); goto bwd_done; }
            for (uint32_t j = 0; j < steps; ++j) {
                const uint32_t it = it_g + j, stage = it % kQS;
                const uint32_t q16 = aQ + stage * (kTileBytes >> 4);
                BWD_WAIT(&bars->pds_ready, it & 1, 33, (int)j);
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t acc0 = j == 0 ? 0u : 1u;
                    // (5) dQ_m = dS K : A = the dS^T buffer read MN-major (query rows), B = K MN-major
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk)
                        mma_ss(tmem + kColDP, desc_mn | (uint64_t)(adS + kk * 128), desc_mn | (uint64_t)(aK + kk * 128),
                               idesc_nn, kk > 0);
                    tc_commit(&bars->dq_full);
                    // (4) dK += dS^T Q : A = dS^T from shared memory (K-major: query columns), B = Q MN-major
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                        mma_ss(tmem + kColDK, desc_k | (uint64_t)(adS + off), desc_mn | (uint64_t)(q16 + kk * 128),
                               idesc_kn, kk > 0 ? 1u : acc0);
                    }
                    tc_commit(&bars->qdo_mma_done[stage]);        // (3), issued a step ago, and (4) are done: the stage may be loaded again
                }
                ok = true;
                if (j + 1 < steps) ok = issue_dp(it + 1) && issue_dv(it + 1, false);
                if (ok && j + 2 < steps) ok = issue_s(it + 2);
                if (!ok) { bars->abort_flag = 1; bwd_report(p.status, 3, 35, (int)j); goto bwd_done; }
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
