// The projections on either side of the attention core (Section II-A: Q = X W_Q, K = X W_K, V = X W_V per
// head, MultiHead = Concat(H_i) W_O), for every virtual rank's sequence shard in one launch:
//
//   C_r[M, N] = A_r[M, K] . W[N, K]^T      bf16 operands, fp32 accumulation in TMEM, bf16 result
//
// with the output columns cut into up to three segments that go to different tensors (Q | K | V, each the
// rank's sequence-sharded [tokens][heads*D] matrix), so the QKV projection writes the shards the reshard reads.
//
// Persistent, one CTA per SM, tile 128 x 256, K in blocks of 64 (one 128-byte-swizzled TMA box per operand):
//   warp 0      TMA producer, 4-stage ring (A 16 KiB + W 32 KiB per stage)
//   warp 1      tcgen05.mma issuer (M = 128, N = 256, K = 16), two 256-column TMEM accumulators so that the
//               epilogue of one tile runs under the main loop of the next
//   warps 2-5   epilogue: tcgen05.ld -> bf16 -> 16-byte global stores (a thread owns an output row)
// Tiles of one row block (all column tiles) are adjacent in the schedule: A is read once from HBM, W stays in L2.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tmap.cuh"

int *basp_status_device_ptr();

namespace {

using namespace ptx;

constexpr int kGemmThreads = 192;
constexpr int kBM = 128, kBN = 256, kBK = 64, kGemmStages = 4;
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2;

template <int R>
struct GemmParams {
    CUtensorMap a[R];
    CUtensorMap w;
    int n_ranks, M, N, K;
    int M_last;                            // rows of the last rank of a group (= M unless the group size does not divide S)
    int n_seg;
    int seg_begin[3], seg_ld[3];           // first output column of the segment; row pitch of its tensor (elements)
    __nv_bfloat16 *seg_ptr[3][R];
    // rotary position embedding applied to the first `rope_segs` segments (Q, K) before the rounding to bf16:
    // head dimension 2 * rope_half, tables [rope_half][rope_S] of cos and sin (feature-major: the 32 rows of a warp are
    // 32 consecutive positions, so a warp's read of one feature is one 128-byte line), position of a row = the token's
    // place in its sequence: local rank (r mod rope_K) * rope_T + row mod rope_T
    int rope_segs, rope_half, rope_T, rope_K, rope_S;
    int rope_T_last;                       // tokens per sequence of a group's last rank
    const float *rope_cos, *rope_sin;
    int *status;
};

struct GemmBars {
    uint64_t full[kGemmStages], empty[kGemmStages], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

#define GEMM_WAIT(bar, parity, role, detail)                                   \
    do {                                                                        \
        if (!mbar_wait((bar), (parity), &bars.abort_flag)) {                   \
            bars.abort_flag = 1;                                                \
            if (atomicCAS(p.status, 0, 5) == 0) {                               \
                p.status[1] = (role); p.status[2] = (int)blockIdx.x; p.status[3] = (detail); \
            }                                                                   \
            goto gemm_done;                                                     \
        }                                                                       \
    } while (0)

template <int R>
__global__ void __launch_bounds__(kGemmThreads, 1) proj_gemm_kernel(const __grid_constant__ GemmParams<R> p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = smem;                                    // kGemmStages x 16 KiB
    uint8_t *sB = smem + kGemmStages * kABytes;            // kGemmStages x 32 KiB
    __shared__ GemmBars bars;

    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
    const int tiles_m = (p.M + kBM - 1) / kBM, tiles_n = p.N / kBN, k_blocks = p.K / kBK;
    const int total = p.n_ranks * tiles_m * tiles_n;

    if (tid == 0) {
        for (int s = 0; s < kGemmStages; ++s) { mbar_init(&bars.full[s], 1); mbar_init(&bars.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&bars.acc_full[a], 1); mbar_init(&bars.acc_empty[a], 4); }
        bars.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(&bars.tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (lane 0 issues)
        uint32_t it = 0;
        for (int tile = blockIdx.x; tile < total; tile += gridDim.x) {
            const int n = tile % tiles_n, m = (tile / tiles_n) % tiles_m, r = tile / (tiles_n * tiles_m);
            for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                const uint32_t s = it % kGemmStages, ph = (it / kGemmStages) & 1;
                GEMM_WAIT(&bars.empty[s], ph ^ 1, 0, kb);
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bars.full[s], kABytes + kBBytes);
                    tma_load_3d(sA + s * kABytes, &p.a[r], &bars.full[s], kb * kBK, 0, m * kBM);
                    tma_load_3d(sB + s * kBBytes, &p.w, &bars.full[s], kb * kBK, 0, n * kBN);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (lane 0 issues)
        const uint32_t idesc = make_idesc_bf16(kBM, kBN, false, false);
        const uint64_t desc = make_smem_desc_sw128(0, 16, 1024);
        const uint32_t a16 = smem_u32(sA) >> 4, b16 = smem_u32(sB) >> 4;
        uint32_t it = 0, tile_cnt = 0;
        for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++tile_cnt) {
            const uint32_t acc = tile_cnt & 1;
            GEMM_WAIT(&bars.acc_empty[acc], ((tile_cnt >> 1) & 1) ^ 1, 1, tile);
            tc_fence_after();
            for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                const uint32_t s = it % kGemmStages, ph = (it / kGemmStages) & 1;
                GEMM_WAIT(&bars.full[s], ph, 2, kb);
                tc_fence_after();
                if (lane == 0) {
                    const uint64_t da = desc | (uint64_t)(a16 + s * (kABytes >> 4));
                    const uint64_t db = desc | (uint64_t)(b16 + s * (kBBytes >> 4));
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk)
                        mma_ss(tmem + acc * kBN, da + kk * 2, db + kk * 2, idesc, (kb > 0) || (kk > 0));
                    tc_commit(&bars.empty[s]);
                }
            }
            if (lane == 0) tc_commit(&bars.acc_full[acc]);
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                       // the TMEM lanes this warp can reach
        const int row = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        uint32_t tile_cnt = 0;
        for (int tile = blockIdx.x; tile < total; tile += gridDim.x, ++tile_cnt) {
            const int n = tile % tiles_n, m = (tile / tiles_n) % tiles_m, r = tile / (tiles_n * tiles_m);
            const uint32_t acc = tile_cnt & 1;
            int seg = 0;
            while (seg + 1 < p.n_seg && n * kBN >= p.seg_begin[seg + 1]) ++seg;
            const int grow = m * kBM + row;
            const bool short_rank = r % p.rope_K == p.rope_K - 1;
            const int Mr = short_rank ? p.M_last : p.M;
            __nv_bfloat16 *dst = p.seg_ptr[seg][r] + (size_t)grow * p.seg_ld[seg] + (n * kBN - p.seg_begin[seg]);
            GEMM_WAIT(&bars.acc_full[acc], (tile_cnt >> 1) & 1, 3, tile);
            tc_fence_after();
            if (seg < p.rope_segs) {
                // Rotate-half form: within a head, column j < D/2 pairs with column j + D/2:
                //   y_j = x_j cos(t_j) - x_{j+D/2} sin(t_j),   y_{j+D/2} = x_{j+D/2} cos(t_j) + x_j sin(t_j),   t_j = pos * theta_j
                // on the fp32 accumulators, one rounding to bf16 afterwards.  A thread owns a row, so both halves of every
                // head of the tile are in its own TMEM lane.
                const int half = p.rope_half, D2 = 2 * half;
                const int pos = (r % p.rope_K) * p.rope_T + (grow % (short_rank ? p.rope_T_last : p.rope_T));
                const float *ct = p.rope_cos + pos, *sn = p.rope_sin + pos;
                for (int j0 = 0; j0 < half; j0 += 32) {
                    // the angles depend on (position, feature) only: one fetch of 32 features serves every head of the tile
                    float cv[32], sv[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const size_t off = (size_t)(j0 + e) * p.rope_S;
                        cv[e] = __ldg(ct + off);
                        sv[e] = __ldg(sn + off);
                    }
                    for (int hb = 0; hb < kBN; hb += D2) {
                        uint32_t lo[32], hi[32];
                        tmem_ld_x32(tmem + acc * kBN + hb + j0 + lane_addr, lo);
                        tmem_ld_x32(tmem + acc * kBN + hb + half + j0 + lane_addr, hi);
                        tmem_wait_ld();
                        if (hb + D2 == kBN && j0 + 32 == half) {    // that was the last read of the accumulator
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&bars.acc_empty[acc]);
                        }
                        if (grow < Mr) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                float yl[8], yh[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const float xl = __uint_as_float(lo[8 * i + e]), xh = __uint_as_float(hi[8 * i + e]);
                                    yl[e] = xl * cv[8 * i + e] - xh * sv[8 * i + e];
                                    yh[e] = xh * cv[8 * i + e] + xl * sv[8 * i + e];
                                }
                                uint4 o4;
                                o4.x = pack_bf16x2(yl[0], yl[1]); o4.y = pack_bf16x2(yl[2], yl[3]);
                                o4.z = pack_bf16x2(yl[4], yl[5]); o4.w = pack_bf16x2(yl[6], yl[7]);
                                *reinterpret_cast<uint4 *>(dst + hb + j0 + i * 8) = o4;
                                o4.x = pack_bf16x2(yh[0], yh[1]); o4.y = pack_bf16x2(yh[2], yh[3]);
                                o4.z = pack_bf16x2(yh[4], yh[5]); o4.w = pack_bf16x2(yh[6], yh[7]);
                                *reinterpret_cast<uint4 *>(dst + hb + half + j0 + i * 8) = o4;
                            }
                        }
                    }
                }
                continue;
            }
#pragma unroll
            for (int c = 0; c < kBN / 32; ++c) {
                uint32_t rr[32];
                tmem_ld_x32(tmem + acc * kBN + c * 32 + lane_addr, rr);
                tmem_wait_ld();
                if (c == kBN / 32 - 1) {                    // the accumulator is in registers: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars.acc_empty[acc]);
                }
                if (grow < Mr) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 o4;
                        o4.x = pack_bf16x2(__uint_as_float(rr[8 * i + 0]), __uint_as_float(rr[8 * i + 1]));
                        o4.y = pack_bf16x2(__uint_as_float(rr[8 * i + 2]), __uint_as_float(rr[8 * i + 3]));
                        o4.z = pack_bf16x2(__uint_as_float(rr[8 * i + 4]), __uint_as_float(rr[8 * i + 5]));
                        o4.w = pack_bf16x2(__uint_as_float(rr[8 * i + 6]), __uint_as_float(rr[8 * i + 7]));
                        *reinterpret_cast<uint4 *>(dst + c * 32 + i * 8) = o4;
                    }
                }
            }
        }
    }

gemm_done:
    tc_fence_before();
    __syncthreads();
    if (bars.abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem, 512);
}

#undef GEMM_WAIT

struct Segment {
    int cols;
    void *const *ptrs;
};

struct Rope {
    int segs;                 // leading segments to rotate (0 = none)
    const float *cos, *sin;   // [D/2][S] each
};

template <int R>
int gemm_launch(const basp_plan *pl, const void *const *a, const void *w, int M, int N, int K, const Segment *segs,
                int n_seg, const Rope &rope, cudaStream_t st) {
    GemmParams<R> prm;
    for (int r = 0; r < pl->N; ++r) {
        int rc = tmap::encode_rows_heads_d(&prm.a[r], a[r], (uint64_t)pl->Bl * basp_rank_tokens(pl, r % pl->K), 1, (uint64_t)K, kBM);
        if (rc != BASP_OK) return rc;
    }
    int rc = tmap::encode_rows_heads_d(&prm.w, w, (uint64_t)N, 1, (uint64_t)K, kBN);
    if (rc != BASP_OK) return rc;
    prm.n_ranks = pl->N; prm.M = M; prm.M_last = pl->Bl * pl->T_last; prm.N = N; prm.K = K; prm.n_seg = n_seg;
    int col = 0;
    for (int s = 0; s < n_seg; ++s) {
        prm.seg_begin[s] = col;
        prm.seg_ld[s] = segs[s].cols;
        for (int r = 0; r < pl->N; ++r) prm.seg_ptr[s][r] = (__nv_bfloat16 *)segs[s].ptrs[r];
        col += segs[s].cols;
    }
    prm.rope_segs = rope.segs; prm.rope_half = pl->D / 2; prm.rope_T = pl->T; prm.rope_T_last = pl->T_last; prm.rope_K = pl->K; prm.rope_S = pl->S;
    prm.rope_cos = rope.cos; prm.rope_sin = rope.sin;
    prm.status = basp_status_device_ptr();
    if (!prm.status) return BASP_ERR_CUDA;
    int dev = 0, sms = 0;
    BASP_CUDA_TRY(cudaGetDevice(&dev));
    BASP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long tiles = (long long)pl->N * ((M + kBM - 1) / kBM) * (N / kBN);
    const int grid = (int)(tiles < sms ? tiles : sms);
    const int smem = kGemmStages * (kABytes + kBBytes) + 1024;
    BASP_CUDA_TRY(cudaFuncSetAttribute(proj_gemm_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    proj_gemm_kernel<R><<<grid, kGemmThreads, smem, st>>>(prm);
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(1);
    return BASP_OK;
}

int gemm_dispatch(const basp_plan *pl, const void *const *a, const void *w, int N, int K, const Segment *segs, int n_seg,
                  const Rope &rope, void *stream) {
    const int M = pl->Bl * pl->T;
    if (K <= 0 || K % kBK != 0) return BASP_ERR_UNSUPPORTED;
    for (int s = 0; s < n_seg; ++s)
        if (segs[s].cols % kBN != 0) return BASP_ERR_UNSUPPORTED;
    if (!w || !a) return BASP_ERR_NULL;
    if (!aligned16(w)) return BASP_ERR_ALIGN;
    for (int r = 0; r < pl->N; ++r) {
        if (!a[r]) return BASP_ERR_NULL;
        if (!aligned16(a[r])) return BASP_ERR_ALIGN;
        for (int s = 0; s < n_seg; ++s) {
            if (!segs[s].ptrs || !segs[s].ptrs[r]) return BASP_ERR_NULL;
            if (!aligned16(segs[s].ptrs[r])) return BASP_ERR_ALIGN;
            for (int r2 = 0; r2 < pl->N; ++r2)
                if (segs[s].ptrs[r] == a[r2] || segs[s].ptrs[r] == w) return BASP_ERR_ALIAS;
        }
    }
    if (rope.segs > 0) {
        // a head's two halves must be whole 32-column chunks of one tile: D = 64 or 128
        if (pl->D != 64 && pl->D != 128) return BASP_ERR_UNSUPPORTED;
        if (!rope.cos || !rope.sin) return BASP_ERR_NULL;
        if (((uintptr_t)rope.cos & 3) || ((uintptr_t)rope.sin & 3)) return BASP_ERR_ALIGN;
    }
    if (pl->N <= 8) return gemm_launch<8>(pl, a, w, M, N, K, segs, n_seg, rope, (cudaStream_t)stream);
    return gemm_launch<BASP_MAX_RANKS>(pl, a, w, M, N, K, segs, n_seg, rope, (cudaStream_t)stream);
}

}  // namespace

extern "C" int basp_qkv_proj(const basp_plan *plan, int hidden, const void *const *x_seq, const void *w_qkv,
                             void *const *q_seq, void *const *k_seq, void *const *v_seq, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    const Segment segs[3] = {{plan->Hq * plan->D, q_seq}, {plan->Hkv * plan->D, k_seq}, {plan->Hkv * plan->D, v_seq}};
    return gemm_dispatch(plan, x_seq, w_qkv, (plan->Hq + 2 * plan->Hkv) * plan->D, hidden, segs, 3, Rope{0, nullptr, nullptr}, stream);
}

extern "C" int basp_qkv_proj_rope(const basp_plan *plan, int hidden, const void *const *x_seq, const void *w_qkv,
                                  const float *rope_cos, const float *rope_sin, void *const *q_seq, void *const *k_seq,
                                  void *const *v_seq, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    const Segment segs[3] = {{plan->Hq * plan->D, q_seq}, {plan->Hkv * plan->D, k_seq}, {plan->Hkv * plan->D, v_seq}};
    return gemm_dispatch(plan, x_seq, w_qkv, (plan->Hq + 2 * plan->Hkv) * plan->D, hidden, segs, 3,
                         Rope{2, rope_cos, rope_sin}, stream);
}

extern "C" int basp_out_proj(const basp_plan *plan, int hidden, const void *const *o_seq, const void *w_o,
                             void *const *y_seq, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    if (hidden <= 0) return BASP_ERR_INVALID;
    const Segment segs[1] = {{hidden, y_seq}};
    return gemm_dispatch(plan, o_seq, w_o, hidden, plan->Hq * plan->D, segs, 1, Rope{0, nullptr, nullptr}, stream);
}
