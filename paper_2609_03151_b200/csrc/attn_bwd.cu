// Backward of causal attention over each virtual rank's head slice (the gradient of the
// Section II-A equation by the chain rule), on tcgen05 tensor cores.
//
//   P_ij = exp(scale q_i.k_j - LSE_i),  Delta_i = dO_i.O_i,
//   dV_j = sum_i P_ij dO_i,  dP_ij = dO_i.v_j,  dS_ij = P_ij (dP_ij - Delta_i),
//   dQ_i = scale sum_j dS_ij k_j,  dK_j = scale sum_i dS_ij q_i.
//
// One persistent CTA per SM.  A work item is one 128-row KV tile n of one (rank, sequence, KV head);
// the CTA walks the query heads of the GQA group and the query tiles m >= n, keeping dK_n and dV_n in
// TMEM for the whole item (no atomics for dK/dV).  Scores are computed TRANSPOSED (S^T = K Q^T, rows
// = keys) so that P^T and dS^T are directly the A operands of the dV and dK products.  Per step:
//   (1) S^T  = K Q^T        SS   -> TMEM [0,128)
//   (2) dP^T = V dO^T       SS   -> TMEM [128,256)
//   compute warps: P^T = exp2(..), dS^T = scale P^T (dP^T - Delta)  ->  P^T bf16 to TMEM, dS^T bf16 to smem
//   (3) dV  += P^T dO       TS   -> TMEM [384,512)
//   (4) dK  += dS^T Q       SS   -> TMEM [256,384)
//   (5) dQ_m = dS K         SS   -> TMEM [128,256)  (A = the dS^T buffer read MN-major)
//   compute warps: dQ_m added to the fp32 accumulator in global memory (red.add, order not fixed).
// Helper kernels: Delta = rowsum(dO * O); fp32 dQ accumulator -> bf16.
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tmap.cuh"

int *basp_status_device_ptr();

namespace {

using namespace ptx;

constexpr int kT = 128;
constexpr int kBwdThreads = 320;          // 8 compute warps + TMA warp + MMA warp

template <int R>
struct BwdParams {
    CUtensorMap q[R], k[R], v[R], dout[R];
    const float *lse[R];
    const float *delta[R];
    float *dq_acc[R];
    __nv_bfloat16 *dk[R], *dv[R];
    int n_ranks, Bl, S, Hq_l, Hkv_l, q_per_kv, causal;
    float scale, scale_log2;
    int *status;
};

struct BwdItem {
    int r, bl, hkv, n, m0, n_qt;
};

template <int R>
__device__ __forceinline__ bool bwd_get_item(const BwdParams<R> &p, int round, BwdItem &it) {
    const int n_kt = p.S / kT;
    const int streams = p.n_ranks * p.Bl * p.Hkv_l;
    const int total = n_kt * streams;
    const int pos = (round & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
    const int i = round * (int)gridDim.x + pos;
    if (i >= total) return false;
    it.n = i / streams;                    // low key tiles are seen by the most query tiles: longest first
    int rem = i - it.n * streams;
    it.hkv = rem % p.Hkv_l;
    rem /= p.Hkv_l;
    it.bl = rem % p.Bl;
    it.r = rem / p.Bl;
    it.n_qt = n_kt;
    it.m0 = p.causal ? it.n : 0;
    return true;
}

struct BwdBars {
    uint64_t kv_full, kv_empty, qdo_full[2], qdo_empty[2];
    uint64_t s_full, stats_full, pds_ready, dq_full, dq_read, dkdv_full, dkdv_read;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void bwd_report(int *status, int code, int role, int detail) {
    if (atomicCAS(status, 0, code) == 0) {
        status[1] = role;
        status[2] = (int)blockIdx.x;
        status[3] = detail;
    }
}

#define BWD_WAIT(bar, parity, role, detail)                                    \
    do {                                                                        \
        if (!mbar_wait((bar), (parity), &bars->abort_flag)) {                  \
            bars->abort_flag = 1;                                               \
            bwd_report(p.status, 3, (role), (detail));                          \
            goto bwd_done;                                                      \
        }                                                                       \
    } while (0)

__device__ __forceinline__ void red_add_v4(float *addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

template <int R>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_kernel(const __grid_constant__ BwdParams<R> p) {
    constexpr int D = 128;
    constexpr int kTileBytes = kT * D * 2;             // 32 KiB
    // dynamic shared memory only, so that the tile area starts at the (1024-byte aligned) window base
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *sK = smem, *sV = smem + kTileBytes;
    uint8_t *sQ = smem + 2 * kTileBytes;               // 2 stages
    uint8_t *sdO = smem + 4 * kTileBytes;              // 2 stages
    uint8_t *sdS = smem + 6 * kTileBytes;              // dS^T [key rows][query cols], two 64-column slabs
    float *s_lse = reinterpret_cast<float *>(smem + 7 * kTileBytes);   // [2][128], already times log2(e)
    float *s_delta = s_lse + 2 * kT;                                   // [2][128]
    BwdBars *bars = reinterpret_cast<BwdBars *>(s_delta + 2 * kT);

    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;

    if (tid == 0) {
        mbar_init(&bars->kv_full, 1); mbar_init(&bars->kv_empty, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(&bars->qdo_full[s], 1); mbar_init(&bars->qdo_empty[s], 1); }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->stats_full, 8);
        mbar_init(&bars->pds_ready, 8);
        mbar_init(&bars->dq_full, 1);
        mbar_init(&bars->dq_read, 8);
        mbar_init(&bars->dkdv_full, 1);
        mbar_init(&bars->dkdv_read, 8);
        bars->abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
        if (bars->abort_flag) bwd_report(p.status, 4, 0, (int)(smem_u32(smem) & 1023u));
        fence_mbar_init();
    }
    if (warp == 8) { tmem_alloc(&bars->tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    constexpr uint32_t kColST = 0, kColDP = 128, kColDK = 256, kColDV = 384;
    if (bars->abort_flag) goto bwd_done;

    if (warp < 8) {
        // ======================================================================= compute warps
        const int w = warp >> 2;                        // which 64-column half of the score tile
        const int row = tid & 127;                      // TMEM lane: key row (scores) / query row (dQ)
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; bwd_get_item(p, round, item); ++round, ++item_n) {
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                const int h = item.hkv * p.q_per_kv + hq;
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const int buf = it_g & 1;
                    {   // row statistics of the query tile: LSE (in log2 units) and Delta
                        const size_t off = ((size_t)item.bl * p.Hq_l + h) * p.S + (size_t)m * kT + row;
                        if (w == 0) s_lse[buf * kT + row] = p.lse[item.r][off] * 1.4426950408889634f;
                        else s_delta[buf * kT + row] = p.delta[item.r][off];
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars->stats_full);
                    }
                    BWD_WAIT(&bars->stats_full, it_g & 1, 10, m);
                    BWD_WAIT(&bars->s_full, it_g & 1, 11, m);
                    tc_fence_after();
                    uint32_t st[64], dp[64];
                    tmem_ld_x32(tmem + kColST + 64 * w + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&st[0]));
                    tmem_ld_x32(tmem + kColST + 64 * w + 32 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&st[32]));
                    tmem_ld_x32(tmem + kColDP + 64 * w + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
                    tmem_ld_x32(tmem + kColDP + 64 * w + 32 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
                    tmem_wait_ld();
                    const bool diag = p.causal && m == item.n;
                    const float *lse_b = s_lse + buf * kT + 64 * w;
                    const float *del_b = s_delta + buf * kT + 64 * w;
#pragma unroll
                    for (int c = 0; c < 64; c += 2) {
                        float p0 = exp2_approx(fmaf(__uint_as_float(st[c]), p.scale_log2, -lse_b[c]));
                        float p1 = exp2_approx(fmaf(__uint_as_float(st[c + 1]), p.scale_log2, -lse_b[c + 1]));
                        if (diag) {                      // query 64w+c sees key `row` iff it is not earlier
                            if (64 * w + c < row) p0 = 0.f;
                            if (64 * w + c + 1 < row) p1 = 0.f;
                        }
                        const float d0 = p0 * (__uint_as_float(dp[c]) - del_b[c]) * p.scale;
                        const float d1 = p1 * (__uint_as_float(dp[c + 1]) - del_b[c + 1]) * p.scale;
                        st[c >> 1] = pack_bf16x2(p0, p1);
                        dp[c >> 1] = pack_bf16x2(d0, d1);
                    }
                    // P^T (bf16) over this half's own score columns: TMEM columns 64w .. 64w+31
                    tmem_st_x32(tmem + kColST + 64 * w + lane_addr, *reinterpret_cast<const uint32_t(*)[32]>(&st[0]));
                    // dS^T row `row`, query columns 64w..64w+63 = one 128-byte line of slab w (128-byte swizzle)
                    {
                        uint8_t *line = sdS + w * 16384 + row * 128;
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch)
                            *reinterpret_cast<uint4 *>(line + ((ch ^ (row & 7)) << 4)) =
                                make_uint4(dp[4 * ch], dp[4 * ch + 1], dp[4 * ch + 2], dp[4 * ch + 3]);
                    }
                    fence_proxy_async_smem();
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->pds_ready);

                    // dQ_m tile: lane = query row, this half owns head-dim columns 64w .. 64w+63
                    BWD_WAIT(&bars->dq_full, it_g & 1, 12, m);
                    tc_fence_after();
                    uint32_t dq[64];
                    tmem_ld_x32(tmem + kColDP + 64 * w + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&dq[0]));
                    tmem_ld_x32(tmem + kColDP + 64 * w + 32 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&dq[32]));
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->dq_read);
                    float *dst = p.dq_acc[item.r] +
                                 (((size_t)item.bl * p.S + (size_t)m * kT + row) * p.Hq_l + h) * D + 64 * w;
#pragma unroll
                    for (int c = 0; c < 64; c += 4)
                        red_add_v4(dst + c, __uint_as_float(dq[c]), __uint_as_float(dq[c + 1]),
                                   __uint_as_float(dq[c + 2]), __uint_as_float(dq[c + 3]));
                }
            }
            // ---- item done: dK_n (half 0) / dV_n (half 1) to global as bf16
            BWD_WAIT(&bars->dkdv_full, item_n & 1, 13, item.n);
            tc_fence_after();
            {
                __nv_bfloat16 *base = (w == 0 ? p.dk[item.r] : p.dv[item.r]) +
                                      (((size_t)item.bl * p.S + (size_t)item.n * kT + row) * p.Hkv_l + item.hkv) * D;
                const uint32_t col0 = (w == 0 ? kColDK : kColDV);
#pragma unroll
                for (int cc = 0; cc < D / 32; ++cc) {
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
                        *reinterpret_cast<uint4 *>(base + cc * 32 + i * 8) = o4;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->dkdv_read);
        }
    } else if (warp == 8) {
        // ======================================================================= TMA producer
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; bwd_get_item(p, round, item); ++round, ++item_n) {
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
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const uint32_t stage = it_g & 1, ph = (it_g >> 1) & 1;
                    BWD_WAIT(&bars->qdo_empty[stage], ph ^ 1, 21, m);
                    if (lane == 0) {
                        mbar_arrive_expect_tx(&bars->qdo_full[stage], 2 * kTileBytes);
                        const int row0 = item.bl * p.S + m * kT;
                        for (int s = 0; s < 2; ++s) {
                            tma_load_3d(sQ + stage * kTileBytes + s * 16384, &p.q[item.r], &bars->qdo_full[stage], s * 64, h, row0);
                            tma_load_3d(sdO + stage * kTileBytes + s * 16384, &p.dout[item.r], &bars->qdo_full[stage], s * 64, h, row0);
                        }
                    }
                }
            }
        }
    } else if (warp == 9) {
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
            BWD_WAIT(&bars->kv_full, item_n & 1, 30, item.n);
            bool first = true;
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const uint32_t stage = it_g & 1, ph = (it_g >> 1) & 1;
                    const uint32_t q16 = aQ + stage * (kTileBytes >> 4), do16 = adO + stage * (kTileBytes >> 4);
                    BWD_WAIT(&bars->qdo_full[stage], ph, 31, m);
                    tc_fence_after();
                    if (lane == 0) {        // (1) S^T = K Q^T
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                            mma_ss(tmem + kColST, desc_k | (uint64_t)(aK + off), desc_k | (uint64_t)(q16 + off), idesc_kk, kk > 0);
                        }
                    }
                    BWD_WAIT(&bars->dq_read, (it_g & 1) ^ 1, 32, m);          // previous dQ tile has left TMEM
                    tc_fence_after();
                    if (lane == 0) {        // (2) dP^T = V dO^T
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                            mma_ss(tmem + kColDP, desc_k | (uint64_t)(aV + off), desc_k | (uint64_t)(do16 + off), idesc_kk, kk > 0);
                        }
                        tc_commit(&bars->s_full);
                    }
                    BWD_WAIT(&bars->pds_ready, it_g & 1, 33, m);
                    if (first) BWD_WAIT(&bars->dkdv_read, (item_n & 1) ^ 1, 34, item.n);
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t acc0 = first ? 0u : 1u;
                        // (3) dV += P^T dO : A = P^T in TMEM (query index along K: 8 columns per 16 queries,
                        //     the second half of the queries starts at column 64), B = dO read MN-major
#pragma unroll
                        for (int kk = 0; kk < kT / 16; ++kk)
                            mma_ts(tmem + kColDV, tmem + kColST + (kk / 4) * 64 + (kk % 4) * 8,
                                   desc_mn | (uint64_t)(do16 + kk * 128), idesc_kn, kk > 0 ? 1u : acc0);
                        // (4) dK += dS^T Q : A = dS^T from shared memory (K-major: query columns), B = Q MN-major
#pragma unroll
                        for (int kk = 0; kk < kT / 16; ++kk) {
                            const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                            mma_ss(tmem + kColDK, desc_k | (uint64_t)(adS + off), desc_mn | (uint64_t)(q16 + kk * 128),
                                   idesc_kn, kk > 0 ? 1u : acc0);
                        }
                        // (5) dQ_m = dS K : A = the same buffer read MN-major (query rows), B = K MN-major
#pragma unroll
                        for (int kk = 0; kk < kT / 16; ++kk)
                            mma_ss(tmem + kColDP, desc_mn | (uint64_t)(adS + kk * 128), desc_mn | (uint64_t)(aK + kk * 128),
                                   idesc_nn, kk > 0);
                        tc_commit(&bars->dq_full);
                        tc_commit(&bars->qdo_empty[stage]);
                    }
                    first = false;
                }
            }
            if (lane == 0) {
                tc_commit(&bars->dkdv_full);
                tc_commit(&bars->kv_empty);
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
    if (warp == 8) tmem_dealloc(tmem, 512);
}

#undef BWD_WAIT

// Delta[bl][h][s] = sum_d O[bl][s][h][d] * dO[bl][s][h][d]; one 16-lane group per (s, h) row of D = 128.
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __nv_bfloat16 *__restrict__ o,
                                                        const __nv_bfloat16 *__restrict__ dout,
                                                        float *__restrict__ delta, int Bl, int S, int H, int D) {
    const int lanes = D / 8;                            // threads per row (16 bytes each)
    const long long rows = (long long)Bl * S * H;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long rowi = gid / lanes;
    const int part = (int)(gid % lanes);
    float acc = 0.f;
    if (rowi < rows) {
        const uint4 a = *reinterpret_cast<const uint4 *>(o + rowi * D + part * 8);
        const uint4 b = *reinterpret_cast<const uint4 *>(dout + rowi * D + part * 8);
        const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc += __uint_as_float(av[i] << 16) * __uint_as_float(bv[i] << 16);
            acc += __uint_as_float(av[i] & 0xffff0000u) * __uint_as_float(bv[i] & 0xffff0000u);
        }
    }
    for (int off = lanes / 2; off > 0; off >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, off, lanes);
    if (rowi < rows && part == 0) {
        const long long h = rowi % H, s = (rowi / H) % S, bl = rowi / ((long long)H * S);
        delta[(bl * H + h) * S + s] = acc;
    }
}

// bf16(dQ accumulator), 8 elements per thread.
__global__ void __launch_bounds__(256) bwd_dq_convert_kernel(const float *__restrict__ acc,
                                                             __nv_bfloat16 *__restrict__ out, long long n8) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const float4 a = reinterpret_cast<const float4 *>(acc)[2 * i], b = reinterpret_cast<const float4 *>(acc)[2 * i + 1];
    uint4 o;
    o.x = pack_bf16x2(a.x, a.y); o.y = pack_bf16x2(a.z, a.w);
    o.z = pack_bf16x2(b.x, b.y); o.w = pack_bf16x2(b.z, b.w);
    reinterpret_cast<uint4 *>(out)[i] = o;
}

size_t bwd_acc_bytes(const basp_plan *p) { return (size_t)p->Bl * p->S * p->Hq_l * p->D * sizeof(float); }
size_t bwd_delta_bytes(const basp_plan *p) { return (((size_t)p->Bl * p->Hq_l * p->S * sizeof(float)) + 255) & ~(size_t)255; }

template <int R>
int bwd_launch(const basp_plan *pl, const void *const *q, const void *const *k, const void *const *v,
               const void *const *o, const void *const *dout, const float *const *lse, void *const *dq,
               void *const *dk, void *const *dv, char *ws, float scale, cudaStream_t st) {
    BwdParams<R> prm;
    const uint64_t rows = (uint64_t)pl->Bl * pl->S;
    const size_t acc_b = bwd_acc_bytes(pl), del_b = bwd_delta_bytes(pl);
    float *acc0 = reinterpret_cast<float *>(ws);
    float *del0 = reinterpret_cast<float *>(ws + (size_t)pl->N * acc_b);
    for (int r = 0; r < pl->N; ++r) {
        int rc = tmap::encode_rows_heads_d(&prm.q[r], q[r], rows, pl->Hq_l, pl->D, kT);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.k[r], k[r], rows, pl->Hkv_l, pl->D, kT);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.v[r], v[r], rows, pl->Hkv_l, pl->D, kT);
        if (rc == BASP_OK) rc = tmap::encode_rows_heads_d(&prm.dout[r], dout[r], rows, pl->Hq_l, pl->D, kT);
        if (rc != BASP_OK) return rc;
        prm.lse[r] = lse[r];
        prm.dq_acc[r] = reinterpret_cast<float *>(reinterpret_cast<char *>(acc0) + (size_t)r * acc_b);
        prm.delta[r] = reinterpret_cast<float *>(reinterpret_cast<char *>(del0) + (size_t)r * del_b);
        prm.dk[r] = (__nv_bfloat16 *)dk[r];
        prm.dv[r] = (__nv_bfloat16 *)dv[r];
    }
    prm.n_ranks = pl->N; prm.Bl = pl->Bl; prm.S = pl->S; prm.Hq_l = pl->Hq_l; prm.Hkv_l = pl->Hkv_l;
    prm.q_per_kv = pl->Hq / pl->Hkv; prm.causal = pl->causal;
    prm.scale = scale == 0.f ? 1.f / sqrtf((float)pl->D) : scale;
    prm.scale_log2 = prm.scale * 1.4426950408889634f;
    prm.status = basp_status_device_ptr();
    if (!prm.status) return BASP_ERR_CUDA;

    BASP_CUDA_TRY(cudaMemsetAsync(acc0, 0, (size_t)pl->N * acc_b, st));
    const long long row_threads = (long long)pl->Bl * pl->S * pl->Hq_l * (pl->D / 8);
    for (int r = 0; r < pl->N; ++r) {
        bwd_delta_kernel<<<(unsigned)((row_threads + 255) / 256), 256, 0, st>>>(
            (const __nv_bfloat16 *)o[r], (const __nv_bfloat16 *)dout[r], const_cast<float *>(prm.delta[r]), pl->Bl,
            pl->S, pl->Hq_l, pl->D);
    }
    BASP_CUDA_TRY(cudaGetLastError());

    int dev = 0, sms = 0;
    BASP_CUDA_TRY(cudaGetDevice(&dev));
    BASP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long items = (long long)(pl->S / kT) * pl->N * pl->Bl * pl->Hkv_l;
    const int grid = (int)(items < sms ? items : sms);
    const int smem = 7 * kT * 128 * 2 + 4 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
    BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attn_bwd_kernel<R><<<grid, kBwdThreads, smem, st>>>(prm);
    BASP_CUDA_TRY(cudaGetLastError());

    const long long n8 = (long long)(acc_b / sizeof(float) / 8);
    for (int r = 0; r < pl->N; ++r)
        bwd_dq_convert_kernel<<<(unsigned)((n8 + 255) / 256), 256, 0, st>>>(prm.dq_acc[r], (__nv_bfloat16 *)dq[r], n8);
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(1 + 2 * pl->N);
    return BASP_OK;
}

}  // namespace

extern "C" size_t basp_attn_bwd_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    return (size_t)p->N * (bwd_acc_bytes(p) + bwd_delta_bytes(p));
}

extern "C" int basp_attn_bwd(const basp_plan *pl, const void *const *q_head, const void *const *k_head,
                             const void *const *v_head, const void *const *o_head, const void *const *do_head,
                             const float *const *lse_shards, void *const *dq_head, void *const *dk_head,
                             void *const *dv_head, void *workspace, size_t workspace_bytes, float softmax_scale,
                             void *stream) {
    if (!pl || !q_head || !k_head || !v_head || !o_head || !do_head || !lse_shards || !dq_head || !dk_head ||
        !dv_head || !workspace)
        return BASP_ERR_NULL;
    if (pl->D != 128 || pl->S % kT != 0) return BASP_ERR_UNSUPPORTED;
    if (!aligned16(workspace)) return BASP_ERR_ALIGN;
    if (workspace_bytes < basp_attn_bwd_workspace_bytes(pl)) return BASP_ERR_WORKSPACE;
    for (int r = 0; r < pl->N; ++r) {
        const void *ptrs[9] = {q_head[r], k_head[r], v_head[r], o_head[r], do_head[r], lse_shards[r],
                               dq_head[r], dk_head[r], dv_head[r]};
        for (int i = 0; i < 9; ++i) {
            if (!ptrs[i]) return BASP_ERR_NULL;
            if (!aligned16(ptrs[i])) return BASP_ERR_ALIGN;
        }
        for (int r2 = 0; r2 < pl->N; ++r2) {
            const void *ins[5] = {q_head[r2], k_head[r2], v_head[r2], o_head[r2], do_head[r2]};
            for (int i = 0; i < 5; ++i)
                if (dq_head[r] == ins[i] || dk_head[r] == ins[i] || dv_head[r] == ins[i]) return BASP_ERR_ALIAS;
        }
    }
    if (pl->N <= 8)
        return bwd_launch<8>(pl, q_head, k_head, v_head, o_head, do_head, lse_shards, dq_head, dk_head, dv_head,
                             (char *)workspace, softmax_scale, (cudaStream_t)stream);
    return bwd_launch<BASP_MAX_RANKS>(pl, q_head, k_head, v_head, o_head, do_head, lse_shards, dq_head, dk_head,
                                      dv_head, (char *)workspace, softmax_scale, (cudaStream_t)stream);
}
