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
//   (5) dQ_m = dS K         SS   -> TMEM [128,256)  (A = the dS^T buffer read MN-major)
//   (4) dK  += dS^T Q       SS   -> TMEM [256,384)
//   drain warps: dQ_m staged through the (now free) Q / dO stage and added to the fp32 accumulator in
//   global memory by TMA reduce-add (order of the additions not fixed), while the compute warps and
//   the tensor core are already on the next step.
// Warps: 16 compute (a quarter of the score columns each), 4 drain, TMA producer, MMA issuer.
// Helper kernels: Delta = rowsum(dO * O); fp32 dQ accumulator -> bf16.
#include <cuda.h>
#include <math.h>

#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"
#include "tmap.cuh"

int *basp_status_device_ptr();

namespace {

using namespace ptx;

constexpr int kT = 128;
constexpr int kBwdComputeWarps = 16;
[[maybe_unused]] constexpr int kBwdDrainWarp0 = kBwdComputeWarps;          // 4 warps that take dQ out of TMEM and reduce-add it
constexpr int kBwdTmaWarp = kBwdComputeWarps + 4;
constexpr int kBwdMmaWarp = kBwdComputeWarps + 5;
constexpr int kBwdThreads = (kBwdComputeWarps + 8) * 32;   // + drain warpgroup + (TMA, MMA, two idle warps)

template <int R>
struct BwdParams {
    CUtensorMap q[R], k[R], v[R], dout[R];
    CUtensorMap dq_acc[R];      // fp32 accumulator, box 32 floats x 1 head x 32 rows (reduce-add target)
    const float *lse[R];
    const float *delta[R];
    __nv_bfloat16 *dk[R], *dv[R];
    __nv_bfloat16 *dq[R];       // the two-pass kernels write dQ directly
    int n_ranks, Bl, S, Hq_l, Hkv_l, q_per_kv, causal;
    int Dg;                     // head dimension in memory (a multiple of 16 up to 128): the tile loads zero-fill the columns
                                // past it, so every product is right as it stands; only the stores have to skip them
    float scale, scale_log2;
    int *status;
};

struct BwdItem {
    int r, bl, hkv, n, m0, n_qt;
};

template <int R>
__device__ __forceinline__ bool bwd_get_item(const BwdParams<R> &p, int round, BwdItem &it) {
    const int n_kt = (p.S + kT - 1) / kT;      // the last tile may be ragged
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
    uint64_t kv_full, kv_empty, qdo_full[3], qdo_empty[2], qdo_mma_done[3];      // (the 64-wide kernel has three stages)
    uint64_t s_full, stats_full[3], pds_ready, dq_full, dq_read, dkdv_full, dkdv_read;
    uint64_t s_full_b[2], dp_full, p_ready;   // the pipelined 64-wide kernel: one S^T barrier per buffer, dP^T and P^T on their own
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

#ifdef BASP_PHASE_TIMING
__device__ long long g_bwd_phase[32];
#define BPH_T(var) const long long var = clock64()
#define BPH_ADD(slot, a, b) do { bacc[(slot) & 7] += (b) - (a); } while (0)
#else
#define BPH_T(var)
#define BPH_ADD(slot, a, b)
#endif

#define BWD_WAIT(bar, parity, role, detail)                                    \
    do {                                                                        \
        if (!mbar_wait((bar), (parity), &bars->abort_flag)) {                  \
            bars->abort_flag = 1;                                               \
            bwd_report(p.status, 3, (role), (detail));                          \
            goto bwd_done;                                                      \
        }                                                                       \
    } while (0)

// D = 128 or 64: the kernel's width (columns of the Q, K, V, dO tiles and of the dQ, dK, dV accumulators).  A tile is D/64
// slabs of [128 rows][64 columns] (one 128-byte swizzled line per row and slab).
template <int D, int R>
__global__ void __launch_bounds__(kBwdThreads, 1) attn_bwd_kernel(const __grid_constant__ BwdParams<R> p) {
    static_assert(D == 64 || D == 128, "kernel widths");
    constexpr int kSlabs = D / 64;
    constexpr int kTileBytes = kT * D * 2;             // 32 KiB (16 KiB at D = 64)
    constexpr int kDqChunks = D / 32;                  // 32-column fp32 chunks of a dQ tile
    // dynamic shared memory only, so that the tile area starts at the (1024-byte aligned) window base
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *sK = smem, *sV = smem + kTileBytes;
    uint8_t *sQ = smem + 2 * kTileBytes;               // 2 stages
    uint8_t *sdO = smem + 4 * kTileBytes;              // 2 stages
    uint8_t *sdS = smem + 6 * kTileBytes;              // dS^T [key rows][query cols], two 64-column slabs (32 KiB)
    float *s_lse = reinterpret_cast<float *>(sdS + 2 * 16384);         // [2][128], already times log2(e)
    float *s_delta = s_lse + 2 * kT;                                   // [2][128]
    BwdBars *bars = reinterpret_cast<BwdBars *>(s_delta + 2 * kT);

    const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
#ifdef BASP_PHASE_TIMING
    long long bacc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#endif

    if (tid == 0) {
        mbar_init(&bars->kv_full, 1); mbar_init(&bars->kv_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->qdo_full[s], 1);
            mbar_init(&bars->qdo_empty[s], 4);                  // every drain warp's reduce-add has read the stage
            mbar_init(&bars->qdo_mma_done[s], 1);
        }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->stats_full[0], 1);
        mbar_init(&bars->stats_full[1], 1);
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
        // (no register change: 16 warps x 80 registers; the pool that setmaxnreg redistributes is what the CTA got at
        //  launch, 768 x 80, so 4 x 32 x 104 for the drain warps has to come out of the last warpgroup's 4 x 32 x 24)
        const int g = warp >> 2;                        // which 32-column quarter of the score tile
        const int row = tid & 127;                      // TMEM lane: key row (scores) / query row (dQ)
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t it_g = 0, item_n = 0;
        BwdItem item;
        for (int round = 0; bwd_get_item(p, round, item); ++round, ++item_n) {
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                const int h = item.hkv * p.q_per_kv + hq;
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const int buf = it_g & 1;
                    BPH_T(t0);
                    BWD_WAIT(&bars->stats_full[buf], (it_g >> 1) & 1, 10, m);   // LSE and Delta of the query tile (producer warp)
                    BPH_T(t0a);
                    BPH_ADD(7, t0, t0a);
                    BWD_WAIT(&bars->s_full, it_g & 1, 11, m);
                    tc_fence_after();
                    BPH_T(t1);
                    uint32_t st[32], dp[32];
                    tmem_ld_x32(tmem + kColST + 32 * g + lane_addr, st);
                    tmem_ld_x32(tmem + kColDP + 32 * g + lane_addr, dp);
                    tmem_wait_ld();
                    BPH_T(t2);
                    const bool diag = p.causal && m == item.n;
                    // A ragged last tile (S is not a multiple of 128) holds rows of the next sequence of the shard, or TMA
                    // zero fill, past the end: those keys and queries take no part (P = 0 makes dS = 0 and with it every
                    // contribution to dV, dQ, dK).
                    // Folded into one column window per thread: this thread's columns c (query 32g + c) count iff
                    // c_lo <= c < c_hi.  Only edge steps (the diagonal, a ragged last tile) carry the test at all: the loop
                    // is instantiated twice so that the common step has no masking code.
                    const bool edge = diag || (m + 1) * kT > p.S || (item.n + 1) * kT > p.S;
                    int c_lo = 0, c_hi = 32;
                    if (edge) {
                        if (diag) c_lo = row - 32 * g;                              // queries earlier than key `row`
                        if (item.n * kT + row >= p.S) c_lo = 32;                    // this thread's key row does not exist
                        if (p.S - m * kT - 32 * g < c_hi) c_hi = p.S - m * kT - 32 * g;   // queries past the end
                    }
                    const float *lse_b = s_lse + buf * kT + 32 * g;
                    const float *del_b = s_delta + buf * kT + 32 * g;
                    auto p_and_ds = [&](auto edge_tag) {
                        constexpr bool kEdge = decltype(edge_tag)::value;
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 l4 = *reinterpret_cast<const float4 *>(lse_b + c);
                            const float4 d4 = *reinterpret_cast<const float4 *>(del_b + c);
                            const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dl[4] = {d4.x, d4.y, d4.z, d4.w};
                            float pv[4], dsv[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                pv[e] = exp2_approx(fmaf(__uint_as_float(st[c + e]), p.scale_log2, -lv[e]));
                                if (kEdge && (c + e < c_lo || c + e >= c_hi)) pv[e] = 0.f;
                                dsv[e] = pv[e] * fmaf(__uint_as_float(dp[c + e]), p.scale, dl[e]);   // dl = -Delta scale
                            }
                            st[c >> 1] = pack_bf16x2(pv[0], pv[1]);
                            st[(c >> 1) + 1] = pack_bf16x2(pv[2], pv[3]);
                            dp[c >> 1] = pack_bf16x2(dsv[0], dsv[1]);
                            dp[(c >> 1) + 1] = pack_bf16x2(dsv[2], dsv[3]);
                        }
                    };
                    if (edge) p_and_ds(std::true_type{});
                    else p_and_ds(std::false_type{});
                    BPH_T(t3);
                    // P^T (bf16) over this quarter's own score columns: TMEM columns 32g .. 32g+15
                    tmem_st_x16(tmem + kColST + 32 * g + lane_addr, *reinterpret_cast<const uint32_t(*)[16]>(&st[0]));
                    // dS^T row `row`, query columns 32g..32g+31 = half a 128-byte line of slab g/2 (128-byte swizzle)
                    {
                        uint8_t *line = sdS + (g >> 1) * 16384 + row * 128;
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch)
                            *reinterpret_cast<uint4 *>(line + (((4 * (g & 1) + ch) ^ (row & 7)) << 4)) =
                                make_uint4(dp[4 * ch], dp[4 * ch + 1], dp[4 * ch + 2], dp[4 * ch + 3]);
                    }
                    fence_proxy_async_smem();
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->pds_ready);
                    BPH_T(t4);
                    BPH_T(t5);
                    BPH_T(t6);
                    BPH_ADD(0, t0a, t1); BPH_ADD(1, t1, t2); BPH_ADD(2, t2, t3); BPH_ADD(3, t3, t4);
                    BPH_ADD(4, t4, t5); BPH_ADD(5, t5, t6); BPH_ADD(6, t0, t0 + 1);
                }
            }
            // ---- item done: dK_n (half 0) / dV_n (half 1) to global as bf16
            BWD_WAIT(&bars->dkdv_full, item_n & 1, 13, item.n);
            tc_fence_after();
            {
                // quarters 0,1 write the two halves (D/2 columns each) of dK, quarters 2,3 those of dV
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
        // dQ_m (lane = query row, D fp32 columns) leaves TMEM through the Q / dO stage of its step, which is free
        // shared memory of exactly its size once the products that read it are done: chunk c ([128 rows][32 floats],
        // 128-byte swizzle) goes to the dO half (the upper half of the chunks; product (3) is complete when dQ is) or
        // the Q half (the lower half; after product (4)).  Each warp adds its 32 rows of a chunk with one TMA reduce-add.
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
                    const uint32_t stage = it_g & 1, ph = (it_g >> 1) & 1;
                    BPH_T(v0);
                    BWD_WAIT(&bars->dq_full, it_g & 1, 12, m);
                    tc_fence_after();
                    BPH_T(v1);
                    constexpr int kHalfCh = kDqChunks / 2;            // chunks per half: 2 (1 at D = 64)
                    uint32_t lo[32 * kHalfCh];
                    auto stage_chunk = [&](int c, const uint32_t *v) {
                        uint8_t *line = (c < kHalfCh ? sQ : sdO) + stage * kTileBytes + (c % kHalfCh) * 16384 + row * 128;
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch)
                            *reinterpret_cast<uint4 *>(line + ((ch ^ (row & 7)) << 4)) =
                                make_uint4(v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
                    };
                    {
                        uint32_t hi[32];
#pragma unroll
                        for (int c = kHalfCh; c < kDqChunks; ++c) {
                            tmem_ld_x32(tmem + kColDP + 32 * c + lane_addr, hi);
                            tmem_wait_ld();
                            stage_chunk(c, hi);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < kHalfCh; ++c)
                        tmem_ld_x32(tmem + kColDP + 32 * c + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(&lo[32 * c]));
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->dq_read);          // TMEM is free for the next dP^T
                    BPH_T(v2);
                    BWD_WAIT(&bars->qdo_mma_done[stage], ph, 14, m);     // product (4) has read the Q half
                    BPH_T(v3);
#pragma unroll
                    for (int c = 0; c < kHalfCh; ++c) stage_chunk(c, &lo[32 * c]);
                    fence_proxy_async_smem();
                    __syncwarp();
#ifndef BWD_NO_RED
                    if (lane == 0) {
                        const int row0 = item.bl * p.S + m * kT + wq * 32;
#pragma unroll
                        for (int c = 0; c < kDqChunks; ++c)
                            if (32 * c < p.Dg)          // a chunk wholly past the head dimension is padding
                            tma_reduce_add_3d(&p.dq_acc[item.r],
                                              (c < kHalfCh ? sQ : sdO) + stage * kTileBytes + (c % kHalfCh) * 16384 + wq * 4096,
                                              32 * c, h, row0);
                        tma_store_commit();
                        tma_store_wait_read<0>();          // these warps have nothing else to do until the next dQ tile
                    }
#endif
                    if (lane == 0) mbar_arrive(&bars->qdo_empty[stage]);
                    BPH_T(v4);
                    BPH_ADD(16, v0, v1); BPH_ADD(17, v1, v2); BPH_ADD(18, v2, v3); BPH_ADD(19, v3, v4); BPH_ADD(20, v0, v0 + 1);
                }
            }
        }
    } else {
      // every warp of the last warpgroup gives registers back at this one place (TMA, MMA and two idle warps)
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
                for (int s = 0; s < kSlabs; ++s) {
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
                        for (int s = 0; s < kSlabs; ++s) {
                            tma_load_3d(sQ + stage * kTileBytes + s * 16384, &p.q[item.r], &bars->qdo_full[stage], s * 64, h, row0);
                            tma_load_3d(sdO + stage * kTileBytes + s * 16384, &p.dout[item.r], &bars->qdo_full[stage], s * 64, h, row0);
                        }
                    }
                    {   // row statistics of the query tile: LSE (to log2 units) and Delta, four rows per lane.  The buffer
                        // has the stage's parity: its last readers (step it-2) finished before the stage was released.
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
                        d4.x *= -p.scale; d4.y *= -p.scale; d4.z *= -p.scale; d4.w *= -p.scale;   // staged as -Delta scale
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
            BWD_WAIT(&bars->kv_full, item_n & 1, 30, item.n);
            bool first = true;
            for (int hq = 0; hq < p.q_per_kv; ++hq) {
                for (int m = item.m0; m < item.n_qt; ++m, ++it_g) {
                    const uint32_t stage = it_g & 1, ph = (it_g >> 1) & 1;
                    const uint32_t q16 = aQ + stage * (kTileBytes >> 4), do16 = adO + stage * (kTileBytes >> 4);
                    BPH_T(u0);
                    BWD_WAIT(&bars->qdo_full[stage], ph, 31, m);
                    tc_fence_after();
                    BPH_T(u1);
                    if (lane == 0) {        // (1) S^T = K Q^T
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                            mma_ss(tmem + kColST, desc_k | (uint64_t)(aK + off), desc_k | (uint64_t)(q16 + off), idesc_kk, kk > 0);
                        }
                    }
                    BPH_T(u2);
                    BWD_WAIT(&bars->dq_read, (it_g & 1) ^ 1, 32, m);          // previous dQ tile has left TMEM
                    tc_fence_after();
                    BPH_T(u3);
                    if (lane == 0) {        // (2) dP^T = V dO^T
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk / 4) * 16384 + (kk % 4) * 32) >> 4;
                            mma_ss(tmem + kColDP, desc_k | (uint64_t)(aV + off), desc_k | (uint64_t)(do16 + off), idesc_kk, kk > 0);
                        }
                        tc_commit(&bars->s_full);
                    }
                    BPH_T(u4);
                    BWD_WAIT(&bars->pds_ready, it_g & 1, 33, m);
                    BPH_T(u5);
                    if (first) BWD_WAIT(&bars->dkdv_read, (item_n & 1) ^ 1, 34, item.n);
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t acc0 = first ? 0u : 1u;
                        // (3) dV += P^T dO : A = P^T in TMEM (query index along K: 8 columns per 16 queries,
                        //     each quarter of 32 queries starts at its own column 32g), B = dO read MN-major
#pragma unroll
                        for (int kk = 0; kk < kT / 16; ++kk)
                            mma_ts(tmem + kColDV, tmem + kColST + (kk / 2) * 32 + (kk % 2) * 8,
                                   desc_mn | (uint64_t)(do16 + kk * 128), idesc_kn, kk > 0 ? 1u : acc0);
                        // (5) dQ_m = dS K : A = the dS^T buffer read MN-major (query rows), B = K MN-major.  When it is
                        //     complete so is (3): the dO half of the stage is free for the drain warps.
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
                        tc_commit(&bars->qdo_mma_done[stage]);
                    }
                    first = false;
                    BPH_T(u6);
                    BPH_ADD(8, u0, u1); BPH_ADD(9, u1, u2); BPH_ADD(10, u2, u3); BPH_ADD(11, u3, u4);
                    BPH_ADD(12, u4, u5); BPH_ADD(13, u5, u6); BPH_ADD(14, u0, u0 + 1);
                }
            }
            if (lane == 0) {
                tc_commit(&bars->dkdv_full);
                tc_commit(&bars->kv_empty);
            }
        }
      }
    }

bwd_done:
#ifdef BASP_PHASE_TIMING
    if (blockIdx.x == 5 && (threadIdx.x & 31) == 0 && (warp == 0 || warp == kBwdMmaWarp || warp == kBwdDrainWarp0)) {
        const int base_ = warp == 0 ? 0 : (warp == kBwdMmaWarp ? 8 : 16);
        for (int i_ = 0; i_ < 8; ++i_) g_bwd_phase[base_ + i_] += bacc[i_];
    }
#endif
    tc_fence_before();
    __syncthreads();
    if (bars->abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) { }
        __syncthreads();
    }
    if (warp == kBwdTmaWarp) tmem_dealloc(tmem, 512);
}

#include "attn_bwd_d64.cuh"
#include "attn_bwd_2pass.cuh"

#undef BWD_WAIT

// Delta[bl][h][s] = sum_d O[bl][s][h][d] * dO[bl][s][h][d]; one 16-lane group per (s, h) row of D <= 128.
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __nv_bfloat16 *__restrict__ o,
                                                        const __nv_bfloat16 *__restrict__ dout,
                                                        float *__restrict__ delta, int Bl, int S, int H, int D) {
    constexpr int lanes = 16;                           // threads per row (16 bytes each; D / 8 of them have data)
    const long long rows = (long long)Bl * S * H;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long rowi = gid / lanes;
    const int part = (int)(gid % lanes);
    float acc = 0.f;
    if (rowi < rows && part * 8 < D) {
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
               void *const *dk, void *const *dv, char *ws, float scale, bool two_pass, cudaStream_t st) {
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
        float *acc_r = reinterpret_cast<float *>(reinterpret_cast<char *>(acc0) + (size_t)r * acc_b);
        rc = tmap::encode_f32_rows_heads_d(&prm.dq_acc[r], acc_r, rows, pl->Hq_l, pl->D, 32);
        if (rc != BASP_OK) return rc;
        prm.delta[r] = reinterpret_cast<float *>(reinterpret_cast<char *>(del0) + (size_t)r * del_b);
        prm.dk[r] = (__nv_bfloat16 *)dk[r];
        prm.dq[r] = (__nv_bfloat16 *)dq[r];
        prm.dv[r] = (__nv_bfloat16 *)dv[r];
    }
    prm.n_ranks = pl->N; prm.Bl = pl->Bl; prm.S = pl->S; prm.Hq_l = pl->Hq_l; prm.Hkv_l = pl->Hkv_l;
    prm.Dg = pl->D;
    prm.q_per_kv = pl->Hq_l / pl->Hkv_l; prm.causal = pl->causal;   // per rank (a replicated KV head serves all of a rank's query heads)
    prm.scale = scale == 0.f ? 1.f / sqrtf((float)pl->D) : scale;
    prm.scale_log2 = prm.scale * 1.4426950408889634f;
    prm.status = basp_status_device_ptr();
    if (!prm.status) return BASP_ERR_CUDA;

    if (!two_pass) BASP_CUDA_TRY(cudaMemsetAsync(acc0, 0, (size_t)pl->N * acc_b, st));
    const long long row_threads = (long long)pl->Bl * pl->S * pl->Hq_l * 16;
    for (int r = 0; r < pl->N; ++r) {
        bwd_delta_kernel<<<(unsigned)((row_threads + 255) / 256), 256, 0, st>>>(
            (const __nv_bfloat16 *)o[r], (const __nv_bfloat16 *)dout[r], const_cast<float *>(prm.delta[r]), pl->Bl,
            pl->S, pl->Hq_l, pl->D);
    }
    BASP_CUDA_TRY(cudaGetLastError());

    int dev = 0, sms = 0;
    BASP_CUDA_TRY(cudaGetDevice(&dev));
    BASP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long n_tiles = (pl->S + kT - 1) / kT;
    const long long items = n_tiles * pl->N * pl->Bl * pl->Hkv_l;
    const int grid = (int)(items < sms ? items : sms);
    if (two_pass) {
        const int smem = 6 * kT * 128 * 2 + 2 * 16384 + 4 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_pass_kernel<0, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_pass_kernel<1, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attn_bwd_pass_kernel<0, R><<<grid, kBwdThreads, smem, st>>>(prm);
        const long long items_q = n_tiles * pl->N * pl->Bl * pl->Hq_l;
        attn_bwd_pass_kernel<1, R><<<(int)(items_q < sms ? items_q : sms), kBwdThreads, smem, st>>>(prm);
        BASP_CUDA_TRY(cudaGetLastError());
        basp_count_launch(2 + pl->N);
        return BASP_OK;
    }
    if (pl->D > 64) {        // 80 .. 128: the 128-wide kernel
        const int smem = 6 * kT * 128 * 2 + 2 * 16384 + 4 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_kernel<128, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attn_bwd_kernel<128, R><<<grid, kBwdThreads, smem, st>>>(prm);
    } else {                 // 16 .. 64: the pipelined 64-wide kernel (attn_bwd_d64.cuh)
#ifdef BASP_BWD64_PLAIN
        const int smem = 6 * kT * 64 * 2 + 2 * 16384 + 4 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_kernel<64, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attn_bwd_kernel<64, R><<<grid, kBwdThreads, smem, st>>>(prm);
#else
        const int smem = (2 + 2 * 3) * kT * 64 * 2 + 4 * 16384 + 2 * 3 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_d64_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attn_bwd_d64_kernel<R><<<grid, kBwdThreads, smem, st>>>(prm);
#endif
    }
    BASP_CUDA_TRY(cudaGetLastError());

    const long long n8 = (long long)(acc_b / sizeof(float) / 8);
    for (int r = 0; r < pl->N; ++r)
        bwd_dq_convert_kernel<<<(unsigned)((n8 + 255) / 256), 256, 0, st>>>(
            reinterpret_cast<const float *>(reinterpret_cast<const char *>(acc0) + (size_t)r * acc_b), (__nv_bfloat16 *)dq[r], n8);
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(1 + 2 * pl->N);
    return BASP_OK;
}

}  // namespace

#ifdef BASP_PHASE_TIMING
extern "C" int basp_debug_bwd_phases(long long *out, int reset) {
    if (out && cudaMemcpyFromSymbol(out, g_bwd_phase, sizeof(long long) * 32) != cudaSuccess) return -1;
    if (reset) { long long z[32] = {0}; if (cudaMemcpyToSymbol(g_bwd_phase, z, sizeof(z)) != cudaSuccess) return -1; }
    return 0;
}
#endif

extern "C" size_t basp_attn_bwd_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    return (size_t)p->N * (bwd_acc_bytes(p) + bwd_delta_bytes(p));
}

namespace {
int bwd_entry(const basp_plan *pl, const void *const *q_head, const void *const *k_head,
              const void *const *v_head, const void *const *o_head, const void *const *do_head,
              const float *const *lse_shards, void *const *dq_head, void *const *dk_head,
              void *const *dv_head, void *workspace, size_t workspace_bytes, float softmax_scale, bool two_pass,
              void *stream) {
    if (!pl || !q_head || !k_head || !v_head || !o_head || !do_head || !lse_shards || !dq_head || !dk_head ||
        !dv_head || !workspace)
        return BASP_ERR_NULL;
    if (pl->D < 16 || pl->D > 128 || pl->D % 16 != 0) return BASP_ERR_UNSUPPORTED;
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
                             (char *)workspace, softmax_scale, two_pass, (cudaStream_t)stream);
    return bwd_launch<BASP_MAX_RANKS>(pl, q_head, k_head, v_head, o_head, do_head, lse_shards, dq_head, dk_head,
                                      dv_head, (char *)workspace, softmax_scale, two_pass, (cudaStream_t)stream);
}
}  // namespace

extern "C" int basp_attn_bwd(const basp_plan *pl, const void *const *q_head, const void *const *k_head,
                             const void *const *v_head, const void *const *o_head, const void *const *do_head,
                             const float *const *lse_shards, void *const *dq_head, void *const *dk_head,
                             void *const *dv_head, void *workspace, size_t workspace_bytes, float softmax_scale,
                             void *stream) {
    return bwd_entry(pl, q_head, k_head, v_head, o_head, do_head, lse_shards, dq_head, dk_head, dv_head, workspace,
                     workspace_bytes, softmax_scale, false, stream);
}

// The same gradients from the two-pass kernels (attn_bwd_2pass.cuh): no reduction through global memory, so the
// result does not depend on the order in which CTAs finish (bit-identical from run to run), at 7 products per tile
// pair instead of 5.
extern "C" int basp_attn_bwd_deterministic(const basp_plan *pl, const void *const *q_head, const void *const *k_head,
                                           const void *const *v_head, const void *const *o_head,
                                           const void *const *do_head, const float *const *lse_shards,
                                           void *const *dq_head, void *const *dk_head, void *const *dv_head,
                                           void *workspace, size_t workspace_bytes, float softmax_scale, void *stream) {
    return bwd_entry(pl, q_head, k_head, v_head, o_head, do_head, lse_shards, dq_head, dk_head, dv_head, workspace,
                     workspace_bytes, softmax_scale, true, stream);
}
