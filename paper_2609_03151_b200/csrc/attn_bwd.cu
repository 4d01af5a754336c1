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
//   (1) S^T  = K Q^T        SS   -> TMEM
//   (2) dP^T = V dO^T       SS   -> TMEM
//   compute warps: P^T = exp2(..) -> bf16 to TMEM;  dS^T = scale P^T (dP^T - Delta) -> bf16 to shared memory
//   (3) dV  += P^T dO       TS
//   (5) dQ_m = dS K         SS   (in the place of dP^T), added to an fp32 accumulator in global memory
//   (4) dK  += dS^T Q       SS
// Warps: 16 compute (a quarter of the score columns each), 4 dQ drain, TMA producer, MMA issuer.
// Three kernels share this file's parameter block, work-item order and barriers: attn_bwd_d128.cuh (head dimensions
// 80 .. 128), attn_bwd_d64.cuh (16 .. 64) and the two-pass form attn_bwd_2pass.cuh; each header says how it orders
// the steps.  Helper kernels here: Delta = rowsum(dO * O); fp32 dQ accumulator -> bf16.
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
    float *dq_accp[R];          // the same accumulator as a plain pointer ([Bl*S][Hq_l][Dg] floats)
    const float *lse[R];
    const float *delta[R];
    __nv_bfloat16 *dk[R], *dv[R];
    __nv_bfloat16 *dq[R];       // the two-pass kernels write dQ directly
    int n_ranks, Bl, S, Hq_l, Hkv_l, q_per_kv, causal;
    int gang;                   // 1: the gang schedule of bwd_get_item_gang (cooperative launch)
    unsigned *gang_sync;        // one arrival counter per gang, zeroed before the launch
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

// The gang schedule for long sequences.  Every key tile's sweep re-reads Q and dO and adds into dQ of the same query
// tiles; whether those bytes come out of the L2 or out of DRAM depends on WHEN the sweeps of one (rank, sequence, KV
// head) pass a query tile.  With the plain deal above the CTAs drift apart after their first items and most of that
// traffic goes to DRAM (measured: 19 KB per step at 16K tokens, 45 KB at 32K, growing with the length), which bounds
// the kernel at 128K tokens.  Here the CTAs with blockIdx % streams == s form the gang of stream s: in round r member j
// takes key tile r G + j (alternate rounds mirrored for balance), and the members start each query-head sweep together
// (bwd_gang_barrier in the producer warp).  Member j starts at its own diagonal tile, j tiles further on than member 0,
// so a query tile is visited by the members one step after another: re-use distance one step of the whole GPU's
// traffic (about 28 MB), well inside the L2.  Cost: a member waits at most G - 1 steps per sweep for the longest one.
template <int R>
__device__ __forceinline__ bool bwd_get_item_gang(const BwdParams<R> &p, int round, BwdItem &it) {
    const int n_kt = (p.S + kT - 1) / kT;
    const int streams = p.n_ranks * p.Bl * p.Hkv_l;
    const int s = (int)blockIdx.x % streams, j = (int)blockIdx.x / streams;
    const int G = ((int)gridDim.x - s + streams - 1) / streams;
    it.n = round * G + ((round & 1) ? G - 1 - j : j);
    if (it.n >= n_kt) return false;       // a mirrored last round can leave a gap: members past the end are simply done
    int rem = s;
    it.hkv = rem % p.Hkv_l;
    rem /= p.Hkv_l;
    it.bl = rem % p.Bl;
    it.r = rem / p.Bl;
    it.n_qt = n_kt;
    it.m0 = it.n;                          // causal only
    return true;
}

// Start of sweep `hq` of round `round`: arrive on the gang's counter and wait (bounded) until every member that has an
// item in this round has arrived.  One lane of the producer warp; the loads it gates hold everything else back.
template <int R>
__device__ __forceinline__ bool bwd_gang_barrier(const BwdParams<R> &p, int round, int hq) {
    const int n_kt = (p.S + kT - 1) / kT;
    const int streams = p.n_ranks * p.Bl * p.Hkv_l;
    const int s = (int)blockIdx.x % streams;
    const int G = ((int)gridDim.x - s + streams - 1) / streams;
    const int active = min(G, n_kt - round * G);
    const unsigned target = (unsigned)(round * G * p.q_per_kv + active * (hq + 1));
    unsigned *ctr = p.gang_sync + s;
    atomicAdd(ctr, 1u);
    const uint64_t t0 = globaltimer_ns();
    while (*reinterpret_cast<volatile unsigned *>(ctr) < target) {
        __nanosleep(200);
        if (globaltimer_ns() - t0 > kWaitLimitNs) return false;
    }
    return true;
}

struct BwdBars {
    uint64_t kv_full, kv_empty, qdo_full[3], qdo_empty[2], qdo_mma_done[3];      // (Q / dO stages: the 64-wide kernel has three)
    uint64_t s_full, stats_full[3], pds_ready, dq_full, dq_read, dkdv_full, dkdv_read;
    uint64_t s_full_b[2], dp_full, p_ready;   // the pipelined kernels: one S^T barrier per buffer, dP^T and P^T on their own
    uint64_t do_full[2], do_free[2];          // the pipelined 128-wide kernel: dO stages are released on their own
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

#include "attn_bwd_d64.cuh"
#include "attn_bwd_d128.cuh"
#include "attn_bwd_2pass.cuh"

#undef BWD_WAIT

// Delta[bl][h][s] = sum_d O[bl][s][h][d] * dO[bl][s][h][d]; one 16-lane group per (s, h) row of D <= 128.
template <int R>
struct BwdHelperPtrs {
    const __nv_bfloat16 *o[R], *dout[R];
    float *delta[R];
    const float *acc[R];
    __nv_bfloat16 *dq[R];
};

// (one launch for every rank: blockIdx.y = rank)
template <int R>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __grid_constant__ BwdHelperPtrs<R> hp, int Bl, int S, int H,
                                                        int D) {
    const __nv_bfloat16 *__restrict__ o = hp.o[blockIdx.y];
    const __nv_bfloat16 *__restrict__ dout = hp.dout[blockIdx.y];
    float *__restrict__ delta = hp.delta[blockIdx.y];
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
template <int R>
__global__ void __launch_bounds__(256) bwd_dq_convert_kernel(const __grid_constant__ BwdHelperPtrs<R> hp, long long n8) {
    const float *__restrict__ acc = hp.acc[blockIdx.y];
    __nv_bfloat16 *__restrict__ out = hp.dq[blockIdx.y];
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const float4 a = reinterpret_cast<const float4 *>(acc)[2 * i], b = reinterpret_cast<const float4 *>(acc)[2 * i + 1];
    uint4 o;
    o.x = pack_bf16x2(a.x, a.y); o.y = pack_bf16x2(a.z, a.w);
    o.z = pack_bf16x2(b.x, b.y); o.w = pack_bf16x2(b.z, b.w);
    reinterpret_cast<uint4 *>(out)[i] = o;
}

constexpr int kMaxGangs = 256;        // arrival counters at the end of the workspace (gang schedule)
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
        prm.dq_accp[r] = acc_r;
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
    prm.gang = 0;
    prm.gang_sync = reinterpret_cast<unsigned *>(ws + (size_t)pl->N * (acc_b + del_b));

    if (!two_pass) BASP_CUDA_TRY(cudaMemsetAsync(acc0, 0, (size_t)pl->N * acc_b, st));
    const long long row_threads = (long long)pl->Bl * pl->S * pl->Hq_l * 16;
    BwdHelperPtrs<R> hp;
    for (int r = 0; r < pl->N; ++r) {
        hp.o[r] = (const __nv_bfloat16 *)o[r];
        hp.dout[r] = (const __nv_bfloat16 *)dout[r];
        hp.delta[r] = const_cast<float *>(prm.delta[r]);
        hp.acc[r] = prm.dq_accp[r];
        hp.dq[r] = (__nv_bfloat16 *)dq[r];
    }
    bwd_delta_kernel<R><<<dim3((unsigned)((row_threads + 255) / 256), (unsigned)pl->N), 256, 0, st>>>(hp, pl->Bl, pl->S, pl->Hq_l, pl->D);
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
        basp_count_launch(3);
        return BASP_OK;
    }
    if (pl->D > 64) {        // 80 .. 128: the pipelined 128-wide kernel (attn_bwd_d128.cuh)
        const int smem2 = 7 * kT * 128 * 2 + 4 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_d128_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem2));
        // The gang schedule (bwd_get_item_gang) pays when a sweep is long against the gang: a member idles at most
        // G - 1 steps per sweep of n_tiles / 2 steps on average.  Its CTAs wait for one another at the sweep starts, so
        // the launch is cooperative (every CTA resident); where that is refused the plain deal runs.
        const long long streams = (long long)pl->N * pl->Bl * pl->Hkv_l;
        const long long G = streams > 0 ? sms / streams : 0;
        bool gang = pl->causal && G >= 2 && n_tiles >= 16 * G && streams <= kMaxGangs;
        if (gang) {
            int coop = 0;
            BASP_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
            gang = coop != 0;
        }
        if (gang) {
            prm.gang = 1;
            BASP_CUDA_TRY(cudaMemsetAsync(prm.gang_sync, 0, kMaxGangs * sizeof(unsigned), st));
            void *args[1] = {(void *)&prm};
            cudaError_t e = cudaLaunchCooperativeKernel((const void *)attn_bwd_d128_kernel<R>, dim3((unsigned)sms), dim3(kBwdThreads),
                                                        args, (size_t)smem2, st);
            if (e != cudaSuccess) {          // not all CTAs can be resident (another context holds SMs): plain deal
                (void)cudaGetLastError();
                gang = false;
                prm.gang = 0;
            }
        }
        if (!gang) attn_bwd_d128_kernel<R><<<grid, kBwdThreads, smem2, st>>>(prm);
    } else {                 // 16 .. 64: the pipelined 64-wide kernel (attn_bwd_d64.cuh)
        const int smem = (2 + 2 * 3) * kT * 64 * 2 + 4 * 16384 + 2 * 3 * kT * (int)sizeof(float) + (int)sizeof(BwdBars);
        BASP_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_d64_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attn_bwd_d64_kernel<R><<<grid, kBwdThreads, smem, st>>>(prm);
    }
    BASP_CUDA_TRY(cudaGetLastError());

    const long long n8 = (long long)(acc_b / sizeof(float) / 8);
    bwd_dq_convert_kernel<R><<<dim3((unsigned)((n8 + 255) / 256), (unsigned)pl->N), 256, 0, st>>>(hp, n8);
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(3);
    return BASP_OK;
}

}  // namespace

extern "C" size_t basp_attn_bwd_workspace_bytes(const basp_plan *p) {
    if (!p) return 0;
    return (size_t)p->N * (bwd_acc_bytes(p) + bwd_delta_bytes(p)) + kMaxGangs * sizeof(unsigned);
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
    if (!scale_ok(softmax_scale)) return BASP_ERR_INVALID;
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
