// Parameter block and tile addressing shared by the attention kernels.
#pragma once
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "ptx.cuh"

namespace {

using namespace ptx;

constexpr int kTile = 128;     // query rows and key rows per tile

template <int R>
struct AttnParams {
    CUtensorMap q[R], k[R], v[R];
    __nv_bfloat16 *o[R];
    float *lse[R];
    int n_ranks, K, Bl, S, T, Hq_l, Hkv_l, q_per_kv;   // q_per_kv: query heads per KV head on a rank
    int kv_rep;             // local ranks sharing one KV head (sequence-sharded K/V: head index = local rank / kv_rep)
    int o_heads;            // heads in one row of the O destination (Hq_l, or Hq when fused)
    int Dg;                 // head dimension in memory, a multiple of 16 up to the kernel's width (64 or 128): the tile
                            // loads zero-fill the columns past it, the products skip them, the epilogue does not store them
    int qb_band;            // query blocks per scheduling band (divides qb_count)
    int r_begin, r_count;   // ranks covered by this launch
    int qb_begin, qb_count; // 256-row query blocks covered by this launch
    int fused, causal, has_lse;
    float scale_log2;       // softmax scale * log2(e)
    int *status;
    // divisors of the item decoding, prepared on the host (a division by a runtime value is some 25 instructions, and
    // the decoding is inlined into every role: instruction fetch matters in this kernel)
    FastDiv div_per_band, div_per_stream, div_q_per_kv, div_hkv_l, div_bl;
    FastDiv div_T, div_K;   // of the fused tile addressing (owner rank of a sequence position, group of a rank)
};

struct TileCoord {
    int rank, row, head;
};

// Where the 128-token tile starting at sequence position s0 of (rank r, sequence bl, local
// head h) is found.  `heads_l` is the number of local heads of that tensor.
template <int R>
__device__ __forceinline__ TileCoord locate(const AttnParams<R> &p, int r, int bl, int s0, int h, int heads_l,
                                            int rep = 1) {
    TileCoord c;
    if (p.fused) {
        const int g = (int)fdiv((uint32_t)r, p.div_K), l = r - g * p.K;
        const int owner = (int)fdiv((uint32_t)s0, p.div_T);
        c.rank = g * p.K + owner;
        c.row = bl * p.T + (s0 - owner * p.T);
        c.head = rep > 1 ? l / rep : l * heads_l + h;
    } else {
        c.rank = r;
        c.row = bl * p.S + s0;
        c.head = h;
    }
    return c;
}

__device__ __forceinline__ void report(int *status, int code, int role, int detail) {
    if (atomicCAS(status, 0, code) == 0) {
        status[1] = role;
        status[2] = (int)blockIdx.x;
        status[3] = detail;
    }
}

}  // namespace
