/*
 * BASP oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what one BASP / Ulysses sequence-parallel
 * attention layer computes: the group plan (Algorithm 1), the batch-aware sequence
 * partition (Algorithm 2), the two group-local all-to-alls written out as index
 * maps (Section IV-C), and causal scaled-dot-product attention from its definition
 * (Section II-A equation plus a causal mask).  It shares no code, header, table or
 * helper with the CUDA library and is only ever called from tests, the smoke check
 * and the benchmark's CPU-baseline leg.
 *
 * Everything is written as the literal loops of the definition: no blocking, no
 * online softmax, no fusion.  OpenMP only spreads independent rows over cores.
 *
 * Tensors are dense row-major.  Elements of the permutation routines are opaque
 * byte groups of `esize` bytes; attention inputs are bf16 bit patterns (uint16_t)
 * widened exactly to fp64.
 *
 * Notation: N ranks, B micro-batch (sequences), G groups (G = B is BASP, G = 1 is
 * standard Ulysses), K = N/G ranks per group, Bl = B/G sequences per group,
 * S tokens per sequence, T = S/K tokens per rank and sequence, H heads, D head dim.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1: K = N / B, num_groups = B, N mod B must be 0, group i holds the
 * contiguous ranks i*K .. i*K+K-1.  Generalised with an explicit group count G
 * (Section IV-C "P GPUs divided into G groups"): K = N / G and each group owns
 * B / G sequences.  G = B reproduces Algorithm 1, G = 1 is standard Ulysses.
 * Returns 0 when valid, -1 otherwise.  out = {K, G, Bl, T}. */
int oracle_plan(int N, int B, int G, int S, int out[4]) {
    if (N <= 0 || B <= 0 || S <= 0) return -1;
    /* BASP: one group per sequence.  More sequences than ranks: the paper's fallback to plain data parallelism,
     * i.e. every rank a group of its own (K = 1) that holds B/N whole sequences. */
    if (G == 0) G = B > N ? N : B;
    if (G <= 0) return -1;
    if (N % G != 0) return -1;      /* "assert N mod B = 0"                  */
    if (B % G != 0) return -1;
    int K = N / G;
    if (S % K != 0) return -1;      /* chunk = L / K must be whole           */
    out[0] = K;
    out[1] = G;
    out[2] = B / G;
    out[3] = S / K;
    return 0;
}

/* Ranks of group i (Algorithm 1, the "ranks <- [iK .. iK+K-1]" line). */
void oracle_group_ranks(int K, int group, int *ranks_out) {
    for (int j = 0; j < K; ++j) ranks_out[j] = group * K + j;
}

/* Algorithm 2 for one rank: group = floor(r / K), local = r mod K, the
 * sequences [group*Bl, (group+1)*Bl) and the tokens [local*T, (local+1)*T);
 * head blocks are the contiguous split of H heads into K parts (KV heads: see below
 * for a group with more ranks than KV heads).
 * out = {group, local, seq_begin, seq_end, token_begin, token_end,
 *        q_head_begin, q_head_end, kv_head_begin, kv_head_end}. */
void oracle_rank_info(int K, int Bl, int T, int Hq, int Hkv, int r, int out[10]) {
    int g = r / K, l = r % K;
    out[0] = g;
    out[1] = l;
    out[2] = g * Bl;
    out[3] = (g + 1) * Bl;
    out[4] = l * T;
    out[5] = (l + 1) * T;
    out[6] = l * (Hq / K);
    out[7] = (l + 1) * (Hq / K);
    if (Hkv % K == 0) {
        out[8] = l * (Hkv / K);
        out[9] = (l + 1) * (Hkv / K);
    } else {
        /* more ranks in the group than KV heads (the paper does not treat grouped-query
         * attention): query head h reads KV head h / (Hq/Hkv), so the K/Hkv consecutive
         * local ranks whose query heads share a KV head each hold that one head. */
        out[8] = l / (K / Hkv);
        out[9] = out[8] + 1;
    }
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2 applied to every rank: X[B][S][H][D] -> shards[N][Bl][T][H][D],
 * shard of rank r = X[g*Bl : (g+1)*Bl, l*T : (l+1)*T, :, :]. */
void oracle_partition(const unsigned char *X, unsigned char *shards, int N, int K, int Bl,
                      int S, int H, int D, int esize) {
    const int T = S / K;
    for (int r = 0; r < N; ++r) {
        const int g = r / K, l = r % K;
        for (int bl = 0; bl < Bl; ++bl)
            for (int t = 0; t < T; ++t)
                for (int h = 0; h < H; ++h)
                    for (int d = 0; d < D; ++d) {
                        size_t dst = ((((size_t)r * Bl + bl) * T + t) * H + h) * D + d;
                        size_t src = ((((size_t)(g * Bl + bl)) * S + (size_t)l * T + t) * H + h) * D + d;
                        memcpy(shards + dst * esize, X + src * esize, (size_t)esize);
                    }
    }
}

/* Inverse of oracle_partition (collect every rank's shard into X). */
void oracle_gather(const unsigned char *shards, unsigned char *X, int N, int K, int Bl,
                   int S, int H, int D, int esize) {
    const int T = S / K;
    for (int r = 0; r < N; ++r) {
        const int g = r / K, l = r % K;
        for (int bl = 0; bl < Bl; ++bl)
            for (int t = 0; t < T; ++t)
                for (int h = 0; h < H; ++h)
                    for (int d = 0; d < D; ++d) {
                        size_t src = ((((size_t)r * Bl + bl) * T + t) * H + h) * D + d;
                        size_t dst = ((((size_t)(g * Bl + bl)) * S + (size_t)l * T + t) * H + h) * D + d;
                        memcpy(X + dst * esize, shards + src * esize, (size_t)esize);
                    }
    }
}

/* First all-to-all of the Ulysses layer, confined to each group (Section IV-C):
 * every rank sends, to local rank m of its group, the heads [m*H/K, (m+1)*H/K) of
 * its T tokens; the receiver concatenates the K chunks in local-rank order.
 *   seq [N][Bl][T][H][D]  ->  head [N][Bl][S][H/K][D]
 *   head[gK+m][bl][s][h'][d] = seq[gK + s/T][bl][s mod T][m*H/K + h'][d]        */
void oracle_s2h(const unsigned char *seq, unsigned char *head, int N, int K, int Bl, int S,
                int H, int D, int esize) {
    const int T = S / K, Hl = H / K, G = N / K;
    for (int g = 0; g < G; ++g)
        for (int m = 0; m < K; ++m)
            for (int bl = 0; bl < Bl; ++bl)
                for (int s = 0; s < S; ++s)
                    for (int hp = 0; hp < Hl; ++hp)
                        for (int d = 0; d < D; ++d) {
                            int sender = g * K + s / T;
                            size_t dst = ((((size_t)(g * K + m) * Bl + bl) * S + s) * Hl + hp) * D + d;
                            size_t src = ((((size_t)sender * Bl + bl) * T + s % T) * H + (m * Hl + hp)) * D + d;
                            memcpy(head + dst * esize, seq + src * esize, (size_t)esize);
                        }
}

/* Second all-to-all (head-sharded back to the sequence owners):
 *   seq[gK+l][bl][t][m*H/K + h'][d] = head[gK+m][bl][l*T + t][h'][d]             */
void oracle_h2s(const unsigned char *head, unsigned char *seq, int N, int K, int Bl, int S,
                int H, int D, int esize) {
    const int T = S / K, Hl = H / K, G = N / K;
    for (int g = 0; g < G; ++g)
        for (int l = 0; l < K; ++l)
            for (int bl = 0; bl < Bl; ++bl)
                for (int t = 0; t < T; ++t)
                    for (int m = 0; m < K; ++m)
                        for (int hp = 0; hp < Hl; ++hp)
                            for (int d = 0; d < D; ++d) {
                                size_t dst = ((((size_t)(g * K + l) * Bl + bl) * T + t) * H + (m * Hl + hp)) * D + d;
                                size_t src = ((((size_t)(g * K + m) * Bl + bl) * S + (size_t)l * T + t) * Hl + hp) * D + d;
                                memcpy(seq + dst * esize, head + src * esize, (size_t)esize);
                            }
}

/* ------------------------------------------------------------------------- */
static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* One output row of Attention(Q,K,V) = softmax(Q K^T * scale) V (Section II-A),
 * with the causal mask j <= i when `causal`, else all j < S.
 *   Q [Bn][S][Hq][D], K,V [Bn][S][Hkv][D] (bf16 bits), query head h reads KV head
 *   floor(h / (Hq/Hkv)).  out_o gets D doubles, *out_lse = ln sum_j exp(s_ij).
 * `scores` is caller scratch of S doubles. */
static void attn_row(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, int S, int Hq,
                     int Hkv, int D, double scale, int causal, int b, int h, int i,
                     double *scores, double *out_o, double *out_lse) {
    const int kv = h / (Hq / Hkv);
    const int n = causal ? i + 1 : S;
    const uint16_t *q = Q + (((size_t)b * S + i) * Hq + h) * D;
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        const uint16_t *k = Kt + (((size_t)b * S + j) * Hkv + kv) * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
        scores[j] = acc * scale;
        if (scores[j] > m) m = scores[j];
    }
    double denom = 0.0;
    for (int j = 0; j < n; ++j) {
        scores[j] = exp(scores[j] - m);
        denom += scores[j];
    }
    for (int d = 0; d < D; ++d) out_o[d] = 0.0;
    for (int j = 0; j < n; ++j) {
        const uint16_t *v = V + (((size_t)b * S + j) * Hkv + kv) * D;
        const double p = scores[j] / denom;
        for (int d = 0; d < D; ++d) out_o[d] += p * bf16_to_f64(v[d]);
    }
    if (out_lse) *out_lse = m + log(denom);
}

/* Every row: O [Bn][S][Hq][D] (fp64), LSE [Bn][Hq][S] (fp64, may be NULL). */
void oracle_attn_fwd(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, double *O,
                     double *LSE, int Bn, int S, int Hq, int Hkv, int D, double scale, int causal) {
    const long rows = (long)Bn * Hq * S;
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)S);
#pragma omp for schedule(dynamic, 16)
        for (long r = 0; r < rows; ++r) {
            int i = (int)(rows - 1 - r) % S; /* long rows first, order is irrelevant */
            int h = (int)(((rows - 1 - r) / S) % Hq);
            int b = (int)((rows - 1 - r) / ((long)S * Hq));
            double lse;
            attn_row(Q, Kt, V, S, Hq, Hkv, D, scale, causal, b, h, i, scores,
                     O + (((size_t)b * S + i) * Hq + h) * D, &lse);
            if (LSE) LSE[((size_t)b * Hq + h) * S + i] = lse;
        }
        free(scores);
    }
}

/* Selected rows only: rows[3*r] = {b, h, i}; O_rows [nrows][D], lse_rows [nrows]. */
void oracle_attn_fwd_rows(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V,
                          const int *rows, int nrows, double *O_rows, double *lse_rows, int S,
                          int Hq, int Hkv, int D, double scale, int causal) {
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)S);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < nrows; ++r) {
            double lse;
            attn_row(Q, Kt, V, S, Hq, Hkv, D, scale, causal, rows[3 * r], rows[3 * r + 1],
                     rows[3 * r + 2], scores, O_rows + (size_t)r * D, &lse);
            if (lse_rows) lse_rows[r] = lse;
        }
        free(scores);
    }
}

/* ------------------------------------------------------------------------- */
/* Backward of the attention equation (Section II-A) by the chain rule, written out:
 *   P_ij  = exp(scale * q_i.k_j - LSE_i)                    (j visible to i)
 *   D_i   = dO_i . O_i                                       ("delta")
 *   dV_j  = sum_i P_ij dO_i
 *   dP_ij = dO_i . v_j
 *   dS_ij = P_ij (dP_ij - D_i)
 *   dQ_i  = scale * sum_j dS_ij k_j
 *   dK_j  = scale * sum_i dS_ij q_i
 * dK and dV of a KV head are summed over the Hq/Hkv query heads that read it.
 * Two literal passes: rows (LSE, O, D, dQ), then columns (dK, dV), each recomputing P from
 * the first pass's LSE.  dO is bf16 bits like the inputs.  Outputs fp64:
 *   dQ [Bn][S][Hq][D], dK, dV [Bn][S][Hkv][D]. */
static void bwd_row_stats(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO,
                          int S, int Hq, int Hkv, int D, double scale, int causal, int b, int h, int i,
                          double *scores, double *o_row, double *lse, double *delta) {
    attn_row(Q, Kt, V, S, Hq, Hkv, D, scale, causal, b, h, i, scores, o_row, lse);
    const uint16_t *go = dO + (((size_t)b * S + i) * Hq + h) * D;
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += bf16_to_f64(go[d]) * o_row[d];
    *delta = acc;
}

/* dQ of one row, given that row's LSE and delta. */
static void bwd_dq_row(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO, int S,
                       int Hq, int Hkv, int D, double scale, int causal, int b, int h, int i, double lse,
                       double delta, double *dq_row) {
    const int kv = h / (Hq / Hkv);
    const int n = causal ? i + 1 : S;
    const uint16_t *q = Q + (((size_t)b * S + i) * Hq + h) * D;
    const uint16_t *go = dO + (((size_t)b * S + i) * Hq + h) * D;
    for (int d = 0; d < D; ++d) dq_row[d] = 0.0;
    for (int j = 0; j < n; ++j) {
        const uint16_t *k = Kt + (((size_t)b * S + j) * Hkv + kv) * D;
        const uint16_t *v = V + (((size_t)b * S + j) * Hkv + kv) * D;
        double s = 0.0, dp = 0.0;
        for (int d = 0; d < D; ++d) {
            s += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
            dp += bf16_to_f64(go[d]) * bf16_to_f64(v[d]);
        }
        const double p = exp(s * scale - lse);
        const double ds = p * (dp - delta);
        for (int d = 0; d < D; ++d) dq_row[d] += scale * ds * bf16_to_f64(k[d]);
    }
}

/* dK and dV of one key column j of KV head kv: sums over the query heads of the group and the
 * rows that see j.  LSE, DELTA are [Bn][Hq][S]. */
static void bwd_dkdv_col(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO,
                         const double *LSE, const double *DELTA, int S, int Hq, int Hkv, int D, double scale,
                         int causal, int b, int kv, int j, double *dk_row, double *dv_row) {
    const int rep = Hq / Hkv;
    const uint16_t *k = Kt + (((size_t)b * S + j) * Hkv + kv) * D;
    const uint16_t *v = V + (((size_t)b * S + j) * Hkv + kv) * D;
    for (int d = 0; d < D; ++d) dk_row[d] = dv_row[d] = 0.0;
    for (int h = kv * rep; h < (kv + 1) * rep; ++h)
        for (int i = causal ? j : 0; i < S; ++i) {
            const uint16_t *q = Q + (((size_t)b * S + i) * Hq + h) * D;
            const uint16_t *go = dO + (((size_t)b * S + i) * Hq + h) * D;
            double s = 0.0, dp = 0.0;
            for (int d = 0; d < D; ++d) {
                s += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
                dp += bf16_to_f64(go[d]) * bf16_to_f64(v[d]);
            }
            const double p = exp(s * scale - LSE[((size_t)b * Hq + h) * S + i]);
            const double ds = p * (dp - DELTA[((size_t)b * Hq + h) * S + i]);
            for (int d = 0; d < D; ++d) {
                dv_row[d] += p * bf16_to_f64(go[d]);
                dk_row[d] += scale * ds * bf16_to_f64(q[d]);
            }
        }
}

void oracle_attn_bwd(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO, double *dQ,
                     double *dK, double *dV, double *LSE, double *DELTA, int Bn, int S, int Hq, int Hkv, int D,
                     double scale, int causal) {
    const long rows = (long)Bn * Hq * S;
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)S);
        double *o_row = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 8)
        for (long r = 0; r < rows; ++r) {
            const long rr = rows - 1 - r;
            const int i = (int)(rr % S), h = (int)((rr / S) % Hq), b = (int)(rr / ((long)S * Hq));
            double lse, delta;
            bwd_row_stats(Q, Kt, V, dO, S, Hq, Hkv, D, scale, causal, b, h, i, scores, o_row, &lse, &delta);
            LSE[((size_t)b * Hq + h) * S + i] = lse;
            DELTA[((size_t)b * Hq + h) * S + i] = delta;
            bwd_dq_row(Q, Kt, V, dO, S, Hq, Hkv, D, scale, causal, b, h, i, lse, delta,
                       dQ + (((size_t)b * S + i) * Hq + h) * D);
        }
        free(scores);
        free(o_row);
    }
    const long cols = (long)Bn * Hkv * S;
#pragma omp parallel for schedule(dynamic, 8)
    for (long c = 0; c < cols; ++c) {
        const int j = (int)(c % S), kv = (int)((c / S) % Hkv), b = (int)(c / ((long)S * Hkv));
        bwd_dkdv_col(Q, Kt, V, dO, LSE, DELTA, S, Hq, Hkv, D, scale, causal, b, kv, j,
                     dK + (((size_t)b * S + j) * Hkv + kv) * D, dV + (((size_t)b * S + j) * Hkv + kv) * D);
    }
}

/* Selected dQ rows: rows[3r] = {b, h, i}; dQ_rows [nrows][D]. */
void oracle_attn_bwd_dq_rows(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO,
                             const int *rows, int nrows, double *dQ_rows, int S, int Hq, int Hkv, int D,
                             double scale, int causal) {
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)S);
        double *o_row = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < nrows; ++r) {
            double lse, delta;
            const int b = rows[3 * r], h = rows[3 * r + 1], i = rows[3 * r + 2];
            bwd_row_stats(Q, Kt, V, dO, S, Hq, Hkv, D, scale, causal, b, h, i, scores, o_row, &lse, &delta);
            bwd_dq_row(Q, Kt, V, dO, S, Hq, Hkv, D, scale, causal, b, h, i, lse, delta, dQ_rows + (size_t)r * D);
        }
        free(scores);
        free(o_row);
    }
}

/* dK and dV of the LAST ncols key columns (j = S-ncols .. S-1) of (b, kv): only the rows i >= S-ncols
 * of the group's query heads see them, so the row statistics cost O(ncols * S * D) per head.
 * dK_cols, dV_cols [ncols][D].  Causal only. */
void oracle_attn_bwd_dkdv_tail(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO,
                               int b, int kv, int ncols, double *dK_cols, double *dV_cols, int S, int Hq,
                               int Hkv, int D, double scale) {
    const int rep = Hq / Hkv, i0 = S - ncols;
    double *lse = (double *)malloc(sizeof(double) * (size_t)rep * ncols);
    double *delta = (double *)malloc(sizeof(double) * (size_t)rep * ncols);
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)S);
        double *o_row = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < rep * ncols; ++r) {
            const int h = kv * rep + r / ncols, i = i0 + r % ncols;
            bwd_row_stats(Q, Kt, V, dO, S, Hq, Hkv, D, scale, 1, b, h, i, scores, o_row, &lse[r], &delta[r]);
        }
        free(scores);
        free(o_row);
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < ncols; ++c) {
        const int j = i0 + c;
        const uint16_t *k = Kt + (((size_t)b * S + j) * Hkv + kv) * D;
        const uint16_t *v = V + (((size_t)b * S + j) * Hkv + kv) * D;
        double *dk_row = dK_cols + (size_t)c * D, *dv_row = dV_cols + (size_t)c * D;
        for (int d = 0; d < D; ++d) dk_row[d] = dv_row[d] = 0.0;
        for (int hh = 0; hh < rep; ++hh)
            for (int i = j; i < S; ++i) {
                const int h = kv * rep + hh;
                const uint16_t *q = Q + (((size_t)b * S + i) * Hq + h) * D;
                const uint16_t *go = dO + (((size_t)b * S + i) * Hq + h) * D;
                double s = 0.0, dp = 0.0;
                for (int d = 0; d < D; ++d) {
                    s += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
                    dp += bf16_to_f64(go[d]) * bf16_to_f64(v[d]);
                }
                const double p = exp(s * scale - lse[hh * ncols + (i - i0)]);
                const double ds = p * (dp - delta[hh * ncols + (i - i0)]);
                for (int d = 0; d < D; ++d) {
                    dv_row[d] += p * bf16_to_f64(go[d]);
                    dk_row[d] += scale * ds * bf16_to_f64(q[d]);
                }
            }
    }
    free(lse);
    free(delta);
}

/* dK and dV of ARBITRARY key columns cols[0..ncols) of (sequence b, KV head kv).  Column j is summed over every row
 * i that sees it (i >= j under the causal mask, all rows otherwise) of the Hq/Hkv query heads that read the KV head, so
 * the row statistics LSE_i and D_i are needed for all rows from the smallest sampled column on: one pass over those
 * rows (each from its own definition, O(i D) per row), shared by all sampled columns, then the column sums written
 * out as in the full backward.  dK_cols, dV_cols [ncols][D]. */
void oracle_attn_bwd_dkdv_cols(const uint16_t *Q, const uint16_t *Kt, const uint16_t *V, const uint16_t *dO,
                               int b, int kv, const int *cols, int ncols, double *dK_cols, double *dV_cols, int S,
                               int Hq, int Hkv, int D, double scale, int causal) {
    const int rep = Hq / Hkv;
    int i0 = 0;
    if (causal) {
        i0 = S;
        for (int c = 0; c < ncols; ++c)
            if (cols[c] < i0) i0 = cols[c];
    }
    const int nrows = S - i0;
    if (ncols <= 0 || nrows <= 0) return;
    double *lse = (double *)malloc(sizeof(double) * (size_t)rep * nrows);
    double *delta = (double *)malloc(sizeof(double) * (size_t)rep * nrows);
#pragma omp parallel
    {
        double *scores = (double *)malloc(sizeof(double) * (size_t)S);
        double *o_row = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 4)
        for (long r = 0; r < (long)rep * nrows; ++r) {
            const long rr = (long)rep * nrows - 1 - r;          /* long rows first; the order is irrelevant */
            const int hh = (int)(rr / nrows), i = i0 + (int)(rr % nrows);
            bwd_row_stats(Q, Kt, V, dO, S, Hq, Hkv, D, scale, causal, b, kv * rep + hh, i, scores, o_row,
                          &lse[(size_t)hh * nrows + (i - i0)], &delta[(size_t)hh * nrows + (i - i0)]);
        }
        free(scores);
        free(o_row);
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < ncols; ++c) {
        const int j = cols[c];
        const uint16_t *k = Kt + (((size_t)b * S + j) * Hkv + kv) * D;
        const uint16_t *v = V + (((size_t)b * S + j) * Hkv + kv) * D;
        double *dk_row = dK_cols + (size_t)c * D, *dv_row = dV_cols + (size_t)c * D;
        for (int d = 0; d < D; ++d) dk_row[d] = dv_row[d] = 0.0;
        for (int hh = 0; hh < rep; ++hh)
            for (int i = causal ? j : 0; i < S; ++i) {
                const int h = kv * rep + hh;
                const uint16_t *q = Q + (((size_t)b * S + i) * Hq + h) * D;
                const uint16_t *go = dO + (((size_t)b * S + i) * Hq + h) * D;
                double s = 0.0, dp = 0.0;
                for (int d = 0; d < D; ++d) {
                    s += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
                    dp += bf16_to_f64(go[d]) * bf16_to_f64(v[d]);
                }
                const double p = exp(s * scale - lse[(size_t)hh * nrows + (i - i0)]);
                const double ds = p * (dp - delta[(size_t)hh * nrows + (i - i0)]);
                for (int d = 0; d < D; ++d) {
                    dv_row[d] += p * bf16_to_f64(go[d]);
                    dk_row[d] += scale * ds * bf16_to_f64(q[d]);
                }
            }
    }
    free(lse);
    free(delta);
}
