/*
 * basp.h -- C ABI of the B200 (sm_100a) BASP attention-layer library (libbasp.so).
 *
 * One BASP / Ulysses sequence-parallel attention layer, with the N ranks of the paper
 * held as N "virtual ranks" whose shards live in ONE GPU's memory:
 *
 *   plan            Algorithm 1 (group creation) + Algorithm 2 (sequence partitioning)
 *   reshard s2h     the group-local all-to-all of Section IV-C, sequence- to head-sharded
 *   attention       softmax(Q K^T / sqrt(d)) V of Section II-A, causal, per head slice
 *   reshard h2s     the reverse all-to-all (head- back to sequence-sharded)
 *   fused layer     the same three steps in one kernel that reads and writes the
 *                   sequence-sharded shards directly
 *
 * Notation: N ranks; B micro-batch (sequences); G groups (G = B is BASP, G = 1 standard
 * Ulysses); K = N/G ranks per group; Bl = B/G sequences per group; S tokens per sequence;
 * T = ceil(S/K) tokens per rank and sequence; Hq / Hkv query / key-value heads; D head dim.
 *
 * Shard layouts (dense, row-major, bf16 unless stated):
 *   sequence-sharded  rank r holds [Bl][T][H][D]    (tokens l*T..(l+1)*T of its sequences; where K does not divide S
 *                     the last rank of a group holds [Bl][S-(K-1)*T][H][D], see basp_plan_create)
 *   head-sharded      rank r holds [Bl][S][H/K][D]  (heads l*H/K..(l+1)*H/K, all tokens)
 *   LSE               rank r holds fp32 [Bl][Hq/K][S] (natural log of the softmax denominator)
 * with l = r mod K the local rank and g = r / K the group.
 *
 * Conventions for every call
 *   - returns 0 (BASP_OK) or a negative BASP_ERR_* code; nothing throws across the ABI;
 *   - "*_shards" arguments are HOST arrays of n_ranks DEVICE pointers; the array is read
 *     during the call and not retained; every device pointer must be 16-byte aligned;
 *   - the caller owns every device buffer (workspace included); the library allocates no
 *     device memory and keeps no pointer after return; the plan is the only library object
 *     (one exception, stated there: basp_layer_fwd_static keeps its scratch in a fixed array
 *     inside the library's device image and remembers that array's address per device);
 *   - launches are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream); no call synchronises the device except basp_get_status and
 *     basp_layer_fwd_host;
 *   - there is no CPU fallback: without a CUDA device every launch returns BASP_ERR_CUDA.
 */
#ifndef BASP_H_
#define BASP_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BASP_OK               0
#define BASP_ERR_INVALID     -1  /* the paper's preconditions fail (N mod G, B > N, S mod K, head splits) */
#define BASP_ERR_UNSUPPORTED -2  /* valid plan, but outside what the kernels implement               */
#define BASP_ERR_NULL        -3  /* a required pointer is NULL                                       */
#define BASP_ERR_ALIGN       -4  /* a device pointer is not 16-byte aligned                          */
#define BASP_ERR_ALIAS       -5  /* an output shard is also an input shard of an out-of-place step   */
#define BASP_ERR_CUDA        -6  /* a CUDA call failed; see basp_last_cuda_error                     */
#define BASP_ERR_TIMEOUT     -7  /* a bounded wait inside a kernel gave up (see basp_get_status)     */
#define BASP_ERR_WORKSPACE   -8  /* workspace too small                                              */

#define BASP_DTYPE_BF16 0
#define BASP_MAX_RANKS  32

typedef struct basp_plan basp_plan; /* opaque; host memory; immutable; may be shared by threads */

/* Algorithm 1's inputs (world size N, micro-batch B) plus the tensor shape of the layer. */
typedef struct basp_config {
    int n_ranks;     /* N, 1..BASP_MAX_RANKS                                              */
    int micro_batch; /* B                                                                 */
    int num_groups;  /* G: 0 -> B (BASP, Algorithm 1); 1 -> standard Ulysses; must divide N and B */
    int seq_len;     /* S, tokens per sequence                                            */
    int n_q_heads;   /* Hq                                                                */
    int n_kv_heads;  /* Hkv (Hq mod Hkv = 0; query head h reads KV head h / (Hq/Hkv))     */
    int head_dim;    /* D                                                                 */
    int dtype;       /* BASP_DTYPE_BF16                                                   */
    int causal;      /* 1: key j visible to query i iff j <= i; 0: full attention         */
} basp_config;

typedef struct basp_plan_info {
    int group_size;        /* K = N / G  (all-to-all participants; Table I)               */
    int num_groups;        /* G                                                           */
    int seqs_per_group;    /* Bl = B / G                                                  */
    int tokens_per_rank;   /* T = ceil(S / K)  (per sequence; tokens per rank = Bl * T = B*S/N when K | S) */
    int tokens_last_rank;  /* tokens per sequence of a group's LAST rank: T, or S - (K-1)*T when K does not divide S */
    int q_heads_per_rank;  /* Hq / K                                                      */
    int kv_heads_per_rank; /* Hkv / K                                                     */
    size_t q_shard_elems;  /* elements of one rank's Q (or O) shard, either layout (a short last rank's */
                           /* sequence-sharded shard holds tokens_last_rank instead of T tokens)   */
    size_t kv_shard_elems; /* elements of one rank's K (or V) shard (sequence-sharded;    */
                           /* head-sharded too unless KV heads are replicated, see below)  */
    size_t lse_shard_elems;/* fp32 elements of one rank's LSE                             */
} basp_plan_info;

/* Algorithm 2's outputs for one rank. Ranges are half-open. */
typedef struct basp_rank_info {
    int group, local_rank;
    int seq_begin, seq_end;         /* sequences of the micro-batch this rank works on     */
    int token_begin, token_end;     /* its token range inside each of those sequences      */
    int q_head_begin, q_head_end;   /* heads it owns after the first all-to-all            */
    int kv_head_begin, kv_head_end;
} basp_rank_info;

/* ---- plan: Algorithm 1 (K = N/B, contiguous rank blocks, N mod B = 0 asserted) and
 * Algorithm 2 (group = r / K, local = r mod K, chunk = S / K), generalised to G groups
 * as in the workload-equivalence paragraph of Section IV-C.
 * With num_groups = 0 and B > N the plan is the paper's data-parallel fallback: N groups of one rank (K = 1), B/N whole
 * sequences per rank, both exchanges identities.
 * Errors: BASP_ERR_NULL; BASP_ERR_INVALID for N mod G != 0, B mod G != 0 (so B > N needs N | B), an empty last rank
 * (below), Hq mod Hkv != 0,
 * Hq mod K != 0, or Hkv and K with neither Hkv mod K = 0 nor K mod Hkv = 0; BASP_ERR_UNSUPPORTED for
 * dtype != bf16, N > BASP_MAX_RANKS or a head slice whose row ((H/K)*D*2 bytes) is not a multiple of 16 bytes.
 * A group with MORE ranks than KV heads (K mod Hkv = 0, K > Hkv; the paper does not treat grouped-query attention)
 * replicates: KV head h is delivered to the K/Hkv consecutive local ranks whose query heads read it, so every rank
 * holds one KV head (kv_heads_per_rank = 1, kv_head_begin = local_rank / (K/Hkv)); its head-sharded K or V shard is
 * [Bl][S][1][D], larger than the sequence-sharded one.  On the way back such a tensor carries gradients:
 * basp_reshard_h2s (and basp_reshard_grads_h2s for dK, dV) ADDS the K/Hkv copies of a head (fp32 sum, one rounding),
 * which is what the backward pass needs; basp_reshard_h2s is therefore not the inverse of basp_reshard_s2h for it.
 * A sequence length that K does not divide (Algorithm 2 writes the chunk as L / K and the paper says nothing about a
 * remainder): the chunk is T = ceil(S / K); local rank l holds tokens [l*T, min((l+1)*T, S)), so only the last rank of
 * a group is short, and its SEQUENCE-sharded shards are the compact [Bl][S - (K-1)*T][H][D] (head-sharded shards and LSE
 * do not change: every rank holds whole sequences there).  (K-1)*T >= S, an empty last rank, is BASP_ERR_INVALID.
 * On success *out owns a host object; release it with basp_plan_destroy. */
int basp_plan_create(const basp_config *cfg, basp_plan **out);
int basp_plan_destroy(basp_plan *plan);
int basp_plan_get_info(const basp_plan *plan, basp_plan_info *info);
int basp_plan_get_rank(const basp_plan *plan, int rank, basp_rank_info *info);
/* ranks_out: host array of K ints; group i is ranks i*K .. i*K+K-1 (Algorithm 1). */
int basp_plan_group_ranks(const basp_plan *plan, int group, int *ranks_out);

/* ---- group formation when B does not divide N.  Algorithm 1 asserts N mod B = 0 and the paper's limitations section
 * leaves the other case to future work; this keeps Algorithm 1's structure (B groups of contiguous ranks, one
 * sequence each) with sizes that differ by at most one: the first N mod B groups have ceil(N/B) ranks, the others
 * floor(N/B).  The result is at most two PARTS, each a uniform plan over its own contiguous ranks and sequences:
 * part 0 covers ranks [0, n_ranks_0) and sequences [0, n_seqs_0) (the larger groups), part 1 the rest.  Every other
 * call of this header is made once per part with part.plan and with the shard arrays advanced by part.rank_begin
 * (`shards + part.rank_begin`); the parts are independent (no exchange crosses a group), so they may run on different
 * streams.  With N mod B = 0 there is one part, identical to basp_plan_create's plan.
 * cfg->num_groups must be 0 or equal to micro_batch (BASP grouping).  Errors: as basp_plan_create for each part
 * (e.g. BASP_ERR_INVALID when a group size divides neither head count); B > N gives the one data-parallel plan.  On success the
 * caller owns parts[i].plan for i < *n_parts (basp_plan_destroy). */
typedef struct basp_plan_part {
    basp_plan *plan;
    int rank_begin, n_ranks;   /* global ranks [rank_begin, rank_begin + n_ranks)            */
    int seq_begin, n_seqs;     /* sequences of the micro-batch [seq_begin, seq_begin + n_seqs) */
    int group_size;            /* ranks per group in this part                               */
} basp_plan_part;
int basp_plan_create_parts(const basp_config *cfg, basp_plan_part parts[2], int *n_parts);

/* ---- reshards: the two all-to-alls of the Ulysses layer confined to each group
 * (Section II-C, Section IV-C), as out-of-place permutations inside device memory.
 *   s2h: head[gK+m][bl][s][h'][d] = seq[gK + s/T][bl][s mod T][m*H/K + h'][d]
 *   h2s: seq[gK+l][bl][t][m*H/K + h'][d] = head[gK+m][bl][l*T + t][h'][d]
 * n_heads = H must be a multiple of K with (H/K)*D*2 bytes a multiple of 16.  Bit-exact.
 * Errors: NULL / ALIGN / ALIAS (a destination shard equal to a source shard) / INVALID
 * (n_heads) / CUDA. */
int basp_reshard_s2h(const basp_plan *plan, int n_heads, const void *const *seq_shards,
                     void *const *head_shards, void *stream);
int basp_reshard_h2s(const basp_plan *plan, int n_heads, const void *const *head_shards,
                     void *const *seq_shards, void *stream);
/* Q (Hq heads), K and V (Hkv heads) in ONE launch. */
int basp_reshard_qkv_s2h(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                         const void *const *v_seq, void *const *q_head, void *const *k_head,
                         void *const *v_head, void *stream);

/* ---- attention over each rank's head slice (Section II-A equation; the tiled,
 * online-softmax evaluation the paper cites from FlashAttention):
 *   O[i] = sum_{j visible} softmax_j(scale * q_i . k_j) v_j,   LSE[i] = ln sum_j exp(scale * q_i . k_j)
 * Inputs/outputs are HEAD-sharded; lse_shards may be NULL (then no LSE is written), else a
 * host array of n_ranks device pointers to fp32 [Bl][Hq/K][S].  softmax_scale = 0 selects
 * 1/sqrt(D); a negative, infinite or NaN scale is BASP_ERR_INVALID in every call that takes one.  bf16 operands, fp32 accumulation and softmax, P rounded to bf16 before P.V.
 * Requires D a multiple of 16 up to 128 (else BASP_ERR_UNSUPPORTED; the kernels are 64 and 128 columns wide, for a
 * D in between the tile loads zero-fill the missing columns); S is arbitrary (a ragged last tile is masked).
 * A bounded wait that expires inside the kernel is reported by basp_get_status. */
int basp_attn_fwd(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                  const void *const *v_head, void *const *o_head, float *const *lse_shards,
                  float softmax_scale, void *stream);

/* ---- the whole layer on SEQUENCE-sharded shards: s2h(Q,K,V) -> attention -> h2s(O).
 * `workspace` is device memory of at least basp_workspace_bytes(plan) bytes (16-byte
 * aligned) that receives the head-sharded Q, K, V and O; its contents afterwards are
 * unspecified.  Three launches.  Errors as above plus BASP_ERR_WORKSPACE. */
int basp_layer_fwd(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                   const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                   void *workspace, size_t workspace_bytes, float softmax_scale, void *stream);
size_t basp_workspace_bytes(const basp_plan *plan);

/* ---- the three-launch layer WITHOUT caller workspace and without any allocation (the paper
 * has no counterpart: this entry point exists for the sake of callers, not of the method).
 * Some callers cannot allocate device memory at the point where they need the layer: the whole
 * device heap may already belong to another allocator or memory pool, or the call sits in a
 * latency-critical loop in which the device-wide synchronisation of cudaMalloc / cudaFree is
 * not acceptable.  For them the head-sharded Q, K, V and O go into a fixed array of
 * BASP_STATIC_SCRATCH_BYTES that is part of this library's image: every GPU that loads the
 * library holds that much memory until the process exits.  The call runs no cudaMalloc, cudaFree
 * or other allocating routine; inputs and outputs are still the caller's.
 *   - Plans whose basp_workspace_bytes exceeds BASP_STATIC_SCRATCH_BYTES are refused with
 *     BASP_ERR_WORKSPACE (basp_last_cuda_error then names both sizes).
 *   - The first call on each device is the set-up call: it looks up the array's device address (one
 *     runtime query, made with that device current), and if nothing of this library's device code
 *     has run on that device before, that is also when the CUDA runtime loads the library's image and
 *     the GPU commits the array's memory.  Make that first call at start-up: before the device's
 *     memory is handed to another pool, and before starting any stream capture.  Later calls leave
 *     the amount of free device memory exactly as they found it.
 *   - All calls on a device share the one array.  It keeps whatever the last call wrote; nothing
 *     needs clearing because each call overwrites every byte it later reads.  Two calls that can
 *     overlap on the GPU (different streams, no dependency) race on it: serialise them.
 * Results are bit-identical to basp_layer_fwd's (the same launches on the same inputs). */
#define BASP_STATIC_SCRATCH_BYTES (16u << 20)
int basp_layer_fwd_static(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                          const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                          float softmax_scale, void *stream);

/* ---- the same layer as ONE kernel: attention tiles are fetched straight from the
 * sequence-sharded sources (token tile at sequence position s lives on rank gK + s/T) and
 * O tiles are stored straight into the sequence-sharded destination, so the head-sharded
 * copies never exist.  Requires T to be a multiple of 128 (a tile must not straddle two ranks) and, where K does not
 * divide S (a short last shard), one sequence per shard (Bl = 1, as in BASP grouping), else BASP_ERR_UNSUPPORTED.
 * No workspace. */
int basp_layer_fwd_fused(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                         const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                         float softmax_scale, void *stream);

/* ---- one physical GPU's share of the path when the n_ranks ranks are spread over several GPUs (Section IV-A:
 * contiguous ranks per GPU; Section IV-C: the exchanges stay inside a group).  Every call takes the same host arrays
 * of n_ranks device pointers as its single-GPU form; entries of ranks on other GPUs are addresses of PEER memory
 * mapped into this process (CUDA IPC or symmetric memory), entries the call does not touch may be NULL.  Only ranks
 * [rank_begin, rank_begin + rank_count) - the ranks this GPU hosts - act:
 *   basp_reshard_qkv_s2h_ranks  pushes their sequence shards into the head shards of every member of their groups
 *                               (plain stores; remote members over NVLink);
 *   basp_attn_fwd_ranks         attention over their own head shards (local memory only);
 *   basp_reshard_h2s_ranks      pulls their sequence shards of O together from the group's head shards (plain loads);
 *   basp_layer_fwd_fused_ranks  the three steps as one kernel: Q/K/V tiles are fetched from the group's sequence
 *                               shards wherever they live (plain TMA tile loads, one per thread block) and O tiles are stored
 *                               into the owner's sequence shard - exchange and attention overlap tile by tile.
 * The caller orders the GPUs on the host: every GPU's inputs are complete before any GPU launches, and nobody reuses
 * a buffer before all GPUs' launches have finished (a barrier of the process group on both sides; the kernels never
 * wait for one another).  The union of the calls over all GPUs equals the single-GPU call bit for bit.
 * Errors as the single-GPU forms; INVALID for a range outside [0, n_ranks). */
int basp_reshard_qkv_s2h_ranks(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                               const void *const *v_seq, void *const *q_head, void *const *k_head,
                               void *const *v_head, int rank_begin, int rank_count, void *stream);
int basp_reshard_h2s_ranks(const basp_plan *plan, int n_heads, const void *const *head_shards,
                           void *const *seq_shards, int rank_begin, int rank_count, void *stream);
int basp_attn_fwd_ranks(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                        const void *const *v_head, void *const *o_head, float *const *lse_shards,
                        float softmax_scale, int rank_begin, int rank_count, void *stream);
int basp_layer_fwd_fused_ranks(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                               const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                               float softmax_scale, int rank_begin, int rank_count, void *stream);

/* After basp_layer_fwd returns, the workspace holds the head-sharded Q, K, V and O of every rank; this call
 * writes their addresses (n_ranks pointers each) so that a training step can keep them for the backward pass
 * instead of resharding again.  (The fixed array of basp_layer_fwd_static cannot be reached from outside.) */
int basp_layer_workspace_shards(const basp_plan *plan, void *workspace, void **q_head, void **k_head,
                                void **v_head, void **o_head);

/* ---- attention backward over each rank's head slice (the paper trains through this layer but
 * never writes the backward out; it is the chain rule applied to the Section II-A equation):
 *   P_ij = exp(scale q_i.k_j - LSE_i),  Delta_i = dO_i.O_i,  dV_j = sum_i P_ij dO_i,
 *   dS_ij = P_ij (dO_i.v_j - Delta_i),  dQ_i = scale sum_j dS_ij k_j,  dK_j = scale sum_i dS_ij q_i,
 * with dK, dV summed over the Hq/Hkv query heads of a KV head.  All operands HEAD-sharded: q, o, do, dq
 * [Bl][S][Hq/K][D]; k, v, dk, dv [Bl][S][Hkv/K][D]; lse as written by the forward.  bf16 in and out,
 * fp32 accumulation; dQ is accumulated with floating-point atomics, so its last bits may differ
 * between runs.  Requires D a multiple of 16 up to 128 (two kernels, 64 and 128 columns wide; a D in between runs on
 * the wider one with the missing columns zero-filled by the tile loads); S is arbitrary (ragged last tiles are masked).
 * `workspace`: device memory of at least basp_attn_bwd_workspace_bytes(plan) bytes (fp32 dQ accumulator, Delta and a
 * few counters).  For long causal sequences at D > 64 the thread blocks that work on one (rank, sequence, KV head)
 * start their sweeps together (they wait for one another inside the launch, every wait bounded), so that launch is
 * made cooperatively; where the device cannot hold all of its blocks at once the ordinary schedule runs instead. */
int basp_attn_bwd(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                  const void *const *v_head, const void *const *o_head, const void *const *do_head,
                  const float *const *lse_shards, void *const *dq_head, void *const *dk_head,
                  void *const *dv_head, void *workspace, size_t workspace_bytes, float softmax_scale,
                  void *stream);
size_t basp_attn_bwd_workspace_bytes(const basp_plan *plan);
/* The same gradients, bit-identical from run to run: two passes (dK and dV with the key tile resident, dQ with the
 * query tile resident) instead of one pass that adds dQ partial sums into a global accumulator in whatever order the
 * thread blocks finish.  Costs the scores and the element-wise part twice (slower than the one-pass form); same
 * arguments, workspace and errors as basp_attn_bwd. */
int basp_attn_bwd_deterministic(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                                const void *const *v_head, const void *const *o_head, const void *const *do_head,
                                const float *const *lse_shards, void *const *dq_head, void *const *dk_head,
                                void *const *dv_head, void *workspace, size_t workspace_bytes, float softmax_scale,
                                void *stream);

/* dQ (Hq heads), dK and dV (Hkv heads) head- to sequence-sharded in ONE launch: the reverse
 * all-to-alls of the gradients. */
int basp_reshard_grads_h2s(const basp_plan *plan, const void *const *dq_head, const void *const *dk_head,
                           const void *const *dv_head, void *const *dq_seq, void *const *dk_seq,
                           void *const *dv_seq, void *stream);

/* ---- backward of the whole layer from SEQUENCE-sharded activations: for a forward pass that kept no head-sharded
 * copies (basp_layer_fwd_fused).  The all-to-alls of Q, K, V, O and dO are redone here (two launches), then the
 * attention backward and the reverse all-to-alls of the gradients.  lse_shards: as written by the forward.  `workspace`
 * of at least basp_layer_bwd_seq_workspace_bytes(plan) bytes holds the head-sharded Q, K, V, O, dO, dQ, dK, dV and the
 * attention-backward workspace. */
int basp_layer_bwd_seq(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                       const void *const *v_seq, const void *const *o_seq, const float *const *lse_shards,
                       const void *const *do_seq, void *const *dq_seq, void *const *dk_seq, void *const *dv_seq,
                       void *workspace, size_t workspace_bytes, float softmax_scale, void *stream);
size_t basp_layer_bwd_seq_workspace_bytes(const basp_plan *plan);

/* ---- backward of the whole layer: all-to-all of dO (sequence- to head-sharded), attention
 * backward on the saved head-sharded Q, K, V, O and LSE of the forward, reverse all-to-alls of
 * dQ, dK, dV.  do_seq / dq_seq / dk_seq / dv_seq are SEQUENCE-sharded.  `workspace` of at least
 * basp_layer_bwd_workspace_bytes(plan) bytes holds the head-sharded dO, dQ, dK, dV and the
 * attention-backward workspace. */
int basp_layer_bwd(const basp_plan *plan, const void *const *q_head, const void *const *k_head,
                   const void *const *v_head, const void *const *o_head, const float *const *lse_shards,
                   const void *const *do_seq, void *const *dq_seq, void *const *dk_seq, void *const *dv_seq,
                   void *workspace, size_t workspace_bytes, float softmax_scale, void *stream);
size_t basp_layer_bwd_workspace_bytes(const basp_plan *plan);

/* ---- the fused layer for callers whose shards are in HOST memory: copies every Q/K/V
 * shard host->device into `device_arena` (device memory, >= basp_host_arena_bytes(plan)
 * bytes), runs the fused kernel, copies every O shard device->host and waits for the stream.
 * Copies and kernels are pipelined: Q travels in pieces of a few 256-row query blocks, one launch per piece
 * starts as soon as the piece and the K and V shards it needs have arrived (with the causal mask the rows of local
 * rank l need the shards of local ranks 0..l of its group only), and its O rows are read back while later pieces
 * are computed; the order on the bus depends on whether the link or the GPU is the longer side (see layer.cu).
 * Copies and kernels run on library-owned streams (created on first use, per device; no device memory) that
 * are joined to `stream` before and after; calls that overlap in time on one device share them and must be
 * serialised by the caller.  Needs T to be a multiple of 256 for the pipelining (else one launch per group).
 * q/k/v/o_seq_host are host arrays of n_ranks HOST pointers (pinned memory makes the copies
 * asynchronous; pageable memory works, slower). */
int basp_layer_fwd_host(const basp_plan *plan, const void *const *q_seq_host,
                        const void *const *k_seq_host, const void *const *v_seq_host,
                        void *const *o_seq_host, void *device_arena, size_t arena_bytes,
                        float softmax_scale, void *stream);
size_t basp_host_arena_bytes(const basp_plan *plan);

/* ---- the projections on either side of the attention core (Section II-A: Q = X W_Q, K = X W_K, V = X W_V for
 * every head, MultiHead = Concat(H_1..H_h) W_O), applied to every rank's sequence shard in one launch.
 *   basp_qkv_proj:  [Q | K | V]_r = X_r . W_qkv^T   X_r: bf16 [Bl*T][hidden] (rank r's tokens), W_qkv: bf16
 *                   [(Hq + 2 Hkv) * D][hidden] (rows: W_Q's heads, then W_K's, then W_V's); the three column blocks
 *                   are written to q_seq[r] ([Bl][T][Hq][D]), k_seq[r], v_seq[r] ([Bl][T][Hkv][D]): the layout
 *                   basp_reshard_qkv_s2h and basp_layer_fwd_fused read.
 *   basp_out_proj:  Y_r = O_r . W_o^T               O_r: bf16 [Bl*T][Hq*D] (the layer's sequence-sharded output),
 *                   W_o: bf16 [hidden][Hq*D], Y_r: bf16 [Bl*T][hidden].
 * bf16 operands, fp32 accumulation, bf16 results.  Requires hidden a multiple of 64 (qkv) / 256 (out) and
 * Hq*D, Hkv*D multiples of 256, else BASP_ERR_UNSUPPORTED.  Weights are shared by all ranks (one device pointer). */
int basp_qkv_proj(const basp_plan *plan, int hidden, const void *const *x_seq, const void *w_qkv,
                  void *const *q_seq, void *const *k_seq, void *const *v_seq, void *stream);
/* The QKV projection with rotary position embedding applied to Q and K in the epilogue (the paper does not treat
 * position encodings; this is the rotate-half convention of the Llama / Qwen models it trains): within a head, feature
 * j < D/2 pairs with feature j + D/2,  y_j = x_j cos - x_{j+D/2} sin,  y_{j+D/2} = x_{j+D/2} cos + x_j sin,  computed
 * on the fp32 accumulators and rounded to bf16 once.  rope_cos / rope_sin: device fp32 tables [D/2][S], FEATURE-major
 * (entry [j][pos]: the 128 rows of an output tile are consecutive positions, so this order reads whole lines), pos =
 * the token's position in its sequence (local rank * T + row mod T).  V is not rotated.  Requires D = 64 or 128. */
int basp_qkv_proj_rope(const basp_plan *plan, int hidden, const void *const *x_seq, const void *w_qkv,
                       const float *rope_cos, const float *rope_sin, void *const *q_seq, void *const *k_seq,
                       void *const *v_seq, void *stream);
int basp_out_proj(const basp_plan *plan, int hidden, const void *const *o_seq, const void *w_o,
                  void *const *y_seq, void *stream);

/* ---- device status.  Every wait inside the kernels (on a shared-memory barrier) is bounded;
 * when one expires the kernel records where, lets its copies drain, frees its tensor memory
 * and returns.  basp_get_status synchronises `stream`, copies the four status words of the
 * current device to status_out (host, 4 ints: {code, role, block, detail}; may be NULL) and
 * returns BASP_OK or BASP_ERR_TIMEOUT.  basp_clear_status zeroes them (asynchronously). */
int basp_get_status(void *stream, int *status_out);
int basp_clear_status(void *stream);

/* Diagnostic: launches a one-CTA kernel whose wait cannot complete, with a wait limit of limit_us microseconds
 * (1 .. 1 000 000), so that a caller can check that an expired wait is reported ({code 2, role 100, block, waited
 * microseconds} through basp_get_status -> BASP_ERR_TIMEOUT) and that the context stays usable afterwards.  The
 * kernel ends by itself; nothing faults.  Clear the status words afterwards with basp_clear_status. */
int basp_selftest_wait_timeout(unsigned int limit_us, void *stream);

const char *basp_strerror(int code);
/* Text of the last CUDA error seen by the calling thread inside this library ("" if none). */
const char *basp_last_cuda_error(void);
/* Number of kernel launches issued by this library in the calling process so far. */
long long basp_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BASP_H_ */
