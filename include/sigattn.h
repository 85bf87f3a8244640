/*
 * sigattn — fused sigmoid self-attention, forward and backward, for NVIDIA B200 (sm_100a).
 *
 * C ABI of libsigattn.so.  Plain pointers and sizes only; no framework types.
 *
 * Operation (Section 2, Eq. 3 of "Theory, Analysis, and Best Practices for Sigmoid
 * Self-Attention"; tiled forward = Algorithm 1, tiled backward = Algorithm 2 of
 * Appendix F.1), per batch b and head h, with i the query row and j the key row:
 *
 *     x_ij = scale * <Q_i, K_j> + bias - slope_h * |i - j|
 *     P_ij = sigmoid(x_ij), and P_ij = 0 where causal != 0 and j > i
 *     O    = P V
 *
 *     dV = P^T dO,  dP = dO V^T,  dS = P * (1 - P) * dP,
 *     dQ = scale * dS K,  dK = scale * dS^T Q
 *
 * The factor in dQ and dK is `scale` (= 1/sqrt(D) in the paper's use), the derivative
 * of the scaled logit; the sqrt(d) printed in the paper's table is a typo.  No row
 * maximum, row sum, log-sum-exp or rowsum(dO * O) exists anywhere: the backward
 * recomputes P from Q, K alone (activation recomputation, Section 4).
 *
 * Layout.  Every tensor is contiguous row-major [B, H, N, D], D innermost.
 * dtype 0: bfloat16 tensors, tensor-core path (tcgen05 MMA, fp32 accumulation).
 * dtype 1: float32 tensors, CUDA-core debug path (exact expf and division).
 * D must be 64 or 128.  Base pointers must be 16-byte aligned.  `alibi_slopes` is
 * NULL or a device pointer to H floats (the positive slope of each head, shared by
 * all batches); NULL behaves like all-zero slopes.
 *
 * Ownership.  All pointers are DEVICE pointers owned by the caller, except where a
 * function says "host".  The library allocates no device memory on these calls; the
 * backward's fp32 dQ accumulator lives in the caller's `workspace`.  Outputs are
 * overwritten in full; inputs are never written.
 *
 * Asynchrony.  Work is enqueued on `stream` (a cudaStream_t; NULL = default stream)
 * and the call returns without synchronising.
 *
 * Errors.  Return value 0 = success; negative = error, nothing was launched:
 *   -1 null pointer            -2 unsupported shape (D not 64/128, a size < 1, too large)
 *   -3 misaligned pointer      -4 bad dtype or flag
 *   -5 workspace too small     -6 device is not sm_100
 *   -7 CUDA runtime/driver error at set-up or launch (see sigattn_last_cuda_error)
 *   -8 a bounded device-side wait expired in an earlier launch (reported by sigattn_check)
 *   -9 problem too large for sigattn_bwd_static_scratch's built-in scratch
 * Arguments are validated before anything is enqueued.
 *
 * Launches in flight.  Some launches hand their work items out dynamically from a device
 * counter owned by the library: the padded-batch, unpadded-batch, row-factor and accumulating
 * entry points, sigattn_fwd_decode, and the plain calls when a problem has so few work items
 * that the library divides them (fewer (batch, head, tile) items than about one per SM).  The
 * library holds 1024 such counters per kernel family and hands them out round robin, so at
 * most 1024 of these launches may be in flight at once in one process (over all streams);
 * beyond that two launches would share a counter and skip or repeat items.  A kernel that
 * sees its counter advance further than one launch can advance it records a device-side
 * error, which sigattn_check reports as -8.
 */
#ifndef SIGATTN_H_
#define SIGATTN_H_

#include <stddef.h>

#if defined(__GNUC__)
#define SIGATTN_API __attribute__((visibility("default")))
#else
#define SIGATTN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define SIGATTN_OK 0
#define SIGATTN_ERR_NULL (-1)
#define SIGATTN_ERR_SHAPE (-2)
#define SIGATTN_ERR_ALIGN (-3)
#define SIGATTN_ERR_FLAG (-4)
#define SIGATTN_ERR_WORKSPACE (-5)
#define SIGATTN_ERR_ARCH (-6)
#define SIGATTN_ERR_CUDA (-7)
#define SIGATTN_ERR_DEVICE_TIMEOUT (-8)
#define SIGATTN_ERR_STATIC_SCRATCH (-9)

#define SIGATTN_DTYPE_BF16 0
#define SIGATTN_DTYPE_FP32 1

/* Forward (Eq. 3; Algorithm 1).  q, k, v: inputs; o: output; all [B, H, N, D].
 * O is bit-reproducible from run to run.  (Calls with so few (batch, head) pairs that they cannot
 * fill the GPU divide the keys of a work item over two thread blocks that add their bf16 shares
 * into the cleared O; the sum of two shares does not depend on their order.) */
SIGATTN_API int sigattn_fwd(const void* q, const void* k, const void* v, void* o,
                int B, int H, int N, int D,
                float scale, float bias, int causal,
                const float* alibi_slopes, int dtype, void* stream);

/* Backward (sigmoid column of the forward/backward table, Appendix F.1; Algorithm 2).
 * q, k, v, d_o: inputs; dq, dk, dv: outputs; all [B, H, N, D].
 * workspace: device scratch of at least sigattn_bwd_workspace_bytes(...) bytes,
 * 256-byte aligned; its contents on entry are irrelevant and on exit unspecified.
 * Two calls that share a workspace must not overlap on the device.
 * dQ sums contributions of different key tiles with floating-point atomics, so its
 * low-order bits may differ from run to run; dK and dV are deterministic.  (With so few
 * (batch, head) pairs that the work items cannot fill the GPU, the query tiles of a key tile are
 * divided over two thread blocks that add their bf16 shares of dK, dV into the cleared outputs;
 * the sum of two shares does not depend on their order.) */
SIGATTN_API int sigattn_bwd(const void* q, const void* k, const void* v, const void* d_o,
                void* dq, void* dk, void* dv,
                int B, int H, int N, int D,
                float scale, float bias, int causal,
                const float* alibi_slopes, int dtype,
                void* workspace, size_t workspace_bytes, void* stream);

/* Backward for callers that cannot obtain device scratch at all.  (The paper has no
 * counterpart: this entry point exists for how the library is embedded, not for the
 * method.)  Who needs it: code that runs where cudaMalloc and friends are off limits -
 * inside a framework's allocator callback or a real-time loop, in a plugin whose host
 * forbids allocations after start-up, or in a process whose memory pool has already
 * handed every byte to someone else - and that therefore cannot pass sigattn_bwd a
 * workspace.  Same operation, arguments and results as sigattn_bwd, minus the workspace:
 * the fp32 dQ accumulator lives in a fixed array inside the library instead.
 *
 * Limits and rules:
 *  - B*H*N*D must not exceed sigattn_bwd_static_scratch_max_elements() (4 Mi elements,
 *    a 16 MiB array that every GPU on which the library is loaded holds until the
 *    process exits); larger problems return SIGATTN_ERR_STATIC_SCRATCH and launch nothing.
 *  - The call allocates nothing: no cudaMalloc, cudaFree or allocating library routine.
 *  - The first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress, with that device current); make that first call outside any
 *    stream capture.
 *  - All calls on a device share the one array.  It keeps whatever the last call left in
 *    it, so every call clears the part it uses before accumulating; two calls that overlap
 *    on the device (different streams, or sigattn_bwd_static_scratch from two threads)
 *    race on it and produce garbage.  Serialise them, e.g. by using one stream. */
SIGATTN_API int sigattn_bwd_static_scratch(const void* q, const void* k, const void* v, const void* d_o,
                               void* dq, void* dk, void* dv,
                               int B, int H, int N, int D,
                               float scale, float bias, int causal,
                               const float* alibi_slopes, int dtype, void* stream);

/* Largest B*H*N*D that sigattn_bwd_static_scratch accepts. */
SIGATTN_API size_t sigattn_bwd_static_scratch_max_elements(void);

/* sigattn_fwd with one bias per (batch, head) instead of one scalar: the speech models of
 * Section 5.4 / Appendix G.4 use b = -log n with n the length of each sample, and a
 * learnable bias is ablated there and in Appendix G.2.2.  `bias_bh` is a DEVICE pointer to
 * B*H floats, row-major [B][H], 4-byte aligned, read while the kernel runs; entry [b][h]
 * takes the place of `bias` for that sequence and head.  Everything else as sigattn_fwd. */
SIGATTN_API int sigattn_fwd_bias_vec(const void* q, const void* k, const void* v, void* o,
                         int B, int H, int N, int D,
                         float scale, const float* bias_bh, int causal,
                         const float* alibi_slopes, int dtype, void* stream);

/* sigattn_bwd with the bias vector of sigattn_fwd_bias_vec, and optionally the gradient
 * of L = sum(O * dO) with respect to it: if `dbias_bh` is not NULL it is a DEVICE pointer
 * to B*H floats that receive db[b][h] = sum over (i, j) of dS_ij (dS = P (1 - P) dP; the
 * bias enters every logit additively).  The paper prints no formula for db; a bias shared
 * by heads or sequences gets the sum of their entries.  The array is cleared and then
 * added into with fp32 atomics, so its last bits depend on the order of the additions.
 * Everything else as sigattn_bwd. */
SIGATTN_API int sigattn_bwd_bias_vec(const void* q, const void* k, const void* v, const void* d_o,
                         void* dq, void* dk, void* dv,
                         int B, int H, int N, int D,
                         float scale, const float* bias_bh, int causal,
                         const float* alibi_slopes, int dtype,
                         float* dbias_bh,
                         void* workspace, size_t workspace_bytes, void* stream);

/* sigattn_bwd with the gradient of a learnable temperature.  The paper's temperature variant
 * (footnote to the list of variants in Section 5; the LayerScale-free ablation of Appendix G.2.2)
 * computes sigmoid(e^t * Q K^T / sqrt(d) + b) V with a learnable scalar t.  The forward needs no
 * entry point of its own: pass scale * e^t as `scale`.  This backward does the same and also
 * returns dL/dt for L = sum(O * dO): with x_ij = scale' q_i k_j + b, dL/dt = sum_ij dS_ij * scale'
 * q_i k_j = sum_i <Q_i, dQ_i> (the paper prints no formula), one value per (batch, head) in
 * `dtemp_bh`, a DEVICE pointer to B*H floats, row-major [B][H]; a temperature shared by heads or
 * sequences gets the sum of their entries.  On the bf16 path the sum is taken in the pass that
 * converts the fp32 dQ accumulator (from the unrounded dQ, with fp32 atomics per block, so its last
 * bits depend on the order); on the fp32 path a separate reduction runs after the gradients.
 * `bias_bh` (NULL: use the scalar `bias`) and `dbias_bh` (NULL: no bias gradient) as in
 * sigattn_bwd_bias_vec.  Everything else as sigattn_bwd. */
SIGATTN_API int sigattn_bwd_dtemp(const void* q, const void* k, const void* v, const void* d_o,
                      void* dq, void* dk, void* dv,
                      int B, int H, int N, int D,
                      float scale, float bias, const float* bias_bh, int causal,
                      const float* alibi_slopes, int dtype,
                      float* dbias_bh, float* dtemp_bh,
                      void* workspace, size_t workspace_bytes, void* stream);

/* Multi-query / grouped-query attention (the multi-query ablation of Section 5.1): k and v
 * (and dk, dv) have H_kv heads, [B, H_kv, N, D], with H a multiple of H_kv; query head h
 * reads key/value head h / (H / H_kv), i.e. consecutive query heads share one.  The paper
 * gives no layout; this is the usual one.  q, o, d_o, dq stay [B, H, N, D].  `bias_bh` is
 * NULL (the scalar `bias` is used) or a DEVICE pointer to B*H floats as in
 * sigattn_fwd_bias_vec (then `bias` is ignored); slopes are per query head.  H_kv == H is
 * plain multi-head attention.  H % H_kv != 0 or H_kv < 1: SIGATTN_ERR_SHAPE. */
SIGATTN_API int sigattn_fwd_gqa(const void* q, const void* k, const void* v, void* o,
                    int B, int H, int H_kv, int N, int D,
                    float scale, float bias, const float* bias_bh, int causal,
                    const float* alibi_slopes, int dtype, void* stream);

/* Backward of sigattn_fwd_gqa: dk, dv are [B, H_kv, N, D] and hold the sums over the query
 * heads that read each key/value head (accumulated on chip: a work item keeps dK_j, dV_j
 * of one key/value head in tensor memory while it walks the query tiles of all its query
 * heads).  When B * H_kv * ceil(N / 128) work items cannot fill the GPU (multi-query attention at
 * a small batch) the query heads of a group are divided over several work items, which add their
 * dK_j, dV_j into the cleared outputs with bf16 reduce-adds; dk and dv then depend on the order of
 * the additions in their last bits, like dq.  `dbias_bh`: NULL or B*H floats as in
 * sigattn_bwd_bias_vec.  The workspace is that of sigattn_bwd for (B, H, N, D). */
SIGATTN_API int sigattn_bwd_gqa(const void* q, const void* k, const void* v, const void* d_o,
                    void* dq, void* dk, void* dv,
                    int B, int H, int H_kv, int N, int D,
                    float scale, float bias, const float* bias_bh, int causal,
                    const float* alibi_slopes, int dtype,
                    float* dbias_bh,
                    void* workspace, size_t workspace_bytes, void* stream);

/* N_q queries against N_k keys and values: q, o (d_o, dq) are [B, H, N_q, D], k, v (dk, dv)
 * are [B, H_kv, N_k, D].  The paper defines self-attention (N_q = N_k); generation with a
 * cache of earlier keys and values, where its inference gains are measured (Appendix F.3),
 * has the queries at the LAST N_q positions: query i sits at position i + N_k - N_q for the
 * causal mask (keys j <= i + N_k - N_q are kept) and for the ALiBi distance.  With causal = 1,
 * N_k >= N_q is required (SIGATTN_ERR_SHAPE otherwise); without a mask any N_q, N_k >= 1 are
 * allowed (cross-attention).  H_kv, bias_bh as in sigattn_fwd_gqa.  N_q = N_k and H_kv = H
 * is sigattn_fwd. */
SIGATTN_API int sigattn_fwd_nk(const void* q, const void* k, const void* v, void* o,
                   int B, int H, int H_kv, int N_q, int N_k, int D,
                   float scale, float bias, const float* bias_bh, int causal,
                   const float* alibi_slopes, int dtype, void* stream);

/* Backward of sigattn_fwd_nk.  The workspace is that of sigattn_bwd for (B, H, N_q, D). */
SIGATTN_API int sigattn_bwd_nk(const void* q, const void* k, const void* v, const void* d_o,
                   void* dq, void* dk, void* dv,
                   int B, int H, int H_kv, int N_q, int N_k, int D,
                   float scale, float bias, const float* bias_bh, int causal,
                   const float* alibi_slopes, int dtype,
                   float* dbias_bh,
                   void* workspace, size_t workspace_bytes, void* stream);

/* One contiguous shard of keys and values (over devices, or over callers that split a long
 * sequence).  Sigmoid attention has no row normalisation (Section 4), so O is the plain
 * sum over shards of the attention of all queries against one shard, dQ likewise, and
 * dK, dV of a shard need only that shard: the distributed setting the paper leaves open in
 * its Limitations needs one sum per tensor and no log-sum-exp.  These are sigattn_fwd_nk /
 * sigattn_bwd_nk with the position of the queries stated instead of implied: `pos0` is the
 * position of query row 0 minus the position of the shard's first key (any value in
 * +-2^30; N_k - N_q reproduces sigattn_fwd_nk).  Query i keeps keys j <= i + pos0 when
 * causal = 1 and measures the ALiBi distance from i + pos0; a query that lies before every
 * key of the shard gets an all-zero row of O (and contributes nothing to the gradients).
 * The caller adds the summands (e.g. one all-reduce). */
SIGATTN_API int sigattn_fwd_shard(const void* q, const void* k, const void* v, void* o,
                      int B, int H, int H_kv, int N_q, int N_k, int D,
                      float scale, float bias, const float* bias_bh, int causal, int pos0,
                      const float* alibi_slopes, int dtype, void* stream);

SIGATTN_API int sigattn_bwd_shard(const void* q, const void* k, const void* v, const void* d_o,
                      void* dq, void* dk, void* dv,
                      int B, int H, int H_kv, int N_q, int N_k, int D,
                      float scale, float bias, const float* bias_bh, int causal, int pos0,
                      const float* alibi_slopes, int dtype,
                      float* dbias_bh,
                      void* workspace, size_t workspace_bytes, void* stream);

/* The same shard calls with the sum fused into the kernels: instead of writing its summand the
 * call ADDS it, in fp32, into an accumulator that the caller owns, so that shards running on
 * different GPUs can add straight into the memory of the GPU that owns the query rows (a peer
 * mapping of its accumulator) and no separate all-reduce or reduce-scatter pass is needed.
 * bf16 only (dtype 1 returns SIGATTN_ERR_FLAG).
 *
 * sigattn_fwd_shard_acc: o_acc, DEVICE pointer to B*H*N_q*D floats [B, H, N_q, D], 16-byte
 *   aligned, receives += P V of this shard; the forward's epilogue issues vector reductions
 *   (red.global.add) per row, nothing else touches it.  No O is written.
 * sigattn_bwd_shard_acc: dq_acc, DEVICE pointer to B*H*N_q*D floats, 256-byte aligned, receives
 *   += dS K of this shard WITHOUT the factor `scale` (TMA reduce-add tiles, as in sigattn_bwd);
 *   dk, dv of the shard are written as in sigattn_bwd_shard; no dq is written.
 * The accumulators must be zero before the first shard adds (the caller clears them) and all
 * shards must have finished (stream or cross-GPU synchronisation, the caller's) before
 * sigattn_acc_to_bf16 turns them into the result: out = bf16(mul * acc), mul = 1 for O and
 * `scale` for dQ; n = number of elements, a multiple of 4; acc and out 16-byte aligned.
 * Accumulators in another GPU's memory are reached with plain reductions and TMA reduce
 * operations only (no multicast load is ever issued on them).  The order of the additions is
 * not fixed, so the last bits of the sums may differ from run to run. */
SIGATTN_API int sigattn_fwd_shard_acc(const void* q, const void* k, const void* v, float* o_acc,
                          int B, int H, int H_kv, int N_q, int N_k, int D,
                          float scale, float bias, const float* bias_bh, int causal, int pos0,
                          const float* alibi_slopes, int dtype, void* stream);

SIGATTN_API int sigattn_bwd_shard_acc(const void* q, const void* k, const void* v, const void* d_o,
                          float* dq_acc, void* dk, void* dv,
                          int B, int H, int H_kv, int N_q, int N_k, int D,
                          float scale, float bias, const float* bias_bh, int causal, int pos0,
                          const float* alibi_slopes, int dtype,
                          float* dbias_bh, void* stream);

/* sigattn_bwd_shard_acc that also ADDS this call's dK, dV of the shard (bf16 TMA reduce-adds) into
 * `dk`, `dv` instead of writing them: a rank that holds one key/value shard and the query rows of
 * several owners calls it once per owner and finds the sums over the owners in dk, dv, with no
 * arithmetic outside the library.  The caller clears dk and dv before the first call; every call adds
 * one bf16-rounded summand, so the result carries one rounding per owner and its last bits depend on
 * the order in which the tiles arrive. */
SIGATTN_API int sigattn_bwd_shard_acc_kv(const void* q, const void* k, const void* v, const void* d_o,
                             float* dq_acc, void* dk, void* dv,
                             int B, int H, int H_kv, int N_q, int N_k, int D,
                             float scale, float bias, const float* bias_bh, int causal, int pos0,
                             const float* alibi_slopes, int dtype,
                             float* dbias_bh, void* stream);

SIGATTN_API int sigattn_acc_to_bf16(const float* acc, void* out, size_t n, float mul, void* stream);

/* Peer mappings for the accumulating shard calls above (the distributed setting the paper's
 * Limitations, Appendix A, leave open; no counterpart in its algorithms).  One process per GPU:
 * the rank that owns a block of query rows keeps the fp32 accumulators for them in its own device
 * memory, exports them once, and every other rank opens the export and passes the mapped address as
 * `o_acc` / `dq_acc`.  All three calls are host-side set-up, not stream operations.
 *
 * sigattn_peer_export: `dev_ptr` is a device pointer of the calling process (any offset inside a
 *   cudaMalloc'd allocation, e.g. a framework tensor); `handle` is HOST memory of
 *   SIGATTN_PEER_HANDLE_BYTES bytes that receives an opaque handle for the allocation that contains
 *   it, `*offset` the byte offset of dev_ptr inside that allocation.  Both travel to the other
 *   processes by any host channel.  The memory must stay allocated while any process has it open.
 * sigattn_peer_open: in ANOTHER process (CUDA cannot open a handle in the process that made it, nor
 *   twice in one process: keep one export per allocation), with the GPU that will run the shard calls
 *   current: maps the allocation and returns the device address that corresponds to dev_ptr in
 *   `*mapped`.  Peer access between the two GPUs is enabled as a side effect if they differ.
 * sigattn_peer_close: unmaps; `mapped` and `offset` as returned / given to sigattn_peer_open.
 * Ordering is the caller's: the owner clears its accumulators before anyone adds, and converts them
 * (sigattn_acc_to_bf16) only after every rank has finished its adding kernels (each rank synchronises
 * its stream, then all ranks meet at a host barrier).  Errors: SIGATTN_ERR_NULL, SIGATTN_ERR_CUDA. */
#define SIGATTN_PEER_HANDLE_BYTES 64
SIGATTN_API int sigattn_peer_export(const void* dev_ptr, void* handle, size_t* offset);
SIGATTN_API int sigattn_peer_open(const void* handle, size_t offset, void** mapped);
SIGATTN_API int sigattn_peer_close(void* mapped, size_t offset);

/* Padded batches of sequences of different lengths (the speech batches of Section 5.4, with
 * b = -log n_b per sample through `bias_bh`): `seqlens` is a DEVICE pointer to B int32, 4-byte
 * aligned, read while the kernels run; entry b is the number n_b of rows of batch entry b that
 * count (values outside [0, N] are clamped).  Keys j >= n_b get weight 0; query rows i >= n_b
 * give all-zero rows of O and take no part in any gradient (their dq rows are zero, dk and dv
 * do not see them; dk, dv rows >= n_b are zero).  What the padding holds does not matter.  The
 * paper does not print this; it is the usual padding mask and makes the call equal to separate
 * calls on the unpadded sequences.  q, k, v share N.  Other arguments as in sigattn_fwd_gqa /
 * sigattn_bwd_gqa. */
SIGATTN_API int sigattn_fwd_varlen(const void* q, const void* k, const void* v, void* o,
                       int B, int H, int H_kv, int N, int D,
                       float scale, float bias, const float* bias_bh, int causal,
                       const int* seqlens,
                       const float* alibi_slopes, int dtype, void* stream);

SIGATTN_API int sigattn_bwd_varlen(const void* q, const void* k, const void* v, const void* d_o,
                       void* dq, void* dk, void* dv,
                       int B, int H, int H_kv, int N, int D,
                       float scale, float bias, const float* bias_bh, int causal,
                       const int* seqlens,
                       const float* alibi_slopes, int dtype,
                       float* dbias_bh,
                       void* workspace, size_t workspace_bytes, void* stream);

/* The same batches stored WITHOUT padding, one sequence after the other along the row axis:
 * q, o are [1, H, T, D], k, v are [1, H_kv, T, D] with T the sum of the lengths, and
 * `cu_seqlens` is a DEVICE pointer to n_seqs + 1 int32 row offsets 0 = c_0 <= c_1 <= ... <=
 * c_{n_seqs} = T (4-byte aligned, read while the kernels run; the caller guarantees that they
 * rise from 0 to T - they are not checked on the device).  Sequence s owns rows [c_s, c_{s+1});
 * the weight of (query i, key j) is kept only if both rows belong to the same sequence (a
 * block-diagonal mask, times the causal mask if asked for; ALiBi distances are i - j as ever),
 * so the call equals n_seqs separate calls.  Empty sequences are allowed.  `bias_sh` is NULL
 * (scalar `bias`) or a DEVICE pointer to n_seqs * H floats, one bias per (sequence, head), e.g.
 * b = -log n_s; `dbias_sh`, if not NULL, receives the matching n_seqs * H gradients.  Tiles are
 * 128 rows whatever the lengths: a tile that spans several short sequences computes all its
 * 128 x 128 logits and masks the foreign ones, so many sequences much shorter than 128 rows cost
 * as much as 128-row ones.  The workspace is that of sigattn_bwd for (1, H, T, D). */
SIGATTN_API int sigattn_fwd_ragged(const void* q, const void* k, const void* v, void* o,
                       int H, int H_kv, int T, int D,
                       const int* cu_seqlens, int n_seqs,
                       float scale, float bias, const float* bias_sh, int causal,
                       const float* alibi_slopes, int dtype, void* stream);

SIGATTN_API int sigattn_bwd_ragged(const void* q, const void* k, const void* v, const void* d_o,
                       void* dq, void* dk, void* dv,
                       int H, int H_kv, int T, int D,
                       const int* cu_seqlens, int n_seqs,
                       float scale, float bias, const float* bias_sh, int causal,
                       const float* alibi_slopes, int dtype,
                       float* dbias_sh,
                       void* workspace, size_t workspace_bytes, void* stream);

/* The ragged calls read `cu_seqlens` on the device and trust it (offsets that do not rise from 0 to T
 * give wrong results, never out-of-range accesses).  A caller that still holds the offsets on the HOST
 * can have them checked before the launch: `host_cu_seqlens` is a host pointer to n_seqs + 1 int32;
 * returns 0 if they start at 0, never decrease and end at T, SIGATTN_ERR_SHAPE otherwise.  No device
 * work.  No counterpart in the paper. */
SIGATTN_API int sigattn_check_cu_seqlens(const int* host_cu_seqlens, int n_seqs, int T);

/* Sequence-length normalisation (Appendix G, the ablation that compares the bias b = -log n with
 * the scaling n^-alpha sigma(Q K^T / sqrt(d)) V and its causal form, the equation labelled
 * "ar_seq_len_normalization"): O_i = r_i sum_j P_ij V_j with one factor r_i per query row, shared by
 * all batch entries and heads.  The factor does not depend on Q, K, V, so the backward is the plain
 * one with dO_i replaced by r_i dO_i (dV = (r P)^T dO, dS = P (1 - P) (r dP)); db, if asked for,
 * is the sum of that dS.  The bf16 backward forms r_i dO_i in one extra pass (rounded to bf16,
 * held in the dq buffer until dq itself is written at the end of the call).
 *
 * row_scale: DEVICE pointer to N_q floats, 4-byte aligned, read only.  sigattn_seqlen_norm fills
 *   such a vector with the paper's factors: N_k^-alpha for every row without a mask; with the
 *   causal mask (pos_i + 1)^-alpha, pos_i = i + N_k - N_q being the query's position and
 *   pos_i + 1 the number of keys the row keeps (the printed n = 3 example reads 1, 0.5, 0.33 as
 *   bases; its exponent is taken as +alpha on these bases, i.e. -alpha on the counts 1, 2, 3).
 *   Any other vector of factors may be passed as well.
 * Other arguments as in sigattn_fwd_nk / sigattn_bwd_nk (bias_bh and dbias_bh as in
 * sigattn_fwd_gqa / sigattn_bwd_gqa).  Errors as there; row_scale == NULL is SIGATTN_ERR_NULL. */
SIGATTN_API int sigattn_fwd_rowscale(const void* q, const void* k, const void* v, void* o,
                         int B, int H, int H_kv, int N_q, int N_k, int D,
                         float scale, float bias, const float* bias_bh, int causal,
                         const float* row_scale,
                         const float* alibi_slopes, int dtype, void* stream);

SIGATTN_API int sigattn_bwd_rowscale(const void* q, const void* k, const void* v, const void* d_o,
                         void* dq, void* dk, void* dv,
                         int B, int H, int H_kv, int N_q, int N_k, int D,
                         float scale, float bias, const float* bias_bh, int causal,
                         const float* row_scale,
                         const float* alibi_slopes, int dtype,
                         float* dbias_bh,
                         void* workspace, size_t workspace_bytes, void* stream);

/* Writes the paper's N_q factors (see above) to the DEVICE vector row_scale, asynchronously on
 * `stream`.  causal = 1 needs N_k >= N_q. */
SIGATTN_API int sigattn_seqlen_norm(float* row_scale, int N_q, int N_k, float alpha, int causal, void* stream);

/* Forward for generation with a cache of keys and values (where the paper measures its
 * inference gains, Appendix F.3): the same operation, arguments and result as sigattn_fwd_nk,
 * plus a scratch buffer that lets the library split the keys of one head over several thread
 * blocks when B * H_kv alone cannot fill the GPU.  Sigmoid attention has no row normalisation
 * (Section 4), so the partial outputs of the splits are plain fp32 sums - no running maximum, no
 * log-sum-exp to merge; they are added with fp32 atomics (the last bits of O may differ from run
 * to run) and converted to bf16 by a second small kernel.  The split is used when the queries of
 * a key/value head fit one pair of tiles (N_q * H / H_kv <= 256) and it shortens the run; otherwise
 * the call is sigattn_fwd_nk and leaves the workspace untouched.
 * workspace: DEVICE scratch of at least sigattn_fwd_decode_workspace_bytes(...) bytes, 256-byte
 * aligned, owned by the caller; two calls that share it must not overlap on the device.  Errors
 * as sigattn_fwd_nk, plus SIGATTN_ERR_WORKSPACE. */
SIGATTN_API int sigattn_fwd_decode(const void* q, const void* k, const void* v, void* o,
                       int B, int H, int H_kv, int N_q, int N_k, int D,
                       float scale, float bias, const float* bias_bh, int causal,
                       const float* alibi_slopes, int dtype,
                       void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of scratch sigattn_fwd_decode needs: B * H * N_q * D floats (0 for the fp32 debug path
 * and for invalid shapes). */
SIGATTN_API size_t sigattn_fwd_decode_workspace_bytes(int B, int H, int N_q, int D, int dtype);

/* Bytes of scratch sigattn_bwd needs for this problem (0 for the fp32 debug path).
 * Returns 0 for invalid shapes as well; sigattn_bwd reports those. */
SIGATTN_API size_t sigattn_bwd_workspace_bytes(int B, int H, int N, int D, int dtype);

/* One forward + backward pass from HOST buffers (pinned memory recommended): copies
 * q, k, v, d_o (and the H slopes, if any) to the device, runs sigattn_fwd and
 * sigattn_bwd, and copies o, dq, dk, dv back; returns without synchronising.  The work is
 * ordered after everything enqueued on `stream` before the call, and whatever is enqueued
 * on `stream` afterwards is ordered after it.  In between, the problem is cut into chunks
 * of whole heads whose copies in, kernels and copies out run on three streams owned by the
 * library (created on the first call on a device), so that both directions of the host
 * link and the kernels overlap; that overlap needs pinned host buffers.  Every tensor pointer and `alibi_slopes_host` are HOST
 * pointers; `device_arena` is DEVICE scratch of at least
 * sigattn_step_host_arena_bytes(...) bytes, 256-byte aligned, owned by the caller (it
 * holds the eight tensors, the slopes and the backward workspace).  The host buffers must
 * stay valid until the stream has finished.  No counterpart in the paper: this is the
 * end-to-end entry for callers whose data lives in host memory. */
SIGATTN_API int sigattn_step_host(const void* q_host, const void* k_host, const void* v_host, const void* d_o_host,
                      void* o_host, void* dq_host, void* dk_host, void* dv_host,
                      int B, int H, int N, int D,
                      float scale, float bias, int causal,
                      const float* alibi_slopes_host, int dtype,
                      void* device_arena, size_t arena_bytes, void* stream);

/* Bytes of device scratch sigattn_step_host needs (0 for invalid shapes). */
SIGATTN_API size_t sigattn_step_host_arena_bytes(int B, int H, int N, int D, int dtype);

/* Optional timing hook: when both are non-NULL cudaEvent_t handles, every following
 * sigattn_bwd on this thread records `start` right before and `stop` right after its
 * main kernel (excluding the dQ-accumulator clear and the dQ conversion) on the call's
 * stream.  Pass NULL, NULL to switch it off.  Returns 0. */
SIGATTN_API int sigattn_bwd_set_timing_events(void* start_event, void* stop_event);

/* Synchronises `stream`, then returns 0 or SIGATTN_ERR_DEVICE_TIMEOUT if any kernel of
 * this library gave up a bounded wait on the current device since the last check
 * (the flag is cleared), or SIGATTN_ERR_CUDA if the stream reports a CUDA error. */
SIGATTN_API int sigattn_check(void* stream);

/* Self-test of the failure path: launches one small kernel whose only thread group waits,
 * with the same bounded wait the attention kernels use but a limit of `limit_us`
 * microseconds (1 .. 100000), on a barrier that nothing ever signals.  The wait gives up,
 * the kernel ends normally and records the event, so the next sigattn_check(stream) must
 * return SIGATTN_ERR_DEVICE_TIMEOUT while the context stays usable.  Returns 0 if the
 * kernel was enqueued.  No counterpart in the paper. */
SIGATTN_API int sigattn_selftest_bounded_wait(int limit_us, void* stream);

/* Text for an error code (static storage, never NULL). */
SIGATTN_API const char* sigattn_strerror(int code);

/* cudaGetErrorString of the CUDA error behind the last SIGATTN_ERR_CUDA on this thread. */
SIGATTN_API const char* sigattn_last_cuda_error(void);

/* Library version: major * 10000 + minor * 100 + patch. */
SIGATTN_API int sigattn_version(void);

/* Number of kernels of this library launched by this process so far (all threads). */
SIGATTN_API unsigned long long sigattn_launch_count(void);

#ifdef __cplusplus
}
#endif

#endif /* SIGATTN_H_ */
