/*
 * gradcache.h - C ABI of the B200 (sm_100a) library that fills the Representation Gradient
 * Cache of Gradient Cache (arXiv 2101.06983, Section 3.3, "Step 2").
 *
 * Given the numerical representations Q (B x d, row i = f(s_i)) and P (N x d, row j = g(t_j))
 * and the relevance map pos_idx (r_i, Section 3.1), the library computes
 *
 *   S_ij     = <Q_i, P_j> / tau                                   (exponent of Eq. 1)
 *   lse_i    = log sum_{allowed j} exp(S_ij)                      (denominator of Eq. 1 / Eq. 4)
 *   loss     = (1/B) sum_i (lse_i - S_{i, r_i})                   (Eq. 1)
 *   G_ij     = (exp(S_ij - lse_i) - [j == r_i]) / B               (Eq. 4; 0 where masked)
 *   dQ_i     = (1/tau) sum_j G_ij P_j                             (Eq. 5)
 *   dP_j     = (1/tau) sum_i G_ij Q_i                             (Eq. 6-7)
 *
 * dQ and dP together are the cache [u_1..u_B, v_1..v_N] of (B + N) d floats (Section 3.3).
 * The paper fixes tau = 1 and has no mask; for general tau these are the exact derivatives of
 * Eq. 1, and eps_j of Eq. 7 is the sum of f(s_k) over every k with r_k = j.  The B x N matrix
 * S is never written to memory.
 *
 * Conventions shared by all calls
 *   - Every pointer is a DEVICE pointer (including loss and dev_status) unless stated; the
 *     caller owns all buffers, including the workspace.  The library allocates nothing.
 *   - Matrices are row-major with unit stride along d; ldq/ldp/lddq/lddp are leading
 *     dimensions in ELEMENTS.  Q/P rows must start on 16-byte boundaries (base address and
 *     ld * element size multiples of 16), dQ/dP likewise; otherwise GC_ERR_ALIGN.
 *   - Q and P may be the same buffer (symmetric loss); dQ/dP are then the derivatives with
 *     respect to each role and the caller adds them.  Outputs may not alias inputs.
 *   - dtype is the element type of Q and P; all outputs are float, accumulation is float.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t, may be NULL for the default
 *     stream) and return a gc_status for host-detectable errors only.  After a first ordinary
 *     call for the same kernels (it sets kernel attributes and creates the side stream), a call
 *     on a capturing stream can be captured into a CUDA graph and replayed: work on the
 *     library's side stream is forked from and joined back into `cuda_stream`.
 *   - Data-dependent errors are OR-ed into *dev_status (may be NULL) on the device:
 *     GC_DEV_POS_RANGE for pos_idx[i] outside [0, N), GC_DEV_POS_MASKED for pos_idx[i] equal
 *     to the masked column.  Such a row contributes pos_logit = 0 and no one-hot term; nothing
 *     is read out of bounds and nothing traps.  GC_DEV_WAIT_LIMIT means a bounded on-chip wait
 *     gave up; outputs are then undefined.  The caller zeroes *dev_status beforehand.
 *   - Results are deterministic: no floating-point atomics, fixed reduction order.
 *   - Host threads: the library keeps small per-device records (SM count, kernel attributes, one
 *     side stream with its events) that are created on first use without locking.  Make calls
 *     from one host thread at a time.  Calls on different streams of one device are allowed; the
 *     work they put on the side stream is serialised there.
 */
#ifndef GRADCACHE_H_
#define GRADCACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GC_OK = 0,
    GC_ERR_NULL = 1,      /* a required pointer is NULL */
    GC_ERR_SHAPE = 2,     /* B, N or d <= 0, ld < d, tau not finite or <= 0 */
    GC_ERR_DTYPE = 3,     /* unknown dtype */
    GC_ERR_MASK = 4,      /* unknown mask mode, or GC_MASK_SELF with N < 2 */
    GC_ERR_ALIGN = 5,     /* a row does not start on a 16-byte boundary */
    GC_ERR_WORKSPACE = 6, /* workspace NULL, misaligned (256 bytes) or too small */
    GC_ERR_CUDA = 7,      /* a CUDA call or launch failed */
    GC_ERR_ARCH = 8,      /* the current device is not compute capability 10.x */
    GC_ERR_LIMIT = 9      /* problem exceeds a built-in limit of the entry point that was called */
} gc_status;

typedef enum { GC_F32 = 0, GC_BF16 = 1 } gc_dtype;
typedef enum { GC_MASK_NONE = 0, GC_MASK_SELF = 1 } gc_mask; /* SELF: drop the pair (i, i) */
typedef enum { GC_OP_FWD = 0, GC_OP_BWD = 1, GC_OP_BUILD = 2, GC_OP_BUILD_STORED = 3 } gc_op;

enum { GC_DEV_POS_RANGE = 1, GC_DEV_POS_MASKED = 2, GC_DEV_WAIT_LIMIT = 4 };

/* Bytes of workspace the given call needs for these sizes on the current device (a multiple
 * of 256).  O((B + N) d), never O(B N), for the three calls of the paper's path;
 * GC_OP_BUILD_STORED adds 2 B N bytes for its weight matrix.  Returns 0 for invalid arguments. */
size_t gc_workspace_bytes(int op, int64_t B, int64_t N, int d, int dtype);

/* Name of the kernel plan the library will use for these sizes:
 *   "tcgen05-one-tile"  one launch for a batch of one tile: B <= 128, N <= 256 (bf16) or N <= 128
 *                       (fp32, on the tensor cores as three bf16 terms), d a multiple of 8 up to 1024
 *   "tcgen05-tiles"     fp32 batches of tile pairs of 128 x 128 whose planes of partial sums,
 *                       4 d (B ceil(N/128) + N ceil(B/128)) bytes of workspace, stay within 2 GiB,
 *                       and bf16 batches of tile pairs of 128 x 256 that make at most two waves of
 *                       CTAs (d a multiple of 8 up to 4096): the same kernel per tile pair, then
 *                       combine and reduce kernels
 *   "tcgen05"           TMA + tcgen05 MMA sweeps with TMEM accumulators; bf16, d a multiple of 64
 *                       up to 4096; one CTA, a CTA pair or a cluster of four per tile, by shape
 *   "simt"              fp32 FMA tiles: every other case (other widths, fp32 batches beyond that)
 * "invalid" for an unknown op, non-positive sizes, or a problem GC_OP_BUILD_STORED refuses.
 * Static string.  With GRADCACHE_PLAN=sweeps in the environment (read at every call; a
 * diagnostic switch) the first two plans are not chosen. */
const char* gc_plan_name(int op, int64_t B, int64_t N, int d, int dtype);

/* Number of kernels one call launches for these sizes (for launch accounting). */
int gc_kernel_launches(int op, int64_t B, int64_t N, int d, int dtype);

/*
 * Forward: Eq. 1.  Writes loss[1], row_lse[B] (natural log) and, if non-NULL, pos_logit[B]
 * (S_{i, r_i}).  An online row maximum / sum runs over passage tiles (Section 3.2, Eq. 4's
 * denominator); the positive logit is picked out of the tile that holds column r_i.
 */
int gc_loss_fwd(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                float* loss, float* row_lse, float* pos_logit,
                void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);

/*
 * Backward: Eq. 5-7 given row_lse[B] from the forward.  Overwrites dQ[B x d] and dP[N x d]
 * (either may be NULL to skip it).  S tiles are recomputed; G is formed in registers.
 */
int gc_loss_bwd(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                const float* row_lse, float* dQ, int64_t lddq, float* dP, int64_t lddp,
                void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);

/*
 * Step 2 of Section 3.3 in one call: loss, row_lse, (pos_logit) and the cache dQ, dP.  Nothing of
 * size B x N is written to global memory.  For bf16 rows (d a multiple of 64) the forward runs
 * inside the dQ sweep; where each row's weights are scaled by its positive logit, the anchor
 * kernel that computes those logits and the sweep overlap (programmatic dependent launch).  Part of the work may be queued on a stream the library owns, between a fork from
 * and a join back into `cuda_stream`: the call is asynchronous on `cuda_stream` alone, but the
 * first such call on a device creates that stream and belongs outside any stream capture.
 */
int gc_build_cache(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                   int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                   float* loss, float* row_lse, float* pos_logit,
                   float* dQ, int64_t lddq, float* dP, int64_t lddp,
                   void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);

/*
 * The same results as gc_build_cache by a different route, kept as a measured comparison point:
 * Eq. 1 and Eq. 5-7 need every logit three times (loss, dQ, dP), and gc_build_cache recomputes
 * them so that nothing of size B x N ever leaves the chip.  This call trades memory for work: one
 * forward sweep writes the un-normalised bf16 softmax weights 2^((S_ij - S_{i,r_i}) log2 e) of
 * all pairs to the workspace (2 B N bytes; 0 at masked pairs and at the positive column, whose
 * terms are added in fp32), and two plain GEMMs over that matrix form dQ and dP.  Rows whose
 * logits lie more than 100 powers of two above their positive logit cannot be stored this way; a
 * device flag then hands the whole call to the recomputing kernels, which are always launched
 * after the GEMMs and return at once when the flag is down.  bf16 inputs with d a multiple of 64
 * only, and a weight matrix of at most 40 GiB: other problems are refused with GC_ERR_LIMIT.
 * Workspace size: gc_workspace_bytes(GC_OP_BUILD_STORED, ...).
 */
int gc_build_cache_stored(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                          const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                          int mask_mode, int dtype, float* loss, float* row_lse, float* pos_logit,
                          float* dQ, int64_t lddq, float* dP, int64_t lddp,
                          void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);

/*
 * Step 3 of Section 3.3 (Eq. 8 for f, Eq. 9 for g) for a linear encoder f(s) = W s: the cached
 * representation gradients u_i of one sub-batch are propagated to the encoder matrix,
 *
 *     dW[a][b] (+)= sum_i U[i][a] * X[i][b],     a < d, b < d_in,
 *
 * the term d f(s_i)/dW applied to u_i being the outer product u_i s_i^T.  Summed over the
 * sub-batches this is the full-batch gradient dL/dW (the equality the paper states after Eq. 9).
 *   U      [rows x d] float, leading dimension ldu: a row range of dQ (or dP) as gc_build_cache
 *          wrote it; pass the pointer to its first row.
 *   X      [rows x d_in] bf16 (x_dtype = GC_BF16; anything else is GC_ERR_DTYPE), leading
 *          dimension ldx: the encoder inputs s_i of the same rows.
 *   dW     [d x d_in] float, leading dimension lddw.  accumulate == 0 overwrites it (first
 *          sub-batch), otherwise the sub-batch's sum is added to it (outer sum of Eq. 8).
 * Each u is used as the sum of two bf16 terms (its rounding and the rounding of the remainder,
 * together exact to 2^-17 |u|), products are exact and accumulation is fp32 on the tensor cores.
 * Limits: d a multiple of 8, d_in a multiple of 64 and at most 4096 (else GC_ERR_LIMIT); rows of
 * U, X and dW start on 16-byte boundaries.  One kernel launch; the partial sums over parts of the
 * sub-batch are exchanged through shared memory, so the workspace is nominal:
 * gc_cache_apply_workspace_bytes returns 256 (0 for sizes outside the limits) and ws must be a
 * 256-byte aligned, caller-owned buffer of at least that size.  Asynchronous on cuda_stream;
 * deterministic; GC_DEV_WAIT_LIMIT in *dev_status (may be NULL) as for the other calls.
 */
size_t gc_cache_apply_workspace_bytes(int64_t rows, int d, int d_in);
int gc_cache_apply(const float* U, int64_t ldu, const void* X, int64_t ldx, int64_t rows, int d,
                   int d_in, int x_dtype, float* dW, int64_t lddw, int accumulate,
                   void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);

/*
 * Section 3.4 (multi-GPU training): after the all-gather every GPU holds all representations,
 * the loss is defined over all of them, and each rank forms the gradients of its own
 * representations only.  These two calls are that rank-local part of Step 2 for a rank that owns
 * query rows [q0, q0 + q_count) and passage rows [p0, p0 + p_count) of the gathered Q [B x d] and
 * P [N x d] (pos_idx [B] indexes rows of the gathered P).  Unlike the paper's scheme a rank does
 * not redo the whole forward: it needs lse_i of its own queries for dQ and, for dP, lse_i of all
 * queries, which the ranks exchange between the two calls (B floats).
 *
 *   gc_shard_fwd_dq  forward (Eq. 1) and dQ (Eq. 5) of the local queries against all passages.
 *       Writes row_lse[q0 .. q0 + q_count) (row_lse and pos_logit point at entry 0 of arrays of
 *       length B), dQ [q_count x d], and *loss_part = (1/B) sum over the local queries of
 *       (lse_i - S_{i,r_i}): the loss of Eq. 1 is the sum of loss_part over the ranks.
 *   gc_shard_dp      dP (Eq. 6-7) of the local passages against all queries, given row_lse of
 *       ALL B queries.  Writes dP [p_count x d].
 *
 * Both scale by 1/B with B the whole batch, so concatenating the ranks' dQ and dP gives exactly
 * what gc_build_cache gives on one GPU (up to rounding order).  GC_MASK_SELF drops the pair of
 * query i and passage i of the WHOLE batch, wherever the rank's rows lie in it; a range outside the
 * matrices is GC_ERR_SHAPE.  Workspace:
 * gc_shard_workspace_bytes, which covers either call.  The collectives are the caller's (the
 * Python package's `sharded` module runs them with torch.distributed).
 */
size_t gc_shard_workspace_bytes(int64_t B, int64_t N, int d, int dtype, int64_t q_count,
                                int64_t p_count);
int gc_shard_fwd_dq(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                    int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                    int64_t q0, int64_t q_count, float* loss_part, float* row_lse,
                    float* pos_logit, float* dQ, int64_t lddq,
                    void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);
int gc_shard_dp(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                const float* row_lse, int64_t p0, int64_t p_count, float* dP, int64_t lddp,
                void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream);

/*
 * Loss variants (Section 3.3, Step 2: the loss computed on the stored representations may vary,
 * and the paper leaves its derivative to automatic differentiation; these calls supply the two
 * derivatives that need no change to the sweeps).
 *
 * Cosine similarity, S_ij = <q_i/|q_i|, p_j/|p_j|> / tau:
 *   gc_row_normalize  Xn[i] = X[i] / |X[i]| in the dtype of X (bf16: round to nearest even) and
 *                     inv_norm[i] = 1/|X[i]| (float; the norm is accumulated in fp32; a zero row
 *                     stays zero with inv_norm 0).  Call it on Q and on P, run gc_build_cache (or
 *                     gc_loss_fwd / gc_loss_bwd) on the unit rows, then
 *   gc_cosine_bwd     dX[i] = inv_norm[i] (dXn[i] - n_i <n_i, dXn[i]>), n_i = inv_norm[i] X[i] in
 *                     fp32: the Jacobian (I - n n^T)/|x| of the normalisation applied to the cache
 *                     rows dXn (dQ or dP of the unit rows).  dX may be the same buffer as dXn.
 * Learnable temperature:
 *   gc_dtau           *dtau = dL/dtau = -(1/tau) sum_i <Q_i, dQ_i>, with Q the rows the sweeps saw
 *                     and dQ their cache rows (Eq. 5 gives <Q_i, dQ_i> = sum_j G_ij S_ij).  Rows
 *                     are summed in a fixed order.  Workspace: gc_dtau_workspace_bytes(B).
 * X, Xn, Q: [rows x d] of dtype (GC_F32 or GC_BF16), leading dimensions in elements, rows on
 * 16-byte boundaries, d a multiple of 8 (else GC_ERR_LIMIT); dXn, dX, dQ float.  Device pointers,
 * asynchronous on cuda_stream, deterministic.
 */
int gc_row_normalize(const void* X, int64_t ldx, int64_t rows, int d, int dtype, void* Xn,
                     int64_t ldxn, float* inv_norm, void* cuda_stream);
int gc_cosine_bwd(const void* X, int64_t ldx, int64_t rows, int d, int dtype, const float* inv_norm,
                  const float* dXn, int64_t lddxn, float* dX, int64_t lddx, void* cuda_stream);
size_t gc_dtau_workspace_bytes(int64_t B);
int gc_dtau(const void* Q, int64_t ldq, const float* dQ, int64_t lddq, int64_t B, int d, float tau,
            int dtype, float* dtau, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Two more loss variants of Section 3.3, Step 2, each one call that runs gc_build_cache and adds
 * what differs from Eq. 1 in fp32 (device pointers, asynchronous on cuda_stream, deterministic:
 * sums into rows of dP that several queries point at are formed in ascending query order).
 *
 *   gc_build_cache_multi_pos   several positives per query, given as a CSR list: query i has the
 *       positives pos_list[pos_ptr[i] .. pos_ptr[i + 1]) (int32, pos_ptr of length B + 1, n_pos =
 *       pos_ptr[B] entries in all, at least one per query, distinct within a query).  Loss of
 *       query i = mean over its positives of -log p_ir, so G_ij = (p_ij - [j in R_i]/|R_i|)/B;
 *       one positive per query is gc_build_cache.  An empty or out-of-range list sets
 *       GC_DEV_POS_RANGE, a positive on the masked diagonal GC_DEV_POS_MASKED.
 *   gc_build_cache_two_direction   L = (L_row + L_col)/2 with L_row = Eq. 1 and L_col its mirror
 *       image over the same B positive pairs: passage r_i is the anchor and the B queries are its
 *       candidates, L_col = (1/B) sum_i (log sum_i' exp(S_{i' r_i}) - S_{i r_i}).  N may exceed B.
 *       No mask (GC_MASK_NONE).  row_lse receives the row direction's logsumexp.
 * Q, P, dQ, dP, loss, row_lse, tau, dtype as in gc_build_cache; d a multiple of 8 (else
 * GC_ERR_LIMIT).  Workspace: gc_multi_pos_workspace_bytes / gc_two_direction_workspace_bytes
 * (0 for invalid arguments), 256-byte aligned, caller-owned.
 */
size_t gc_multi_pos_workspace_bytes(int64_t B, int64_t N, int d, int dtype, int64_t n_pos);
int gc_build_cache_multi_pos(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                             const int32_t* pos_ptr, const int32_t* pos_list, int64_t n_pos,
                             int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                             float* loss, float* row_lse, float* dQ, int64_t lddq, float* dP,
                             int64_t lddp, void* ws, size_t ws_bytes, int* dev_status,
                             void* cuda_stream);
size_t gc_two_direction_workspace_bytes(int64_t B, int64_t N, int d, int dtype);
int gc_build_cache_two_direction(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                                 const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                                 int dtype, float* loss, float* row_lse, float* dQ, int64_t lddq,
                                 float* dP, int64_t lddp, void* ws, size_t ws_bytes,
                                 int* dev_status, void* cuda_stream);

/*
 * Distance Gradient Cache (Section 5, Eq. 10-13) in tiled form.  The similarity of pair (i, j) is
 * a distance d_ij = Phi(f(s_i), g(t_j)) computed by the caller's network; the loss is Eq. 1 with
 * d_ij / tau as the logit.  The paper stores all B x N values w_ij = dL/dd_ij.  Here the caller
 * walks its sub-batch pairs twice and hands over one block of distances at a time, so nothing of
 * size B x N is kept:
 *   gc_dist_begin       resets the per-row state run_m, run_l, pos_d (float [B] each, caller-owned)
 *   gc_dist_accumulate  folds D_block [bq x bn] (float, leading dimension ldd; rows i0.., columns
 *                       j0.. of the full matrix) into the running maximum and sum of its rows and
 *                       records d_{i,r_i}/tau where column r_i lies in the block.  Blocks of the
 *                       same rows must be accumulated one after the other (stream order does).
 *   gc_dist_finish      row_lse[i] = log sum_j exp(d_ij / tau) over the allowed pairs, loss = Eq. 1;
 *                       pos_idx errors go to *dev_status as in gc_loss_fwd
 *   gc_dist_w_block     W_block[r][c] = w_ij = (exp(d_ij / tau - lse_i) - [j == r_i]) / (B tau), 0
 *                       at the masked pair: the block of the Distance Gradient Cache that Eq. 11
 *                       (dL/dOmega = sum w_ij dPhi_ij/dOmega) and Eq. 12-13 (u_i = sum_j w_ij
 *                       dd_ij/df(s_i), v_j likewise) consume for this sub-batch pair
 *   gc_dist_dot_block   D_block[r][c] = <Q[i0 + r], P[j0 + c]> for the dot-product distance (then
 *                       Eq. 12-13 reduce to Eq. 5-7: u = W P, v = W^T Q); Q, P as in gc_loss_fwd,
 *                       d a multiple of 8 (else GC_ERR_LIMIT)
 * A block outside the B x N matrix is GC_ERR_SHAPE.  Device pointers, asynchronous on cuda_stream,
 * deterministic (fixed reduction order); fp32 arithmetic.
 */
int gc_dist_begin(float* run_m, float* run_l, float* pos_d, int64_t B, void* cuda_stream);
int gc_dist_accumulate(const float* D_block, int64_t ldd, int64_t i0, int64_t bq, int64_t j0,
                       int64_t bn, const int32_t* pos_idx, int64_t B, int64_t N, float tau,
                       int mask_mode, float* run_m, float* run_l, float* pos_d, void* cuda_stream);
int gc_dist_finish(const float* run_m, const float* run_l, const float* pos_d,
                   const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode, float* row_lse,
                   float* loss, int* dev_status, void* cuda_stream);
int gc_dist_w_block(const float* D_block, int64_t ldd, int64_t i0, int64_t bq, int64_t j0,
                    int64_t bn, const int32_t* pos_idx, const float* row_lse, int64_t B, int64_t N,
                    float tau, int mask_mode, float* W_block, int64_t ldw, void* cuda_stream);
int gc_dist_dot_block(const void* Q, int64_t ldq, const void* P, int64_t ldp, int64_t B, int64_t N,
                      int d, int dtype, int64_t i0, int64_t bq, int64_t j0, int64_t bn,
                      float* D_block, int64_t ldd, void* cuda_stream);

/*
 * Forward with library-owned scratch (no counterpart in the paper: it exists for the sake of
 * callers, not of the method).  Same inputs, outputs and results as gc_loss_fwd, but the caller
 * passes no workspace.  It is meant for callers that cannot obtain device memory at the point of
 * the call: code running under a host framework that owns every byte of the device through its
 * own pool and offers no allocation hook to a C library, and loops on a hot path where an
 * allocator call is unwelcome because it may synchronise the whole device or fail late.  The
 * call itself allocates nothing and frees nothing, on the device or through any library.
 *
 * The scratch (per-part row maxima, row sums and the gathered positive logits) lives in a
 * fixed array of GC_STATIC_SCRATCH_BYTES inside the library image, so every GPU that loads the
 * library carries that much extra memory until the process exits.  Problems whose forward
 * scratch (gc_static_scratch_need: the slots the forward sweep itself writes, not the larger
 * workspace of the other calls) exceeds it are refused with GC_ERR_LIMIT and nothing is
 * launched.  The first call on each device looks up the array's device address (once, with that
 * device current); make that first call outside any stream capture.  All calls on a device
 * share the one array, and it keeps whatever the previous call left: the kernels overwrite
 * every entry they later read, so nothing has to be cleared, but two calls that overlap on the
 * GPU (different streams, no ordering between them) would race on it.  Serialise them.
 */
#define GC_STATIC_SCRATCH_BYTES (2u << 20)
size_t gc_static_scratch_need(int64_t B, int64_t N, int d, int dtype);
int gc_loss_fwd_static(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                       const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                       int mask_mode, int dtype, float* loss, float* row_lse, float* pos_logit,
                       int* dev_status, void* cuda_stream);

/*
 * Measurement aid (not part of the paper's method).  After gc_profile_enable(sets) with sets >= 1
 * every call brackets its three main kernels - the forward sweep, the dQ sweep (Eq. 5) and the
 * dP sweep (Eq. 6-7) - with CUDA events recorded on the call's own stream; gc_profile_enable(0)
 * switches it off.  Call number c since the enable (0, 1, ...) uses event set c % sets, so up to
 * `sets` calls (at most 256, else GC_ERR_LIMIT) can be queued back to back and read afterwards:
 * gc_profile_read_call(c, ...) waits for that call's events and returns each kernel's duration
 * in milliseconds (0 for a kernel the call did not launch; GC_ERR_LIMIT when call c was never
 * made or its set has been reused); gc_profile_read does the same for the most recent call.
 * Host pointers.  One series of event sets per process: use it for single-stream measurement
 * runs only.  While it is on, the event between the anchor kernel and the fused sweep keeps
 * the sweep from starting early (see gc_build_cache).
 */
int gc_profile_enable(int sets);
int gc_profile_read(float* ms_fwd, float* ms_dq, float* ms_dp);
int gc_profile_read_call(int64_t call, float* ms_fwd, float* ms_dq, float* ms_dp);

/*
 * Test aid (no counterpart in the paper).  Every wait a tensor-core kernel of this library makes
 * on an on-chip barrier is bounded: when the limit passes, the CTA stops waiting, ORs
 * GC_DEV_WAIT_LIMIT into *dev_status and returns, and the context stays usable.  This call
 * launches one small CTA that runs that same wait helper, with a limit of limit_ns nanoseconds
 * (1 .. 1e8, else GC_ERR_LIMIT), on a barrier that nothing arrives on, so that the give-up path
 * can be observed without any fault: afterwards *dev_status has GC_DEV_WAIT_LIMIT set and
 * *waited_ns (device pointer, may be NULL) holds how long the wait lasted.  Asynchronous on
 * cuda_stream.
 */
int gc_selftest_wait_limit(uint64_t limit_ns, int* dev_status, unsigned long long* waited_ns,
                           void* cuda_stream);

/* Human-readable name of a gc_status value.  Static string. */
const char* gc_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* GRADCACHE_H_ */
