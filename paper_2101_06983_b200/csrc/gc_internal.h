// Internal declarations shared by the translation units of libgradcache (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "gradcache.h"

namespace gc {

// A kernel launched with a gate returns at once unless (*flag != 0) == (want != 0); with
// flag == NULL it always runs.  The flag is written by an earlier kernel of the same call.
struct Gate {
    const int* flag;
    int want;
};
#ifdef __CUDACC__
// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute
// may start while the kernel before it in the stream still runs; dep_wait() returns once that
// kernel has completed and its writes are visible (at once for an ordinary launch);
// dep_release() in the earlier kernel lets the later one be scheduled early.
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_release() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ bool gate_closed(const Gate& g) {
    return g.flag && ((*g.flag != 0) != (g.want != 0));
}
// Logsumexp of row i from its per-part (scale, sum) slots, slot g at [g * pitch + i]: the one
// definition every kernel that merges slots uses, with explicit roundings so that all of them
// get the same bits.
__device__ __forceinline__ float combined_lse(const float* __restrict__ part_m,
                                              const float* __restrict__ part_l, int slots,
                                              int64_t pitch, int64_t i) {
    float m = -INFINITY;
    for (int g = 0; g < slots; ++g) m = fmaxf(m, part_m[(int64_t)g * pitch + i]);
    float l = 0.f;
    for (int g = 0; g < slots; ++g) {
        const float mg = part_m[(int64_t)g * pitch + i];
        if (mg > -INFINITY) l = __fmaf_rn(part_l[(int64_t)g * pitch + i], expf(mg - m), l);
    }
    return __fadd_rn(m, logf(l));
}
#endif

// One problem instance as the entry points receive it.
struct Problem {
    const void* Q;
    const void* P;
    const int32_t* pos_idx;
    int64_t ldq, ldp;
    int64_t B, N;
    int d;
    float tau;
    int mask_mode;
    int dtype;
    int64_t b_total;        // rows of the whole batch when Q holds a slice of it (0: B): the mean
                            // of Eq. 1 and the 1/B of Eq. 4 run over this many queries
    int64_t mask_shift;     // GC_MASK_SELF drops the pair (query i, passage j) with j == i +
                            // mask_shift: 0 for whole matrices, first query row minus first
                            // passage row (in the whole batch) when Q or P is a slice
};

// The two tile sweeps share one shape: a stationary row tile X, a streamed row tile Y,
// S_xy = <X_x, Y_y> / tau, a weight W_xy derived from S, and acc_x += sum_y W_xy Y_y.
//   SWEEP_DQ: x = query i,   y = passage j, W = exp(S - lse[x]) - [y == pos[x]]   (Eq. 5)
//   SWEEP_DP: x = passage j, y = query i,   W = exp(S - lse[y]) - [x == pos[y]]   (Eq. 6-7)
// In both, W = 0 for the masked pair (query index == passage index under GC_MASK_SELF).
enum SweepMode { SWEEP_DQ = 0, SWEEP_DP = 1 };

struct SweepArgs {
    const void* X;          // stationary rows  [nx x d]
    const void* Y;          // streamed rows    [ny x d]
    int64_t ldx, ldy;
    int64_t nx, ny;
    int d;
    int mode;               // SweepMode
    int mask_mode;
    int64_t mask_delta;     // masked pair: y == x + mask_delta (+mask_shift for x = query, - for x = passage)
    int dtype;
    float inv_tau;
    float out_scale;        // 1 / (B * tau), applied where the final value is written
    const float* row_lse;   // [B], indexed by the query index
    const int32_t* pos_idx; // [B], indexed by the query index
    float* out;             // [nx x d] final output (used when groups == 1)
    int64_t ldo;
    float* partial;         // [groups x nx x d] unscaled partial sums (used when groups > 1)
    int groups;             // the y range is split into this many contiguous parts
    int* dev_status;        // may be NULL
    Gate gate;
    // SWEEP_DP of the tensor-core kernels only: when slot_l is set, row_lse is not read; the
    // logsumexp of each streamed query is merged from these forward slots ([slots][ny]) instead.
    const float* slot_m;
    const float* slot_l;
    int slots;
};

struct FwdArgs {
    Problem p;
    float* part_m;          // [groups x B] running maximum of each part
    float* part_l;          // [groups x B] sum of exp(S - m) of each part
    float* pos_logit;       // [B] written only by the owner of column pos_idx[i]
    float* red;             // scratch of the loss reduction that follows; the sweep clears its
                            // first word (the block ticket)
    int groups;
    int* dev_status;        // may be NULL
    Gate gate;
};

// How one call is carried out for given sizes on the current device.
struct Plan {
    int tc;                 // 1: tcgen05 kernels, 0: SIMT kernels
    int tiles;              // 1: batch of a few tiles on the one-tile tcgen05 kernel
    int tiles_y;            // its passage tiles (slots per row of its forward)
    int g_fwd, g_dq, g_dp;  // split factors of the streamed range
    size_t off_m, off_l, off_pos, off_red, off_accq, off_accp;
    size_t total;           // workspace bytes (multiple of 256)
    int launches_fwd, launches_bwd;
    int fused;              // 1: gc_build_cache runs the forward inside the dQ sweep
    int anchored;           // 1: ... with the positive logit as the fixed scale of each row (four-
                            // CTA sweep); the online-maximum sweep then is its gated fallback
    int launches_build;
    // Stored-weights plan of gc_build_cache (tcgen05 only): one forward sweep keeps the bf16
    // weights, two GEMMs form the gradients; the sweeps above stay as its fallback.
    int mat;
    int g_mq, g_mp;         // split factors of the two GEMMs' contraction ranges
    int64_t ldw;            // row pitch of the stored weights, elements
    size_t off_ref, off_flag, off_qs, off_w;
};

int sm_count();
Plan make_plan(int64_t B, int64_t N, int d, int dtype, bool stored = false);

// gc_combine.cu
cudaError_t launch_lse_combine(const float* part_m, const float* part_l, const float* pos_ws,
                               const int32_t* pos_idx, int groups, int64_t B, int64_t N,
                               int mask_mode, float* row_lse, float* pos_logit, float* loss,
                               float* red, int* dev_status, Gate gate, cudaStream_t st,
                               int64_t mean_over = 0, int64_t mask_shift = 0);
cudaError_t launch_shift_pos(const int32_t* pos_idx, int64_t B, int64_t first, int64_t count,
                             int32_t* out, cudaStream_t st);
cudaError_t launch_pos_check(const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode,
                             int* dev_status, cudaStream_t st, int64_t mask_shift = 0);
cudaError_t launch_fused_dq_finalize(const float* partial, int groups, const float* part_m,
                                     const float* row_ref2, const float* row_lse,
                                     const float* pos_ws, const int32_t* pos_idx, const void* P,
                                     int64_t ldp, int64_t B, int64_t N, int d, int mask_mode,
                                     float scale, float* out, int64_t ldo, Gate gate,
                                     cudaStream_t st, int64_t mask_shift = 0);
cudaError_t launch_partial_reduce(const float* partial, int groups, int64_t rows, int d,
                                  float scale, float* out, int64_t ldo, Gate gate,
                                  cudaStream_t st);
cudaError_t launch_pos_anchor(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                              const int32_t* pos_idx, int64_t B, int64_t N, int d, int mask_mode,
                              float c1, float* ref2, int* range_flag, cudaStream_t st,
                              int64_t mask_shift = 0);
cudaError_t launch_scale_rows(const void* Q, int64_t ldq, int64_t B, int d, const float* ref2,
                              const float* row_lse, void* Qs, cudaStream_t st);
cudaError_t launch_dp_positive(const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode,
                               const float* pos_ws, const float* row_lse, const void* Q,
                               int64_t ldq, int d, float scale, float* out, int64_t ldo,
                               cudaStream_t st, int64_t mask_shift = 0);

// gc_simt.cu
cudaError_t simt_launch_fwd(const FwdArgs& a, cudaStream_t st);
cudaError_t simt_launch_sweep(const SweepArgs& a, cudaStream_t st);
int simt_fwd_groups(int64_t B, int64_t N);
int simt_sweep_groups(int64_t nx, int64_t ny, int d);

// gc_tc.cu
bool tc_supported(int64_t B, int64_t N, int d, int dtype);
cudaError_t tc_launch_fwd(const FwdArgs& a, cudaStream_t st);
cudaError_t tc_launch_sweep(const SweepArgs& a, cudaStream_t st);
int tc_fwd_groups(int64_t B, int64_t N, int d);
bool tc_fused_applicable(int d);
bool tc_anchor_applicable(int d);
cudaError_t tc_launch_anchored_dq(const FwdArgs& a, float* partial, int groups,
                                  const float* row_ref, int* range_flag, cudaStream_t st,
                                  bool overlap_prev = false);
cudaError_t tc_launch_fused_dq(const FwdArgs& a, float* partial, int groups, cudaStream_t st);
int tc_sweep_groups(int64_t nx, int64_t ny, int d);
cudaError_t tc_launch_fwd_store(const FwdArgs& a, void* weights, int64_t ldw, const float* row_ref,
                                int* range_flag, cudaStream_t st);

// gc_quad.cu
bool quad_applicable(int64_t nx, int d);
// gc_narrow.cu: the gradient sweeps of rows of 64 or 128 bf16 values
bool narrow_applicable(int d, int dtype);
cudaError_t narrow_launch_anchored_dq(const FwdArgs& a, float* partial, int groups,
                                      const float* row_ref, int* range_flag, cudaStream_t st,
                                      bool overlap_prev);
cudaError_t narrow_launch_sweep(const SweepArgs& a, cudaStream_t st);
int quad_groups(int64_t nx, int64_t ny);
cudaError_t quad_launch_sweep(const SweepArgs& a, cudaStream_t st);
cudaError_t quad_launch_fused_dq(const FwdArgs& a, float* partial, int groups, const float* row_ref,
                                 int* range_flag, cudaStream_t st, bool overlap_prev = false);

// gc_small.cu
bool small_applicable(int64_t B, int64_t N, int d, int dtype);
cudaError_t launch_small(int op, const Problem& pr, const float* row_lse_in, float* loss,
                         float* row_lse, float* pos_logit, float* dQ, int64_t lddq, float* dP,
                         int64_t lddp, int* dev_status, cudaStream_t st);

bool small_tiled_applicable(int64_t B, int64_t N, int d, int dtype);
int small_tiles_x(int64_t B);
int small_tiles_y(int64_t N, int dtype);
cudaError_t launch_small_tiled_fwd(const Problem& pr, float* part_m, float* part_l, float* pos_ws,
                                   float* red, int* dev_status, cudaStream_t st);
cudaError_t launch_small_tiled_bwd(const Problem& pr, const float* row_lse, float* dQ, int64_t lddq,
                                   float* partial_q, float* dP, int64_t lddp, float* partial_p,
                                   int* dev_status, cudaStream_t st);

// gc_gemm.cu
int gemm_groups(int64_t m_rows, int64_t k_len, int d);
cudaError_t launch_weight_gemm(const void* weights, int64_t ldw, int64_t B, int64_t N, int transpose,
                               const void* V, int64_t ldv, int d, int groups, float out_scale,
                               float* out, int64_t ldo, float* partial, int* dev_status,
                               cudaStream_t st);

}  // namespace gc
