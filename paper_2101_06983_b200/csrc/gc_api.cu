// C-ABI entry points: argument validation, plan selection, workspace carve-up and the launch
// sequence of each call.  Every numerical step runs in the kernels of the other files.
#include <math.h>

#include "gc_internal.h"

namespace gc {

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return 148;
    }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            n <= 0) {
            cudaGetLastError();
            n = 148;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Largest weight matrix gc_build_cache will ask the workspace to hold.
constexpr size_t kMaxStoredWeightBytes = (size_t)40 << 30;

Plan make_plan(int64_t B, int64_t N, int d, int dtype, bool stored) {
    Plan pl{};
    pl.tc = tc_supported(B, N, d, dtype) ? 1 : 0;
    if (pl.tc) {
        pl.g_fwd = tc_fwd_groups(B, N, d);
        pl.g_dq = tc_sweep_groups(B, N, d);
        pl.g_dp = tc_sweep_groups(N, B, d);
    } else {
        pl.g_fwd = simt_fwd_groups(B, N);
        pl.g_dq = simt_sweep_groups(B, N, d);
        pl.g_dp = simt_sweep_groups(N, B, d);
    }
    // fp32 batches of a few tiles: the one-tile tcgen05 kernel per tile pair (gc_small.cu); its
    // slots and partial planes share the regions of the plan it replaces
    pl.tiles = small_tiled_applicable(B, N, d, dtype) ? 1 : 0;
    pl.tiles_y = pl.tiles ? small_tiles_y(N, dtype) : 0;
    const int tiles_x = pl.tiles ? small_tiles_x(B) : 0, tiles_y = pl.tiles ? small_tiles_y(N, dtype) : 0;
    pl.fused = (pl.tc && tc_fused_applicable(d)) ? 1 : 0;
    // 1: four-CTA sweeps (rows of two column halves); 2: narrow rows (two S buffers)
    pl.anchored = (pl.fused && quad_applicable(B, d)) ? 1
                  : (pl.tc && !pl.fused && tc_anchor_applicable(d)) ? 2 : 0;
    size_t dpad = (size_t)((d + 3) & ~3);
    // (max, sum) slots: the forward sweep writes g_fwd of them per row, the fused sweep 2 g_dq,
    // the anchored fused sweep 4 g_dq
    size_t slots = (size_t)pl.g_fwd;
    if (pl.fused && (size_t)(2 * pl.g_dq) > slots) slots = (size_t)(2 * pl.g_dq);
    if (pl.anchored == 1 && (size_t)(4 * pl.g_dq) > slots) slots = (size_t)(4 * pl.g_dq);
    if (pl.anchored == 2 && (size_t)(4 * pl.g_dq) > slots) slots = (size_t)(4 * pl.g_dq);
    if ((size_t)tiles_y > slots) slots = (size_t)tiles_y;
    const int planes_q = pl.g_dq > tiles_y ? pl.g_dq : tiles_y;
    const int planes_p = pl.g_dp > tiles_x ? pl.g_dp : tiles_x;
    size_t off = 0;
    pl.off_m = off;    off += align256(sizeof(float) * slots * (size_t)B);
    pl.off_l = off;    off += align256(sizeof(float) * slots * (size_t)B);
    pl.off_pos = off;  off += align256(sizeof(float) * (size_t)B);
    pl.off_red = off;  off += 2048;      // loss reduction: block ticket + up to 256 block sums
    pl.off_accq = off;
    if (planes_q > 1 || pl.fused || pl.anchored)
        off += align256(sizeof(float) * (size_t)planes_q * (size_t)B * dpad);
    pl.off_accp = off;
    if (planes_p > 1) off += align256(sizeof(float) * (size_t)planes_p * (size_t)N * dpad);
    pl.launches_fwd = 2;  // sweep + combine
    pl.launches_bwd = 2 + (pl.g_dq > 1 ? 1 : 0) + (pl.g_dp > 1 ? 1 : 0);
    pl.launches_build = pl.fused ? 4 + (pl.g_dp > 1 ? 1 : 0) : pl.launches_fwd + pl.launches_bwd;
    if (pl.anchored == 1) pl.launches_build = 1 + 2 * pl.launches_build;   // anchor, sequence, fallback
    // anchor, fused sweep, combine, finalize, dP sweep (+ reduce), then the gated forward + sweeps
    if (pl.anchored == 2)
        pl.launches_build = 5 + (pl.g_dp > 1 ? 1 : 0) + pl.launches_fwd + pl.launches_bwd;
    // Stored weights: B x N bf16 (pitch rounded up to 64 elements), kept when they fit the limit
    // below; the gradient partials share the regions of the sweeps they replace.
    if (pl.anchored) {
        pl.off_ref = off;   off += align256(sizeof(float) * (size_t)B);
        pl.off_flag = off;  off += 256;
    }
    pl.ldw = (N + 63) / 64 * 64;
    const size_t w_bytes = (size_t)B * (size_t)pl.ldw * 2;
    pl.mat = (stored && pl.tc && w_bytes <= kMaxStoredWeightBytes) ? 1 : 0;
    if (pl.mat) {
        pl.g_mq = gemm_groups(B, N, d);
        pl.g_mp = gemm_groups(N, B, d);
        size_t accq = align256(sizeof(float) * (size_t)pl.g_mq * (size_t)B * dpad);
        size_t accp = pl.g_mp > 1 ? align256(sizeof(float) * (size_t)pl.g_mp * (size_t)N * dpad) : 0;
        if (pl.off_accp - pl.off_accq < accq) {       // grow the dQ partial region
            size_t old_accp = off - pl.off_accp;
            pl.off_accp = pl.off_accq + accq;
            off = pl.off_accp + old_accp;
        }
        if (off - pl.off_accp < accp) off = pl.off_accp + accp;
        if (!pl.anchored) {
            pl.off_ref = off;   off += align256(sizeof(float) * (size_t)B);
            pl.off_flag = off;  off += 256;
        }
        pl.off_qs = off;    off += align256((size_t)B * (size_t)d * 2);
        pl.off_w = off;     off += align256(w_bytes);
        // anchor, sweep, combine, row scaling, dQ GEMM, dQ finalize, dP GEMM (+ reduce),
        // positive terms, then the gated fallback sequence
        pl.launches_build = 8 + (pl.g_mp > 1 ? 1 : 0) + pl.launches_build;
    }
    pl.total = off;
    return pl;
}

namespace {

// Optional per-kernel timing (gc_profile_enable): in the event set of the current call, events
// 2k / 2k+1 bracket kernel k.  Call number c since the enable uses set c % sets, so that a run of
// up to `sets` calls can be queued without a host synchronisation in between and read afterwards.
constexpr int kMaxProfileSets = 256;
struct Profile {
    bool on = false;
    int sets = 0;               // sets in use
    int created = 0;            // sets whose events exist
    int64_t calls = 0;          // calls begun since the enable
    cudaEvent_t ev[kMaxProfileSets][6];
    bool used[kMaxProfileSets][3];
};
Profile g_prof;

// Every entry point that times kernels begins with this.
void profile_begin_call() {
    if (!g_prof.on) return;
    const int set = (int)(g_prof.calls % g_prof.sets);
    for (int k = 0; k < 3; ++k) g_prof.used[set][k] = false;
    ++g_prof.calls;
}
int profile_set() { return (int)((g_prof.calls - 1) % g_prof.sets); }

struct KernelTimer {
    int k;
    cudaStream_t st;
    KernelTimer(int kernel, cudaStream_t s) : k(kernel), st(s) {   // kernel < 0: not timed
        if (g_prof.on && g_prof.calls > 0 && k >= 0) {
            cudaEventRecord(g_prof.ev[profile_set()][2 * k], st);
            g_prof.used[profile_set()][k] = true;
        }
    }
    ~KernelTimer() {
        if (g_prof.on && g_prof.calls > 0 && k >= 0)
            cudaEventRecord(g_prof.ev[profile_set()][2 * k + 1], st);
    }
};

int elem_size(int dtype) { return dtype == GC_BF16 ? 2 : 4; }

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

int check_common(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                 int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype) {
    if (!Q || !P || !pos_idx) return GC_ERR_NULL;
    if (dtype != GC_F32 && dtype != GC_BF16) return GC_ERR_DTYPE;
    if (B <= 0 || N <= 0 || d <= 0 || ldq < d || ldp < d) return GC_ERR_SHAPE;
    if (B > (int64_t)1 << 30 || N > (int64_t)1 << 30 || d > (1 << 20)) return GC_ERR_SHAPE;
    if (!(tau > 0.f) || !isfinite(tau)) return GC_ERR_SHAPE;
    if (mask_mode != GC_MASK_NONE && mask_mode != GC_MASK_SELF) return GC_ERR_MASK;
    if (mask_mode == GC_MASK_SELF && N < 2) return GC_ERR_MASK;
    int es = elem_size(dtype);
    if (!aligned16(Q) || !aligned16(P) || (ldq * es) % 16 != 0 || (ldp * es) % 16 != 0)
        return GC_ERR_ALIGN;
    return GC_OK;
}

int check_grad_out(const float* g, int64_t ld, int d) {
    if (!g) return GC_OK;
    if (ld < d) return GC_ERR_SHAPE;
    if (!aligned16(g) || (ld * 4) % 16 != 0) return GC_ERR_ALIGN;
    return GC_OK;
}

int check_ws(const void* ws, size_t ws_bytes, size_t need) {
    if (need == 0) return GC_OK;
    if (!ws || ((uintptr_t)ws & 255) != 0 || ws_bytes < need) return GC_ERR_WORKSPACE;
    return GC_OK;
}

int check_device() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return GC_ERR_CUDA; }
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return GC_ERR_CUDA;
    }
    return major == 10 ? GC_OK : GC_ERR_ARCH;
}

Problem make_problem(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                     const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                     int mask_mode, int dtype) {
    Problem p;
    p.Q = Q; p.P = P; p.pos_idx = pos_idx; p.ldq = ldq; p.ldp = ldp; p.B = B; p.N = N; p.d = d;
    p.tau = tau; p.mask_mode = mask_mode; p.dtype = dtype;
    p.b_total = 0;
    p.mask_shift = 0;
    return p;
}

constexpr Gate kOpen = {nullptr, 0};

// 1 / (B tau) of Eq. 4-7, with B the whole batch when the call covers a slice of the queries
float grad_scale(const Problem& p) {
    return 1.f / ((float)(p.b_total > 0 ? p.b_total : p.B) * p.tau);
}

int run_fwd(const Problem& p, const Plan& pl, char* ws, float* loss, float* row_lse,
            float* pos_logit, int* dev_status, cudaStream_t st, Gate gate = kOpen) {
    FwdArgs fa{};
    fa.p = p;
    fa.gate = gate;
    fa.part_m = reinterpret_cast<float*>(ws + pl.off_m);
    fa.part_l = reinterpret_cast<float*>(ws + pl.off_l);
    fa.pos_logit = reinterpret_cast<float*>(ws + pl.off_pos);
    fa.red = reinterpret_cast<float*>(ws + pl.off_red);
    fa.groups = pl.g_fwd;
    fa.dev_status = dev_status;
    cudaError_t e;
    {
        KernelTimer t(gate.flag ? -1 : 0, st);
        e = pl.tc ? tc_launch_fwd(fa, st) : simt_launch_fwd(fa, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_lse_combine(fa.part_m, fa.part_l, fa.pos_logit, p.pos_idx, fa.groups, p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, fa.red, dev_status,
                           gate, st, p.b_total, p.mask_shift);
    return e == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

// `timed`: bracket the sweep with the profiling events (only the sweeps that normally run are).
int run_sweep(const Problem& p, const Plan& pl, char* ws, int mode, const float* row_lse,
              float* out, int64_t ldo, int* dev_status, cudaStream_t st, Gate gate = kOpen,
              bool timed = true, const float* slot_m = nullptr, const float* slot_l = nullptr,
              int slots = 0) {
    SweepArgs sa{};
    sa.gate = gate;
    sa.slot_m = slot_m; sa.slot_l = slot_l; sa.slots = slots;
    const bool dq = (mode == SWEEP_DQ);
    sa.X = dq ? p.Q : p.P;   sa.ldx = dq ? p.ldq : p.ldp;   sa.nx = dq ? p.B : p.N;
    sa.Y = dq ? p.P : p.Q;   sa.ldy = dq ? p.ldp : p.ldq;   sa.ny = dq ? p.N : p.B;
    sa.d = p.d;
    sa.mode = mode;
    sa.mask_mode = p.mask_mode;
    sa.mask_delta = dq ? p.mask_shift : -p.mask_shift;
    sa.dtype = p.dtype;
    sa.inv_tau = 1.f / p.tau;
    sa.out_scale = grad_scale(p);
    sa.row_lse = row_lse;
    sa.pos_idx = p.pos_idx;
    sa.out = out;
    sa.ldo = ldo;
    sa.groups = dq ? pl.g_dq : pl.g_dp;
    sa.partial = reinterpret_cast<float*>(ws + (dq ? pl.off_accq : pl.off_accp));
    sa.dev_status = dev_status;
    cudaError_t e;
    {
        KernelTimer t(timed ? (dq ? 1 : 2) : -1, st);
        e = pl.tc ? tc_launch_sweep(sa, st) : simt_launch_sweep(sa, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    if (sa.groups > 1) {
        e = launch_partial_reduce(sa.partial, sa.groups, sa.nx, sa.d, sa.out_scale, out, ldo, gate,
                                  st);
        if (e != cudaSuccess) return GC_ERR_CUDA;
    }
    return GC_OK;
}

// gc_build_cache for wide bf16 rows: fused forward + dQ sweep, combine, dQ finalize.
int run_fused_fwd_dq(const Problem& p, const Plan& pl, char* ws, float* loss, float* row_lse,
                     float* pos_logit, float* dQ, int64_t lddq, int* dev_status,
                     cudaStream_t st, Gate gate = kOpen) {
    FwdArgs fa{};
    fa.p = p;
    fa.gate = gate;
    fa.part_m = reinterpret_cast<float*>(ws + pl.off_m);
    fa.part_l = reinterpret_cast<float*>(ws + pl.off_l);
    fa.pos_logit = reinterpret_cast<float*>(ws + pl.off_pos);
    fa.red = reinterpret_cast<float*>(ws + pl.off_red);
    fa.groups = 2 * pl.g_dq;
    fa.dev_status = dev_status;
    float* partial = reinterpret_cast<float*>(ws + pl.off_accq);
    cudaError_t e;
    {
        KernelTimer t(gate.flag ? -1 : 1, st);
        e = tc_launch_fused_dq(fa, partial, pl.g_dq, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_lse_combine(fa.part_m, fa.part_l, fa.pos_logit, p.pos_idx, fa.groups, p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, fa.red, dev_status,
                           gate, st, p.b_total, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_fused_dq_finalize(partial, pl.g_dq, fa.part_m, nullptr, row_lse, fa.pos_logit,
                                 p.pos_idx, p.P, p.ldp, p.B, p.N, p.d, p.mask_mode,
                                 grad_scale(p), dQ, lddq, gate, st, p.mask_shift);
    return e == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

// The sequence that tracks the running row maximum: forward (fused into the dQ sweep for wide
// rows), dQ, dP.  With a gate every kernel of it is gated.
int run_online_sweeps(const Problem& p, const Plan& pl, char* w, float* loss, float* row_lse,
                      float* pos_logit, float* dQ, int64_t lddq, float* dP, int64_t lddp,
                      int* dev_status, cudaStream_t st, Gate gate = kOpen, bool want_dp = true) {
    int rc;
    if (pl.fused) {
        if ((rc = run_fused_fwd_dq(p, pl, w, loss, row_lse, pos_logit, dQ, lddq, dev_status, st,
                                   gate)))
            return rc;
    } else {
        if ((rc = run_fwd(p, pl, w, loss, row_lse, pos_logit, dev_status, st, gate))) return rc;
        if ((rc = run_sweep(p, pl, w, SWEEP_DQ, row_lse, dQ, lddq, dev_status, st, gate,
                            gate.flag == nullptr)))
            return rc;
    }
    if (!want_dp) return GC_OK;
    return run_sweep(p, pl, w, SWEEP_DP, row_lse, dP, lddp, dev_status, st, gate,
                     gate.flag == nullptr);
}

// A side stream and three events per device, created on first use: work that is off a call's
// critical path (the dQ finalize, the gated fallback) runs there between a fork from and a join
// back into the caller's stream, so the call stays asynchronous on that stream alone.
struct SideStream {
    bool tried = false, ok = false;
    cudaStream_t st = nullptr;
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
};
SideStream* side_stream() {
    static SideStream per_dev[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return nullptr;
    }
    SideStream& s = per_dev[dev];
    if (!s.tried) {
        s.tried = true;
        bool good = cudaStreamCreateWithFlags(&s.st, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; i < 3 && good; ++i)
            good = cudaEventCreateWithFlags(&s.ev[i], cudaEventDisableTiming) == cudaSuccess;
        if (!good) cudaGetLastError();
        s.ok = good;
    }
    return s.ok ? &s : nullptr;
}

// gc_build_cache for rows of two column halves (four-CTA sweeps).  The forward is fused into the
// dQ sweep with the positive logit as each row's fixed scale (anchor kernel), so no running
// maximum has to be agreed across the cluster.  A weight beyond 2^100 raises the range flag; the
// kernels after the fused sweep run only while it is down, and the online-maximum sequence, which
// is always launched, runs only when it is up and then produces every output.
//
//   caller's stream:  anchor, fused sweep, dP sweep (+ reduce), which merges the forward slots
//                     of its streamed queries itself
//   side stream:      after the fused sweep: combine (row_lse, loss), dQ finalize, then the
//                     gated online-maximum sequence
// Both are joined back before the call returns.  Without a side stream everything is queued on
// the caller's stream in dependency order with the combine before the dP sweep.  Narrow rows
// (two S buffers in tensor memory) take the same sequence with the one-CTA sweeps, and forward,
// dQ and dP sweeps as the gated fallback.
int run_anchored_build(const Problem& p, const Plan& pl, char* ws, float* loss, float* row_lse,
                       float* pos_logit, float* dQ, int64_t lddq, float* dP, int64_t lddp,
                       int* dev_status, cudaStream_t st, bool want_dp = true) {
    float* ref2 = reinterpret_cast<float*>(ws + pl.off_ref);
    int* flag = reinterpret_cast<int*>(ws + pl.off_flag);
    const Gate in_range = {flag, 0}, out_of_range = {flag, 1};
    SideStream* side = side_stream();
    cudaStream_t aux = side ? side->st : st;
    FwdArgs fa{};
    fa.p = p;
    fa.part_m = reinterpret_cast<float*>(ws + pl.off_m);
    fa.part_l = reinterpret_cast<float*>(ws + pl.off_l);
    fa.pos_logit = reinterpret_cast<float*>(ws + pl.off_pos);
    fa.red = reinterpret_cast<float*>(ws + pl.off_red);
    fa.groups = 4 * pl.g_dq;      // per part: two duty pairs, or two softmax groups, x two column halves
    fa.dev_status = dev_status;
    float* partial = reinterpret_cast<float*>(ws + pl.off_accq);
    // The fused sweep is launched with programmatic serialization: it starts (loads, first S
    // tiles) while the anchor kernel still runs, and only its softmax warps wait for the
    // anchors.  Per-kernel timing (gc_profile_enable) records an event between the two launches,
    // which serialises them, so the overlap is left out while it is on.
    const bool overlap = !g_prof.on;
    cudaError_t e = launch_pos_anchor(p.Q, p.ldq, p.P, p.ldp, p.pos_idx, p.B, p.N, p.d, p.mask_mode,
                                      1.4426950408889634f / p.tau, ref2, flag, st, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    {
        KernelTimer t(1, st);
        e = pl.anchored == 1
                ? quad_launch_fused_dq(fa, partial, pl.g_dq, ref2, flag, st, overlap)
                : tc_launch_anchored_dq(fa, partial, pl.g_dq, ref2, flag, st, overlap);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    // Wide rows: a sweep step is long enough to hide the slot merge of the streamed queries,
    // so the dP sweep does not wait for the combine.  Narrow rows have short steps: there the
    // combine stays on the caller's stream and the dP sweep reads row_lse (8192 x 8192 x 128:
    // 0.100 ms per call against 0.114 with the merge inside the dP sweep).
    const bool dp_merges = side && pl.anchored == 1 && want_dp;
    cudaStream_t comb = dp_merges ? aux : st;
    if (dp_merges && (cudaEventRecord(side->ev[0], st) != cudaSuccess ||
                      cudaStreamWaitEvent(aux, side->ev[0], 0) != cudaSuccess))
        return GC_ERR_CUDA;
    e = launch_lse_combine(fa.part_m, fa.part_l, fa.pos_logit, p.pos_idx, fa.groups, p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, fa.red, dev_status,
                           in_range, comb, p.b_total, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    if (side && !dp_merges && (cudaEventRecord(side->ev[0], st) != cudaSuccess ||
                               cudaStreamWaitEvent(aux, side->ev[0], 0) != cudaSuccess))
        return GC_ERR_CUDA;
    e = launch_fused_dq_finalize(partial, pl.g_dq, nullptr, ref2, row_lse, fa.pos_logit, p.pos_idx,
                                 p.P, p.ldp, p.B, p.N, p.d, p.mask_mode,
                                 grad_scale(p), dQ, lddq, in_range, aux, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    int rc;
    if (side) {
        if ((rc = run_online_sweeps(p, pl, ws, loss, row_lse, pos_logit, dQ, lddq, dP, lddp,
                                    dev_status, aux, out_of_range, want_dp)))
            return rc;
        if (dp_merges)
            rc = run_sweep(p, pl, ws, SWEEP_DP, row_lse, dP, lddp, dev_status, st, in_range, true,
                           fa.part_m, fa.part_l, fa.groups);
        else if (want_dp)
            rc = run_sweep(p, pl, ws, SWEEP_DP, row_lse, dP, lddp, dev_status, st, in_range);
        if (rc) return rc;
        if (cudaEventRecord(side->ev[2], aux) != cudaSuccess ||
            cudaStreamWaitEvent(st, side->ev[2], 0) != cudaSuccess)
            return GC_ERR_CUDA;
        return GC_OK;
    }
    if (want_dp &&
        (rc = run_sweep(p, pl, ws, SWEEP_DP, row_lse, dP, lddp, dev_status, st, in_range)))
        return rc;
    return run_online_sweeps(p, pl, ws, loss, row_lse, pos_logit, dQ, lddq, dP, lddp, dev_status, st,
                             out_of_range, want_dp);
}

int run_build_sweeps(const Problem& p, const Plan& pl, char* w, float* loss, float* row_lse,
                     float* pos_logit, float* dQ, int64_t lddq, float* dP, int64_t lddp,
                     int* dev_status, cudaStream_t st, bool want_dp = true) {
    if (pl.anchored)
        return run_anchored_build(p, pl, w, loss, row_lse, pos_logit, dQ, lddq, dP, lddp, dev_status,
                                  st, want_dp);
    return run_online_sweeps(p, pl, w, loss, row_lse, pos_logit, dQ, lddq, dP, lddp, dev_status, st,
                             kOpen, want_dp);
}

// gc_build_cache with stored weights (Eq. 1, 5, 6-7 without recomputing a logit):
//   anchor      ref2_i = log2(e) S_{i,r_i}, the scale all weights of row i are measured against
//   sweep       W~_ij = 2^(s2_ij - ref2_i) as bf16 (0 at masked pairs and at the positive), the
//               row sums in fp32, pos_logit; a weight beyond 2^100 raises the range flag
//   combine     row_lse, loss
//   dQ          (2^(ref2_i - lse2_i) sum_j W~_ij P_j + (p_pos - 1) P_pos) / (B tau)
//   dP          (sum_i W~_ij Q'_i) / (B tau) with Q'_i = 2^(ref2_i - lse2_i) Q_i, then the
//               positive terms (p_pos - 1) Q_i / (B tau) added in fp32 in query order
// When the range flag is up (logits more than 100 powers of two above the positive's) these
// results are not usable; the gated recomputing sequence that follows then overwrites them all.
int run_build_stored(const Problem& p, const Plan& pl, char* w, float* loss, float* row_lse,
                     float* pos_logit, float* dQ, int64_t lddq, float* dP, int64_t lddp,
                     int* dev_status, cudaStream_t st) {
    float* ref2 = reinterpret_cast<float*>(w + pl.off_ref);
    int* flag = reinterpret_cast<int*>(w + pl.off_flag);
    void* qs = w + pl.off_qs;
    void* weights = w + pl.off_w;
    float* partq = reinterpret_cast<float*>(w + pl.off_accq);
    float* partp = reinterpret_cast<float*>(w + pl.off_accp);
    const float scale = grad_scale(p);
    cudaError_t e = launch_pos_anchor(p.Q, p.ldq, p.P, p.ldp, p.pos_idx, p.B, p.N, p.d, p.mask_mode,
                                      1.4426950408889634f / p.tau, ref2, flag, st, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    FwdArgs fa{};
    fa.p = p;
    fa.part_m = reinterpret_cast<float*>(w + pl.off_m);
    fa.part_l = reinterpret_cast<float*>(w + pl.off_l);
    fa.pos_logit = reinterpret_cast<float*>(w + pl.off_pos);
    fa.red = reinterpret_cast<float*>(w + pl.off_red);
    fa.groups = pl.g_fwd;
    fa.dev_status = dev_status;
    {
        KernelTimer t(0, st);
        e = tc_launch_fwd_store(fa, weights, pl.ldw, ref2, flag, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_lse_combine(fa.part_m, fa.part_l, fa.pos_logit, p.pos_idx, fa.groups, p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, fa.red, dev_status,
                           kOpen, st, p.b_total, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_scale_rows(p.Q, p.ldq, p.B, p.d, ref2, row_lse, qs, st);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    {
        KernelTimer t(1, st);
        e = launch_weight_gemm(weights, pl.ldw, p.B, p.N, 0, p.P, p.ldp, p.d, pl.g_mq, 1.f,
                               nullptr, 0, partq, dev_status, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_fused_dq_finalize(partq, pl.g_mq, nullptr, ref2, row_lse, fa.pos_logit, p.pos_idx,
                                 p.P, p.ldp, p.B, p.N, p.d, p.mask_mode, scale, dQ, lddq, kOpen,
                                 st, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    {
        KernelTimer t(2, st);
        e = launch_weight_gemm(weights, pl.ldw, p.B, p.N, 1, qs, p.d, p.d, pl.g_mp, scale, dP, lddp,
                               partp, dev_status, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    if (pl.g_mp > 1) {
        e = launch_partial_reduce(partp, pl.g_mp, p.N, p.d, scale, dP, lddp, kOpen, st);
        if (e != cudaSuccess) return GC_ERR_CUDA;
    }
    e = launch_dp_positive(p.pos_idx, p.B, p.N, p.mask_mode, fa.pos_logit, row_lse, p.Q, p.ldq, p.d,
                           scale, dP, lddp, st, p.mask_shift);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    const Gate out_of_range = {flag, 1};
    return run_online_sweeps(p, pl, w, loss, row_lse, pos_logit, dQ, lddq, dP, lddp, dev_status, st,
                             out_of_range);
}

}  // namespace
}  // namespace gc

using namespace gc;

namespace {

// One-tile batches: the whole call is one launch (gc_small.cu); timed as the fused sweep.
int run_small(int op, const Problem& p, const float* row_lse_in, float* loss, float* row_lse,
              float* pos_logit, float* dQ, int64_t lddq, float* dP, int64_t lddp, int* dev_status,
              cudaStream_t st) {
    KernelTimer t(1, st);
    return launch_small(op, p, row_lse_in, loss, row_lse, pos_logit, dQ, lddq, dP, lddp, dev_status,
                        st) == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

// fp32 batches of a few tiles (gc_small.cu): forward = tile kernel + combine, gradients = tile
// kernel + one reduce per side that has several planes.
int run_tiles_fwd(const Problem& p, const Plan& pl, char* ws, float* loss, float* row_lse,
                  float* pos_logit, int* dev_status, cudaStream_t st) {
    float* part_m = reinterpret_cast<float*>(ws + pl.off_m);
    float* part_l = reinterpret_cast<float*>(ws + pl.off_l);
    float* pos_ws = reinterpret_cast<float*>(ws + pl.off_pos);
    float* red = reinterpret_cast<float*>(ws + pl.off_red);
    cudaError_t e;
    {
        KernelTimer t(0, st);
        e = launch_small_tiled_fwd(p, part_m, part_l, pos_ws, red, dev_status, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_lse_combine(part_m, part_l, pos_ws, p.pos_idx, small_tiles_y(p.N, p.dtype), p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, red, dev_status, kOpen, st,
                           p.b_total, p.mask_shift);
    return e == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int run_tiles_bwd(const Problem& p, const Plan& pl, char* ws, const float* row_lse, float* dQ,
                  int64_t lddq, float* dP, int64_t lddp, int* dev_status, cudaStream_t st) {
    float* partial_q = reinterpret_cast<float*>(ws + pl.off_accq);
    float* partial_p = reinterpret_cast<float*>(ws + pl.off_accp);
    cudaError_t e;
    {
        KernelTimer t(1, st);
        e = launch_small_tiled_bwd(p, row_lse, dQ, lddq, partial_q, dP, lddp, partial_p, dev_status,
                                   st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    const int tx = small_tiles_x(p.B), ty = small_tiles_y(p.N, p.dtype);
    if (dQ && ty > 1 &&
        launch_partial_reduce(partial_q, ty, p.B, p.d, grad_scale(p), dQ, lddq, kOpen, st) != cudaSuccess)
        return GC_ERR_CUDA;
    if (dP && tx > 1 &&
        launch_partial_reduce(partial_p, tx, p.N, p.d, grad_scale(p), dP, lddp, kOpen, st) != cudaSuccess)
        return GC_ERR_CUDA;
    return GC_OK;
}

}  // namespace

// Scratch for gc_loss_fwd_static.  In host code this name is only a handle for the symbol: the
// address a kernel can use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[GC_STATIC_SCRATCH_BYTES];

namespace {

// The forward sweep alone writes g_fwd (scale, sum) slots per row: lays those regions, the
// gathered positive logits and the loss scratch out back to back (the workspace layout of the
// other calls reserves the slots of the widest build plan) and returns the bytes they take.
size_t forward_layout(Plan* pl, int64_t B, int64_t N) {
    size_t slots = (size_t)pl->g_fwd;
    if (pl->tiles && (size_t)pl->tiles_y > slots) slots = (size_t)pl->tiles_y;
    size_t off = 0;
    pl->off_m = off;    off += align256(sizeof(float) * slots * (size_t)B);
    pl->off_l = off;    off += align256(sizeof(float) * slots * (size_t)B);
    pl->off_pos = off;  off += align256(sizeof(float) * (size_t)B);
    pl->off_red = off;  off += 2048;
    return off;
}

// Device address of g_static_scratch on the current device, or nullptr on failure.
void* static_scratch_ptr() {
    static void* cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return nullptr;
    }
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        cached[dev] = ptr;
    }
    return cached[dev];
}

}  // namespace

extern "C" {

size_t gc_workspace_bytes(int op, int64_t B, int64_t N, int d, int dtype) {
    if (op < GC_OP_FWD || op > GC_OP_BUILD_STORED || B <= 0 || N <= 0 || d <= 0) return 0;
    if (dtype != GC_F32 && dtype != GC_BF16) return 0;
    // one layout serves the three calls of the paper's path; the stored-weights build appends its
    // own regions to it
    return make_plan(B, N, d, dtype, op == GC_OP_BUILD_STORED).total;
}

const char* gc_plan_name(int op, int64_t B, int64_t N, int d, int dtype) {
    if (op < GC_OP_FWD || op > GC_OP_BUILD_STORED || B <= 0 || N <= 0 || d <= 0) return "invalid";
    if (op == GC_OP_BUILD_STORED && !make_plan(B, N, d, dtype, true).mat) return "invalid";
    if (op != GC_OP_BUILD_STORED && small_applicable(B, N, d, dtype)) return "tcgen05-one-tile";
    if (op != GC_OP_BUILD_STORED && small_tiled_applicable(B, N, d, dtype)) return "tcgen05-tiles";
    return tc_supported(B, N, d, dtype) ? "tcgen05" : "simt";
}

int gc_kernel_launches(int op, int64_t B, int64_t N, int d, int dtype) {
    if (B <= 0 || N <= 0 || d <= 0) return 0;
    if (op >= GC_OP_FWD && op <= GC_OP_BUILD && small_applicable(B, N, d, dtype)) return 1;
    if (op >= GC_OP_FWD && op <= GC_OP_BUILD && small_tiled_applicable(B, N, d, dtype)) {
        const int reduces = (small_tiles_y(N, dtype) > 1 ? 1 : 0) + (small_tiles_x(B) > 1 ? 1 : 0);
        if (op == GC_OP_FWD) return 2;                  // tile kernel, combine
        if (op == GC_OP_BWD) return 2 + reduces;        // pos_idx validation, tile kernel, reduces
        return 3 + reduces;
    }
    Plan pl = make_plan(B, N, d, dtype);
    if (op == GC_OP_FWD) return pl.launches_fwd;
    if (op == GC_OP_BWD) return pl.launches_bwd + 1;   // + pos_idx validation
    if (op == GC_OP_BUILD) return pl.launches_build;
    if (op == GC_OP_BUILD_STORED) return make_plan(B, N, d, dtype, true).launches_build;
    return 0;
}

int gc_loss_fwd(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype, float* loss,
                float* row_lse, float* pos_logit, void* ws, size_t ws_bytes, int* dev_status,
                void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (!loss || !row_lse) return GC_ERR_NULL;
    Plan pl = make_plan(B, N, d, dtype);
    if ((rc = check_ws(ws, ws_bytes, pl.total))) return rc;
    if ((rc = check_device())) return rc;
    profile_begin_call();
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (small_applicable(B, N, d, dtype))
        return run_small(GC_OP_FWD, p, nullptr, loss, row_lse, pos_logit, nullptr, 0, nullptr, 0,
                         dev_status, static_cast<cudaStream_t>(cuda_stream));
    if (pl.tiles)
        return run_tiles_fwd(p, pl, static_cast<char*>(ws), loss, row_lse, pos_logit, dev_status,
                             static_cast<cudaStream_t>(cuda_stream));
    return run_fwd(p, pl, static_cast<char*>(ws), loss, row_lse, pos_logit, dev_status,
                   static_cast<cudaStream_t>(cuda_stream));
}

size_t gc_static_scratch_need(int64_t B, int64_t N, int d, int dtype) {
    if (B <= 0 || N <= 0 || d <= 0 || (dtype != GC_F32 && dtype != GC_BF16)) return 0;
    Plan pl = make_plan(B, N, d, dtype);
    return forward_layout(&pl, B, N);
}

int gc_loss_fwd_static(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                       const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                       int mask_mode, int dtype, float* loss, float* row_lse, float* pos_logit,
                       int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (!loss || !row_lse) return GC_ERR_NULL;
    Plan pl = make_plan(B, N, d, dtype);
    if (forward_layout(&pl, B, N) > (size_t)GC_STATIC_SCRATCH_BYTES) return GC_ERR_LIMIT;
    if ((rc = check_device())) return rc;
    void* scratch = static_scratch_ptr();
    if (!scratch) return GC_ERR_CUDA;
    profile_begin_call();
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (small_applicable(B, N, d, dtype))      // one launch, no scratch at all
        return run_small(GC_OP_FWD, p, nullptr, loss, row_lse, pos_logit, nullptr, 0, nullptr, 0,
                         dev_status, static_cast<cudaStream_t>(cuda_stream));
    if (pl.tiles)
        return run_tiles_fwd(p, pl, static_cast<char*>(scratch), loss, row_lse, pos_logit,
                             dev_status, static_cast<cudaStream_t>(cuda_stream));
    return run_fwd(p, pl, static_cast<char*>(scratch), loss, row_lse, pos_logit, dev_status,
                   static_cast<cudaStream_t>(cuda_stream));
}

int gc_loss_bwd(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                const float* row_lse, float* dQ, int64_t lddq, float* dP, int64_t lddp, void* ws,
                size_t ws_bytes, int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (!row_lse) return GC_ERR_NULL;
    if ((rc = check_grad_out(dQ, lddq, d))) return rc;
    if ((rc = check_grad_out(dP, lddp, d))) return rc;
    Plan pl = make_plan(B, N, d, dtype);
    if ((rc = check_ws(ws, ws_bytes, pl.total))) return rc;
    if ((rc = check_device())) return rc;
    profile_begin_call();
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (small_applicable(B, N, d, dtype) && (dQ || dP))
        return run_small(GC_OP_BWD, p, row_lse, nullptr, nullptr, nullptr, dQ, lddq, dP, lddp,
                         dev_status, st);
    if (dev_status && launch_pos_check(pos_idx, B, N, mask_mode, dev_status, st) != cudaSuccess)
        return GC_ERR_CUDA;
    char* w = static_cast<char*>(ws);
    if (pl.tiles && (dQ || dP))
        return run_tiles_bwd(p, pl, w, row_lse, dQ, lddq, dP, lddp, dev_status, st);
    if (dQ && (rc = run_sweep(p, pl, w, SWEEP_DQ, row_lse, dQ, lddq, dev_status, st))) return rc;
    if (dP && (rc = run_sweep(p, pl, w, SWEEP_DP, row_lse, dP, lddp, dev_status, st))) return rc;
    return GC_OK;
}

int gc_build_cache(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                   int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype, float* loss,
                   float* row_lse, float* pos_logit, float* dQ, int64_t lddq, float* dP,
                   int64_t lddp, void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (!loss || !row_lse || !dQ || !dP) return GC_ERR_NULL;
    if ((rc = check_grad_out(dQ, lddq, d))) return rc;
    if ((rc = check_grad_out(dP, lddp, d))) return rc;
    Plan pl = make_plan(B, N, d, dtype);
    if ((rc = check_ws(ws, ws_bytes, pl.total))) return rc;
    if ((rc = check_device())) return rc;
    profile_begin_call();
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    char* w = static_cast<char*>(ws);
    if (small_applicable(B, N, d, dtype))
        return run_small(GC_OP_BUILD, p, nullptr, loss, row_lse, pos_logit, dQ, lddq, dP, lddp,
                         dev_status, st);
    if (pl.tiles) {
        if ((rc = run_tiles_fwd(p, pl, w, loss, row_lse, pos_logit, dev_status, st))) return rc;
        return run_tiles_bwd(p, pl, w, row_lse, dQ, lddq, dP, lddp, dev_status, st);
    }
    return run_build_sweeps(p, pl, w, loss, row_lse, pos_logit, dQ, lddq, dP, lddp, dev_status, st);
}

int gc_build_cache_stored(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                          const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                          int mask_mode, int dtype, float* loss, float* row_lse, float* pos_logit,
                          float* dQ, int64_t lddq, float* dP, int64_t lddp, void* ws,
                          size_t ws_bytes, int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (!loss || !row_lse || !dQ || !dP) return GC_ERR_NULL;
    if ((rc = check_grad_out(dQ, lddq, d))) return rc;
    if ((rc = check_grad_out(dP, lddp, d))) return rc;
    Plan pl = make_plan(B, N, d, dtype, true);
    if (!pl.mat) return GC_ERR_LIMIT;       // not a tcgen05 shape, or the weights exceed the limit
    if ((rc = check_ws(ws, ws_bytes, pl.total))) return rc;
    if ((rc = check_device())) return rc;
    profile_begin_call();
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    return run_build_stored(p, pl, static_cast<char*>(ws), loss, row_lse, pos_logit, dQ, lddq, dP,
                            lddp, dev_status, st);
}

size_t gc_shard_workspace_bytes(int64_t B, int64_t N, int d, int dtype, int64_t q_count,
                                int64_t p_count) {
    if (B <= 0 || N <= 0 || d <= 0 || q_count <= 0 || p_count <= 0 || q_count > B || p_count > N)
        return 0;
    if (dtype != GC_F32 && dtype != GC_BF16) return 0;
    const size_t a = make_plan(q_count, N, d, dtype).total;
    const size_t b = make_plan(B, p_count, d, dtype).total + align256(sizeof(int32_t) * (size_t)B);
    return a > b ? a : b;
}

int gc_shard_fwd_dq(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                    int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype, int64_t q0,
                    int64_t q_count, float* loss_part, float* row_lse, float* pos_logit, float* dQ,
                    int64_t lddq, void* ws, size_t ws_bytes, int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (q0 < 0 || q_count <= 0 || q0 + q_count > B) return GC_ERR_SHAPE;
    if (!loss_part || !row_lse || !dQ) return GC_ERR_NULL;
    if ((rc = check_grad_out(dQ, lddq, d))) return rc;
    Plan pl = make_plan(q_count, N, d, dtype);
    if ((rc = check_ws(ws, ws_bytes, pl.total))) return rc;
    if ((rc = check_device())) return rc;
    profile_begin_call();
    const char* q_first = static_cast<const char*>(Q) + (size_t)q0 * (size_t)ldq * elem_size(dtype);
    Problem p = make_problem(q_first, ldq, P, ldp, pos_idx + q0, q_count, N, d, tau, mask_mode, dtype);
    p.b_total = B;
    p.mask_shift = q0;             // local query i is query q0 + i of the batch
    return run_build_sweeps(p, pl, static_cast<char*>(ws), loss_part, row_lse + q0,
                            pos_logit ? pos_logit + q0 : nullptr, dQ, lddq, nullptr, 0, dev_status,
                            static_cast<cudaStream_t>(cuda_stream), false);
}

int gc_shard_dp(const void* Q, int64_t ldq, const void* P, int64_t ldp, const int32_t* pos_idx,
                int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                const float* row_lse, int64_t p0, int64_t p_count, float* dP, int64_t lddp, void* ws,
                size_t ws_bytes, int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (p0 < 0 || p_count <= 0 || p0 + p_count > N) return GC_ERR_SHAPE;
    if (!row_lse || !dP) return GC_ERR_NULL;
    if ((rc = check_grad_out(dP, lddp, d))) return rc;
    Plan pl = make_plan(B, p_count, d, dtype);
    const size_t need = pl.total + align256(sizeof(int32_t) * (size_t)B);
    if ((rc = check_ws(ws, ws_bytes, need))) return rc;
    if ((rc = check_device())) return rc;
    profile_begin_call();
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* w = static_cast<char*>(ws);
    // positives counted from the slice's first passage; those outside the slice match no row
    int32_t* pos_local = reinterpret_cast<int32_t*>(w + pl.total);
    if (dev_status && launch_pos_check(pos_idx, B, N, mask_mode, dev_status, st) != cudaSuccess)
        return GC_ERR_CUDA;
    if (launch_shift_pos(pos_idx, B, p0, p_count, pos_local, st) != cudaSuccess) return GC_ERR_CUDA;
    const char* p_first = static_cast<const char*>(P) + (size_t)p0 * (size_t)ldp * elem_size(dtype);
    Problem p = make_problem(Q, ldq, p_first, ldp, pos_local, B, p_count, d, tau, mask_mode, dtype);
    p.mask_shift = -p0;            // local passage j is passage p0 + j of the batch
    return run_sweep(p, pl, w, SWEEP_DP, row_lse, dP, lddp, dev_status, st);
}

int gc_profile_enable(int sets) {
    if (sets < 0 || sets > kMaxProfileSets) return GC_ERR_LIMIT;
    for (; g_prof.created < sets; ++g_prof.created)
        for (int i = 0; i < 6; ++i)
            if (cudaEventCreate(&g_prof.ev[g_prof.created][i]) != cudaSuccess) return GC_ERR_CUDA;
    g_prof.on = sets > 0;
    g_prof.sets = sets;
    g_prof.calls = 0;
    for (int s = 0; s < sets; ++s)
        for (int k = 0; k < 3; ++k) g_prof.used[s][k] = false;
    return GC_OK;
}

int gc_profile_read_call(int64_t call, float* ms_fwd, float* ms_dq, float* ms_dp) {
    if (!ms_fwd || !ms_dq || !ms_dp) return GC_ERR_NULL;
    float* dst[3] = {ms_fwd, ms_dq, ms_dp};
    for (int k = 0; k < 3; ++k) *dst[k] = 0.f;
    if (g_prof.sets == 0 || call < 0 || call >= g_prof.calls || call < g_prof.calls - g_prof.sets)
        return GC_ERR_LIMIT;                 // never made, or its event set has been reused
    const int set = (int)(call % g_prof.sets);
    for (int k = 0; k < 3; ++k) {
        if (!g_prof.used[set][k]) continue;
        if (cudaEventSynchronize(g_prof.ev[set][2 * k + 1]) != cudaSuccess) return GC_ERR_CUDA;
        if (cudaEventElapsedTime(dst[k], g_prof.ev[set][2 * k], g_prof.ev[set][2 * k + 1]) !=
            cudaSuccess)
            return GC_ERR_CUDA;
    }
    return GC_OK;
}

int gc_profile_read(float* ms_fwd, float* ms_dq, float* ms_dp) {
    if (!ms_fwd || !ms_dq || !ms_dp) return GC_ERR_NULL;
    if (g_prof.calls == 0) {
        *ms_fwd = *ms_dq = *ms_dp = 0.f;
        return GC_OK;
    }
    return gc_profile_read_call(g_prof.calls - 1, ms_fwd, ms_dq, ms_dp);
}

const char* gc_status_string(int status) {
    switch (status) {
        case GC_OK: return "ok";
        case GC_ERR_NULL: return "a required pointer is NULL";
        case GC_ERR_SHAPE: return "bad shape, leading dimension or temperature";
        case GC_ERR_DTYPE: return "unknown dtype";
        case GC_ERR_MASK: return "bad mask mode";
        case GC_ERR_ALIGN: return "rows must start on 16-byte boundaries";
        case GC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GC_ERR_CUDA: return "a CUDA call failed";
        case GC_ERR_ARCH: return "device is not compute capability 10.x";
        case GC_ERR_LIMIT:
            return "problem exceeds a built-in limit of this entry point (static scratch size, or "
                   "dtype / shape / size of the stored weights)";
        default: return "unknown status";
    }
}

}  // extern "C"
