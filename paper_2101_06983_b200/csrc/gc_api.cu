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

Plan make_plan(int64_t B, int64_t N, int d, int dtype) {
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
    pl.fused = (pl.tc && tc_fused_applicable(d)) ? 1 : 0;
    size_t dpad = (size_t)((d + 3) & ~3);
    // (max, sum) slots: the forward sweep writes g_fwd of them per row, the fused sweep 2 g_dq
    size_t slots = (size_t)pl.g_fwd;
    if (pl.fused && (size_t)(2 * pl.g_dq) > slots) slots = (size_t)(2 * pl.g_dq);
    size_t off = 0;
    pl.off_m = off;    off += align256(sizeof(float) * slots * (size_t)B);
    pl.off_l = off;    off += align256(sizeof(float) * slots * (size_t)B);
    pl.off_pos = off;  off += align256(sizeof(float) * (size_t)B);
    pl.off_accq = off;
    if (pl.g_dq > 1 || pl.fused) off += align256(sizeof(float) * (size_t)pl.g_dq * (size_t)B * dpad);
    pl.off_accp = off;
    if (pl.g_dp > 1) off += align256(sizeof(float) * (size_t)pl.g_dp * (size_t)N * dpad);
    pl.total = off;
    pl.launches_fwd = 2;  // sweep + combine
    pl.launches_bwd = 2 + (pl.g_dq > 1 ? 1 : 0) + (pl.g_dp > 1 ? 1 : 0);
    pl.launches_build = pl.fused ? 4 + (pl.g_dp > 1 ? 1 : 0) : pl.launches_fwd + pl.launches_bwd;
    return pl;
}

namespace {

// Optional per-kernel timing (gc_profile_enable): events 2k / 2k+1 bracket kernel k.
struct Profile {
    bool on = false;
    bool created = false;
    cudaEvent_t ev[6];
    bool used[3] = {false, false, false};
};
Profile g_prof;

struct KernelTimer {
    int k;
    cudaStream_t st;
    KernelTimer(int kernel, cudaStream_t s) : k(kernel), st(s) {
        if (g_prof.on) { cudaEventRecord(g_prof.ev[2 * k], st); g_prof.used[k] = true; }
    }
    ~KernelTimer() {
        if (g_prof.on) cudaEventRecord(g_prof.ev[2 * k + 1], st);
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
    return p;
}

int run_fwd(const Problem& p, const Plan& pl, char* ws, float* loss, float* row_lse,
            float* pos_logit, int* dev_status, cudaStream_t st) {
    FwdArgs fa;
    fa.p = p;
    fa.part_m = reinterpret_cast<float*>(ws + pl.off_m);
    fa.part_l = reinterpret_cast<float*>(ws + pl.off_l);
    fa.pos_logit = reinterpret_cast<float*>(ws + pl.off_pos);
    fa.groups = pl.g_fwd;
    fa.dev_status = dev_status;
    cudaError_t e;
    {
        KernelTimer t(0, st);
        e = pl.tc ? tc_launch_fwd(fa, st) : simt_launch_fwd(fa, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_lse_combine(fa.part_m, fa.part_l, fa.pos_logit, p.pos_idx, fa.groups, p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, dev_status, st);
    return e == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int run_sweep(const Problem& p, const Plan& pl, char* ws, int mode, const float* row_lse,
              float* out, int64_t ldo, int* dev_status, cudaStream_t st) {
    SweepArgs sa;
    const bool dq = (mode == SWEEP_DQ);
    sa.X = dq ? p.Q : p.P;   sa.ldx = dq ? p.ldq : p.ldp;   sa.nx = dq ? p.B : p.N;
    sa.Y = dq ? p.P : p.Q;   sa.ldy = dq ? p.ldp : p.ldq;   sa.ny = dq ? p.N : p.B;
    sa.d = p.d;
    sa.mode = mode;
    sa.mask_mode = p.mask_mode;
    sa.dtype = p.dtype;
    sa.inv_tau = 1.f / p.tau;
    sa.out_scale = 1.f / ((float)p.B * p.tau);
    sa.row_lse = row_lse;
    sa.pos_idx = p.pos_idx;
    sa.out = out;
    sa.ldo = ldo;
    sa.groups = dq ? pl.g_dq : pl.g_dp;
    sa.partial = reinterpret_cast<float*>(ws + (dq ? pl.off_accq : pl.off_accp));
    sa.dev_status = dev_status;
    cudaError_t e;
    {
        KernelTimer t(dq ? 1 : 2, st);
        e = pl.tc ? tc_launch_sweep(sa, st) : simt_launch_sweep(sa, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    if (sa.groups > 1) {
        e = launch_partial_reduce(sa.partial, sa.groups, sa.nx, sa.d, sa.out_scale, out, ldo, st);
        if (e != cudaSuccess) return GC_ERR_CUDA;
    }
    return GC_OK;
}

// gc_build_cache for wide bf16 rows: fused forward + dQ sweep, combine, dQ finalize.
int run_fused_fwd_dq(const Problem& p, const Plan& pl, char* ws, float* loss, float* row_lse,
                     float* pos_logit, float* dQ, int64_t lddq, int* dev_status,
                     cudaStream_t st) {
    FwdArgs fa;
    fa.p = p;
    fa.part_m = reinterpret_cast<float*>(ws + pl.off_m);
    fa.part_l = reinterpret_cast<float*>(ws + pl.off_l);
    fa.pos_logit = reinterpret_cast<float*>(ws + pl.off_pos);
    fa.groups = 2 * pl.g_dq;
    fa.dev_status = dev_status;
    float* partial = reinterpret_cast<float*>(ws + pl.off_accq);
    cudaError_t e;
    {
        KernelTimer t(1, st);
        e = tc_launch_fused_dq(fa, partial, pl.g_dq, st);
    }
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_lse_combine(fa.part_m, fa.part_l, fa.pos_logit, p.pos_idx, fa.groups, p.B, p.N,
                           p.mask_mode, row_lse, pos_logit, loss, dev_status, st);
    if (e != cudaSuccess) return GC_ERR_CUDA;
    e = launch_fused_dq_finalize(partial, pl.g_dq, fa.part_m, row_lse, fa.pos_logit, p.pos_idx, p.P,
                                 p.ldp, p.B, p.N, p.d, p.mask_mode,
                                 1.f / ((float)p.B * p.tau), dQ, lddq, st);
    return e == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

}  // namespace
}  // namespace gc

using namespace gc;

// Scratch for gc_loss_fwd_static.  In host code this name is only a handle for the symbol: the
// address a kernel can use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_scratch[GC_STATIC_SCRATCH_BYTES];

namespace {

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
    if (op < GC_OP_FWD || op > GC_OP_BUILD || B <= 0 || N <= 0 || d <= 0) return 0;
    if (dtype != GC_F32 && dtype != GC_BF16) return 0;
    return make_plan(B, N, d, dtype).total;   // one layout serves all three calls
}

const char* gc_plan_name(int op, int64_t B, int64_t N, int d, int dtype) {
    (void)op;
    if (B <= 0 || N <= 0 || d <= 0) return "invalid";
    return tc_supported(B, N, d, dtype) ? "tcgen05" : "simt";
}

int gc_kernel_launches(int op, int64_t B, int64_t N, int d, int dtype) {
    if (B <= 0 || N <= 0 || d <= 0) return 0;
    Plan pl = make_plan(B, N, d, dtype);
    if (op == GC_OP_FWD) return pl.launches_fwd;
    if (op == GC_OP_BWD) return pl.launches_bwd + 1;   // + pos_idx validation
    if (op == GC_OP_BUILD) return pl.launches_build;
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
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    return run_fwd(p, pl, static_cast<char*>(ws), loss, row_lse, pos_logit, dev_status,
                   static_cast<cudaStream_t>(cuda_stream));
}

size_t gc_static_scratch_need(int64_t B, int64_t N, int d, int dtype) {
    if (B <= 0 || N <= 0 || d <= 0 || (dtype != GC_F32 && dtype != GC_BF16)) return 0;
    return make_plan(B, N, d, dtype).off_accq;   // the forward part of the workspace layout
}

int gc_loss_fwd_static(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                       const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                       int mask_mode, int dtype, float* loss, float* row_lse, float* pos_logit,
                       int* dev_status, void* cuda_stream) {
    int rc = check_common(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (rc) return rc;
    if (!loss || !row_lse) return GC_ERR_NULL;
    Plan pl = make_plan(B, N, d, dtype);
    if (pl.off_accq > (size_t)GC_STATIC_SCRATCH_BYTES) return GC_ERR_LIMIT;
    if ((rc = check_device())) return rc;
    void* scratch = static_scratch_ptr();
    if (!scratch) return GC_ERR_CUDA;
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
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
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    if (dev_status && launch_pos_check(pos_idx, B, N, mask_mode, dev_status, st) != cudaSuccess)
        return GC_ERR_CUDA;
    char* w = static_cast<char*>(ws);
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
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Problem p = make_problem(Q, ldq, P, ldp, pos_idx, B, N, d, tau, mask_mode, dtype);
    char* w = static_cast<char*>(ws);
    if (pl.fused) {
        if ((rc = run_fused_fwd_dq(p, pl, w, loss, row_lse, pos_logit, dQ, lddq, dev_status, st)))
            return rc;
    } else {
        if ((rc = run_fwd(p, pl, w, loss, row_lse, pos_logit, dev_status, st))) return rc;
        if ((rc = run_sweep(p, pl, w, SWEEP_DQ, row_lse, dQ, lddq, dev_status, st))) return rc;
    }
    if ((rc = run_sweep(p, pl, w, SWEEP_DP, row_lse, dP, lddp, dev_status, st))) return rc;
    return GC_OK;
}

int gc_profile_enable(int on) {
    if (on && !g_prof.created) {
        for (int i = 0; i < 6; ++i)
            if (cudaEventCreate(&g_prof.ev[i]) != cudaSuccess) return GC_ERR_CUDA;
        g_prof.created = true;
    }
    g_prof.on = (on != 0);
    for (int k = 0; k < 3; ++k) g_prof.used[k] = false;
    return GC_OK;
}

int gc_profile_read(float* ms_fwd, float* ms_dq, float* ms_dp) {
    if (!ms_fwd || !ms_dq || !ms_dp) return GC_ERR_NULL;
    float* dst[3] = {ms_fwd, ms_dq, ms_dp};
    for (int k = 0; k < 3; ++k) {
        *dst[k] = 0.f;
        if (!g_prof.created || !g_prof.used[k]) continue;
        if (cudaEventSynchronize(g_prof.ev[2 * k + 1]) != cudaSuccess) return GC_ERR_CUDA;
        if (cudaEventElapsedTime(dst[k], g_prof.ev[2 * k], g_prof.ev[2 * k + 1]) != cudaSuccess)
            return GC_ERR_CUDA;
        g_prof.used[k] = false;
    }
    return GC_OK;
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
        case GC_ERR_LIMIT: return "problem needs more scratch than the library's built-in area holds";
        default: return "unknown status";
    }
}

}  // extern "C"
