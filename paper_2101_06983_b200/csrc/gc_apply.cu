// Step 3 of Gradient Cache for a linear encoder f(s) = W s (Section 3.3, Eq. 8; Eq. 9 for g):
// the representation gradients of one sub-batch, read from the cache, times the sub-batch's
// encoder inputs,
//
//     dW[a][b] (+)= sum_i U[i][a] X[i][b]          U: rows x d fp32 (cache slice), X: rows x d_in bf16
//
// as one tensor-core GEMM with fp32 accumulation.  The cache is fp32 and the tensor cores take
// bf16, so every u is split into two bf16 terms, hi = rn(u) and lo = rn(u - hi), whose sum
// misses u by at most 2^-17 |u|; the two terms sit side by side as 2 d output rows:
//
//     Ucat = [hi(U) | lo(U)]  (rows x 2 d),   T = Ucat^T X  (2 d x d_in),   dW = T[0:d] + T[d:2d]
//
// which is the transposed-A product of gc_gemm.cu (MN-major A, contraction split over CTAs,
// unscaled fp32 partials) reading X as it is.  A last kernel adds the two halves of every
// partial in part order and either overwrites dW (first sub-batch) or adds to it (the outer sum
// of Eq. 8).  No atomics: deterministic.
#include <cuda_bf16.h>

#include "gc_internal.h"

namespace gc {

namespace {

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// One thread per 4 columns of a U row: hi at column c, lo at column d + c of the 2 d wide row.
__global__ void __launch_bounds__(256)
apply_prep_kernel(const float* __restrict__ U, int64_t ldu, int64_t rows, int d,
                  __nv_bfloat16* __restrict__ Ucat) {
    const int64_t items = rows * (d / 4);
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < items;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / (d / 4);
        const int c = 4 * (int)(e - i * (d / 4));
        const float4 u = *reinterpret_cast<const float4*>(U + i * ldu + c);
        const float v[4] = {u.x, u.y, u.z, u.w};
        __nv_bfloat16 hi[4], lo[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            hi[k] = __float2bfloat16_rn(v[k]);
            lo[k] = __float2bfloat16_rn(v[k] - __bfloat162float(hi[k]));
        }
        __nv_bfloat16* row = Ucat + i * (2 * (int64_t)d);
        *reinterpret_cast<uint2*>(row + c) = *reinterpret_cast<const uint2*>(hi);
        *reinterpret_cast<uint2*>(row + d + c) = *reinterpret_cast<const uint2*>(lo);
    }
}

// dW[a][b] = (accumulate ? dW[a][b] : 0) + sum_g (partial[g][a][b] + partial[g][d + a][b]), parts
// in index order; a partial plane is [2 d][d_in].
__global__ void __launch_bounds__(256)
apply_reduce_kernel(const float4* __restrict__ partial, int groups, int d, int d_in4,
                    float* __restrict__ dW, int64_t lddw, int accumulate) {
    const int64_t total = (int64_t)d * d_in4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int g = 0; g < groups; ++g) {
            const float4 h = partial[(int64_t)g * 2 * total + e];
            const float4 l = partial[(int64_t)g * 2 * total + total + e];
            s.x += h.x + l.x; s.y += h.y + l.y; s.z += h.z + l.z; s.w += h.w + l.w;
        }
        const int64_t a = e / d_in4;
        const int b = 4 * (int)(e - a * d_in4);
        float4* dst = reinterpret_cast<float4*>(dW + a * lddw + b);
        if (accumulate) {
            const float4 o = *dst;
            s.x += o.x; s.y += o.y; s.z += o.z; s.w += o.w;
        }
        *dst = s;
    }
}

struct ApplyPlan {
    int groups;
    size_t off_u, off_part, total;
};

ApplyPlan make_apply_plan(int64_t rows, int d, int d_in) {
    ApplyPlan pl{};
    pl.groups = gemm_groups(2 * (int64_t)d, rows, d_in);
    size_t off = 0;
    pl.off_u = off;    off += align256((size_t)2 * rows * d * sizeof(__nv_bfloat16));
    pl.off_part = off; off += align256((size_t)pl.groups * 2 * d * d_in * sizeof(float));
    pl.total = off;
    return pl;
}

bool apply_shape_ok(int64_t rows, int d, int d_in) {
    return rows > 0 && rows <= ((int64_t)1 << 30) && d > 0 && d_in > 0 && d <= (1 << 20);
}

}  // namespace

}  // namespace gc

using namespace gc;

extern "C" {

size_t gc_cache_apply_workspace_bytes(int64_t rows, int d, int d_in) {
    if (!apply_shape_ok(rows, d, d_in) || d % 8 != 0 || d_in % 64 != 0 || d_in > 4096) return 0;
    return make_apply_plan(rows, d, d_in).total;
}

int gc_cache_apply(const float* U, int64_t ldu, const void* X, int64_t ldx, int64_t rows, int d,
                   int d_in, int x_dtype, float* dW, int64_t lddw, int accumulate, void* ws,
                   size_t ws_bytes, int* dev_status, void* cuda_stream) {
    if (!U || !X || !dW) return GC_ERR_NULL;
    if (x_dtype != GC_BF16) return GC_ERR_DTYPE;
    if (!apply_shape_ok(rows, d, d_in) || ldu < d || ldx < d_in || lddw < d_in) return GC_ERR_SHAPE;
    if (d % 8 != 0 || d_in % 64 != 0 || d_in > 4096) return GC_ERR_LIMIT;
    if (((uintptr_t)U & 15) || ((uintptr_t)X & 15) || ((uintptr_t)dW & 15) || (ldu * 4) % 16 ||
        (ldx * 2) % 16 || (lddw * 4) % 16)
        return GC_ERR_ALIGN;
    const ApplyPlan pl = make_apply_plan(rows, d, d_in);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < pl.total) return GC_ERR_WORKSPACE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return GC_ERR_CUDA;
    }
    if (major != 10) return GC_ERR_ARCH;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* w = static_cast<char*>(ws);
    __nv_bfloat16* Ucat = reinterpret_cast<__nv_bfloat16*>(w + pl.off_u);
    float* partial = reinterpret_cast<float*>(w + pl.off_part);

    const int64_t items = rows * (d / 4);
    int blocks = (int)((items + 255) / 256);
    if (blocks > 8 * sm_count()) blocks = 8 * sm_count();
    apply_prep_kernel<<<blocks, 256, 0, st>>>(U, ldu, rows, d, Ucat);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    // Ucat is the [B x N] = [rows x 2 d] operand read transposed: output rows are its columns
    if (launch_weight_gemm(Ucat, 2 * (int64_t)d, rows, 2 * (int64_t)d, 1, X, ldx, d_in, pl.groups,
                           1.f, nullptr, 0, partial, dev_status, st) != cudaSuccess)
        return GC_ERR_CUDA;
    const int64_t total = (int64_t)d * (d_in / 4);
    blocks = (int)((total + 255) / 256);
    if (blocks > 8 * sm_count()) blocks = 8 * sm_count();
    apply_reduce_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(partial), pl.groups,
                                                d, d_in / 4, dW, lddw, accumulate ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

}  // extern "C"
