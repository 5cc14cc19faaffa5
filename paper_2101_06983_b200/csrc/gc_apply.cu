// Step 3 of Gradient Cache for a linear encoder f(s) = W s (Section 3.3, Eq. 8; Eq. 9 for g):
// the representation gradients of one sub-batch, read from the cache, times the sub-batch's
// encoder inputs,
//
//     dW[a][b] (+)= sum_i U[i][a] X[i][b]          U: rows x d fp32 (cache slice), X: rows x d_in bf16
//
// as one tensor-core GEMM with fp32 accumulation.  The cache is fp32 and the tensor cores take
// bf16, so every u is split into two bf16 terms, hi = rn(u) and lo = rn(u - hi), whose sum
// misses u by at most 2^-17 |u|; the two terms are stacked along the contraction:
//
//     Ucat = [hi(U); lo(U)]  (2 rows x d),  Xcat = [X; X]  (2 rows x d_in),  dW = Ucat^T Xcat
//
// which is the transposed-A product of gc_gemm.cu (MN-major A, contraction split over CTAs,
// unscaled fp32 partials).  A last kernel sums the partials in part order and either overwrites
// dW (first sub-batch) or adds to it (the outer sum of Eq. 8).  No atomics: deterministic.
#include <cuda_bf16.h>

#include "gc_internal.h"

namespace gc {

namespace {

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// One thread per 4 columns of a U row (hi / lo split) or per 8 columns of an X row (two copies).
__global__ void __launch_bounds__(256)
apply_prep_kernel(const float* __restrict__ U, int64_t ldu, const __nv_bfloat16* __restrict__ X,
                  int64_t ldx, int64_t rows, int d, int d_in, __nv_bfloat16* __restrict__ Ucat,
                  __nv_bfloat16* __restrict__ Xcat) {
    const int64_t u_items = rows * (d / 4);
    const int64_t x_items = rows * (d_in / 8);
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < u_items + x_items;
         e += (int64_t)gridDim.x * blockDim.x) {
        if (e < u_items) {
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
            *reinterpret_cast<uint2*>(Ucat + i * d + c) = *reinterpret_cast<const uint2*>(hi);
            *reinterpret_cast<uint2*>(Ucat + (rows + i) * d + c) = *reinterpret_cast<const uint2*>(lo);
        } else {
            const int64_t f = e - u_items;
            const int64_t i = f / (d_in / 8);
            const int c = 8 * (int)(f - i * (d_in / 8));
            const uint4 x = *reinterpret_cast<const uint4*>(X + i * ldx + c);
            *reinterpret_cast<uint4*>(Xcat + i * d_in + c) = x;
            *reinterpret_cast<uint4*>(Xcat + (rows + i) * d_in + c) = x;
        }
    }
}

// dW[a][b] = (accumulate ? dW[a][b] : 0) + sum_g partial[g][a][b], parts in index order.
__global__ void __launch_bounds__(256)
apply_reduce_kernel(const float4* __restrict__ partial, int groups, int d, int d_in4,
                    float* __restrict__ dW, int64_t lddw, int accumulate) {
    const int64_t total = (int64_t)d * d_in4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        float4 s = partial[e];
        for (int g = 1; g < groups; ++g) {
            const float4 v = partial[(int64_t)g * total + e];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
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
    size_t off_u, off_x, off_part, total;
};

ApplyPlan make_apply_plan(int64_t rows, int d, int d_in) {
    ApplyPlan pl{};
    pl.groups = gemm_groups(d, 2 * rows, d_in);
    size_t off = 0;
    pl.off_u = off;    off += align256((size_t)2 * rows * d * sizeof(__nv_bfloat16));
    pl.off_x = off;    off += align256((size_t)2 * rows * d_in * sizeof(__nv_bfloat16));
    pl.off_part = off; off += align256((size_t)pl.groups * d * d_in * sizeof(float));
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
    __nv_bfloat16* Xcat = reinterpret_cast<__nv_bfloat16*>(w + pl.off_x);
    float* partial = reinterpret_cast<float*>(w + pl.off_part);

    const int64_t items = rows * (d / 4) + rows * (d_in / 8);
    int blocks = (int)((items + 255) / 256);
    if (blocks > 8 * sm_count()) blocks = 8 * sm_count();
    apply_prep_kernel<<<blocks, 256, 0, st>>>(U, ldu, static_cast<const __nv_bfloat16*>(X), ldx,
                                              rows, d, d_in, Ucat, Xcat);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    // Ucat is the [B x N] = [2 rows x d] operand read transposed: output rows are its columns
    if (launch_weight_gemm(Ucat, d, 2 * rows, d, 1, Xcat, d_in, d_in, pl.groups, 1.f, nullptr, 0,
                           partial, dev_status, st) != cudaSuccess)
        return GC_ERR_CUDA;
    const int64_t total = (int64_t)d * (d_in / 4);
    blocks = (int)((total + 255) / 256);
    if (blocks > 8 * sm_count()) blocks = 8 * sm_count();
    apply_reduce_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(partial), pl.groups,
                                                d, d_in / 4, dW, lddw, accumulate ? 1 : 0);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

}  // extern "C"
