// Loss variants around the Step 2 sweeps (Section 3.3: the loss on the stored representations may
// vary; the paper leaves its derivative to automatic differentiation).  Two of them need nothing
// from the sweeps but their inputs and outputs:
//
//   cosine similarity    S_ij = <q_i/|q_i|, p_j/|p_j|> / tau.  gc_row_normalize forms the unit rows
//                        the sweeps then see; gc_cosine_bwd takes the gradient with respect to the
//                        unit rows back through the normalisation, dx = (g - n <n, g>) / |x|.
//   learnable tau        dL/dtau = -(1/tau) sum_ij G_ij S_ij = -(1/tau) sum_i <q_i, dQ_i>, because
//                        <q_i, dQ_i> = sum_j G_ij <q_i, p_j> / tau (Eq. 5).  gc_dtau reduces the
//                        cache rows against the rows they belong to, in a fixed order.
//
// All three are bound by HBM traffic: one warp per row, 16-byte loads, fp32 arithmetic.
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// element k .. k + 3 of a row as floats (d is a multiple of 4; rows start on 16-byte boundaries)
template <bool BF16>
__device__ __forceinline__ float4 load4(const void* row, int k) {
    if (BF16) {
        const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(row) + k);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        return make_float4(a.x, a.y, b.x, b.y);
    }
    return *reinterpret_cast<const float4*>(static_cast<const float*>(row) + k);
}
template <bool BF16>
__device__ __forceinline__ void store4(void* row, int k, float4 v) {
    if (BF16) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
        uint2 raw;
        raw.x = *reinterpret_cast<uint32_t*>(&a);
        raw.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(row) + k) = raw;
    } else {
        *reinterpret_cast<float4*>(static_cast<float*>(row) + k) = v;
    }
}

template <bool BF16>
__global__ void __launch_bounds__(256)
row_normalize_kernel(const void* __restrict__ X, int64_t ldx, int64_t rows, int d,
                     void* __restrict__ Xn, int64_t ldxn, float* __restrict__ inv_norm) {
    const int lane = threadIdx.x & 31;
    const size_t es = BF16 ? 2 : 4;
    for (int64_t i = blockIdx.x * 8 + (threadIdx.x >> 5); i < rows; i += (int64_t)gridDim.x * 8) {
        const char* src = static_cast<const char*>(X) + (size_t)i * (size_t)ldx * es;
        float ss = 0.f;
        for (int k = 4 * lane; k < d; k += 128) {
            const float4 v = load4<BF16>(src, k);
            ss = fmaf(v.x, v.x, ss); ss = fmaf(v.y, v.y, ss);
            ss = fmaf(v.z, v.z, ss); ss = fmaf(v.w, v.w, ss);
        }
        ss = warp_sum(ss);
        const float inv = ss > 0.f ? 1.0f / sqrtf(ss) : 0.f;       // a zero row stays zero
        if (lane == 0) inv_norm[i] = inv;
        char* dst = static_cast<char*>(Xn) + (size_t)i * (size_t)ldxn * es;
        for (int k = 4 * lane; k < d; k += 128) {
            const float4 v = load4<BF16>(src, k);
            store4<BF16>(dst, k, make_float4(v.x * inv, v.y * inv, v.z * inv, v.w * inv));
        }
    }
}

// dX_i = inv_i (g_i - n_i <n_i, g_i>) with n_i = inv_i x_i formed in fp32 from the original row
template <bool BF16>
__global__ void __launch_bounds__(256)
cosine_bwd_kernel(const void* __restrict__ X, int64_t ldx, const float* __restrict__ inv_norm,
                  const float* G, int64_t ldg, int64_t rows, int d, float* dX, int64_t lddx) {
    const int lane = threadIdx.x & 31;
    const size_t es = BF16 ? 2 : 4;
    for (int64_t i = blockIdx.x * 8 + (threadIdx.x >> 5); i < rows; i += (int64_t)gridDim.x * 8) {
        const char* src = static_cast<const char*>(X) + (size_t)i * (size_t)ldx * es;
        const float* g = G + i * ldg;
        const float inv = inv_norm[i];
        float dot = 0.f;
        for (int k = 4 * lane; k < d; k += 128) {
            const float4 x = load4<BF16>(src, k);
            const float4 gv = *reinterpret_cast<const float4*>(g + k);
            dot = fmaf(x.x * inv, gv.x, dot); dot = fmaf(x.y * inv, gv.y, dot);
            dot = fmaf(x.z * inv, gv.z, dot); dot = fmaf(x.w * inv, gv.w, dot);
        }
        dot = warp_sum(dot);
        float* out = dX + i * lddx;
        for (int k = 4 * lane; k < d; k += 128) {
            const float4 x = load4<BF16>(src, k);
            const float4 gv = *reinterpret_cast<const float4*>(g + k);
            float4 o;
            o.x = inv * (gv.x - x.x * inv * dot); o.y = inv * (gv.y - x.y * inv * dot);
            o.z = inv * (gv.z - x.z * inv * dot); o.w = inv * (gv.w - x.w * inv * dot);
            *reinterpret_cast<float4*>(out + k) = o;
        }
    }
}

// row_dot[i] = <q_i, dQ_i>
template <bool BF16>
__global__ void __launch_bounds__(256)
row_dot_kernel(const void* __restrict__ Q, int64_t ldq, const float* __restrict__ dQ, int64_t lddq,
               int64_t rows, int d, float* __restrict__ row_dot) {
    const int lane = threadIdx.x & 31;
    const size_t es = BF16 ? 2 : 4;
    for (int64_t i = blockIdx.x * 8 + (threadIdx.x >> 5); i < rows; i += (int64_t)gridDim.x * 8) {
        const char* src = static_cast<const char*>(Q) + (size_t)i * (size_t)ldq * es;
        const float* g = dQ + i * lddq;
        float dot = 0.f;
        for (int k = 4 * lane; k < d; k += 128) {
            const float4 x = load4<BF16>(src, k);
            const float4 gv = *reinterpret_cast<const float4*>(g + k);
            dot = fmaf(x.x, gv.x, dot); dot = fmaf(x.y, gv.y, dot);
            dot = fmaf(x.z, gv.z, dot); dot = fmaf(x.w, gv.w, dot);
        }
        dot = warp_sum(dot);
        if (lane == 0) row_dot[i] = dot;
    }
}
// *out = scale * sum_i v[i]: one block, every thread a fixed strided share, then fixed trees
__global__ void __launch_bounds__(1024)
ordered_sum_kernel(const float* __restrict__ v, int64_t n, float scale, float* __restrict__ out) {
    __shared__ float part[32];
    float s = 0.f;
    for (int64_t i = threadIdx.x; i < n; i += 1024) s += v[i];
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        float t = warp_sum(part[threadIdx.x]);
        if (threadIdx.x == 0) *out = t * scale;
    }
}

int grid_for(int64_t rows) {
    int64_t blocks = (rows + 7) / 8;
    const int cap = sm_count() * 8;
    return (int)(blocks > cap ? cap : blocks);
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

int check_rows(const void* X, int64_t ldx, int64_t rows, int d, int dtype) {
    if (!X) return GC_ERR_NULL;
    if (dtype != GC_F32 && dtype != GC_BF16) return GC_ERR_DTYPE;
    if (rows <= 0 || d <= 0 || ldx < d) return GC_ERR_SHAPE;
    const int es = dtype == GC_BF16 ? 2 : 4;
    if (!aligned16(X) || (ldx * es) % 16 != 0) return GC_ERR_ALIGN;
    if (d % 8 != 0) return GC_ERR_LIMIT;
    return GC_OK;
}
int check_f32(const float* X, int64_t ldx, int d) {
    if (!X) return GC_ERR_NULL;
    if (ldx < d) return GC_ERR_SHAPE;
    if (!aligned16(X) || (ldx * 4) % 16 != 0) return GC_ERR_ALIGN;
    return GC_OK;
}

}  // namespace
}  // namespace gc

using namespace gc;

extern "C" {

int gc_row_normalize(const void* X, int64_t ldx, int64_t rows, int d, int dtype, void* Xn,
                     int64_t ldxn, float* inv_norm, void* cuda_stream) {
    int rc = check_rows(X, ldx, rows, d, dtype);
    if (rc) return rc;
    if ((rc = check_rows(Xn, ldxn, rows, d, dtype))) return rc;
    if (!inv_norm) return GC_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (dtype == GC_BF16)
        row_normalize_kernel<true><<<grid_for(rows), 256, 0, st>>>(X, ldx, rows, d, Xn, ldxn, inv_norm);
    else
        row_normalize_kernel<false><<<grid_for(rows), 256, 0, st>>>(X, ldx, rows, d, Xn, ldxn, inv_norm);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int gc_cosine_bwd(const void* X, int64_t ldx, int64_t rows, int d, int dtype, const float* inv_norm,
                  const float* dXn, int64_t lddxn, float* dX, int64_t lddx, void* cuda_stream) {
    int rc = check_rows(X, ldx, rows, d, dtype);
    if (rc) return rc;
    if (!inv_norm) return GC_ERR_NULL;
    if ((rc = check_f32(dXn, lddxn, d))) return rc;
    if ((rc = check_f32(dX, lddx, d))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (dtype == GC_BF16)
        cosine_bwd_kernel<true><<<grid_for(rows), 256, 0, st>>>(X, ldx, inv_norm, dXn, lddxn, rows, d,
                                                               dX, lddx);
    else
        cosine_bwd_kernel<false><<<grid_for(rows), 256, 0, st>>>(X, ldx, inv_norm, dXn, lddxn, rows,
                                                                d, dX, lddx);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

size_t gc_dtau_workspace_bytes(int64_t B) {
    return B > 0 ? (((size_t)B * sizeof(float)) + 255) & ~(size_t)255 : 0;
}

int gc_dtau(const void* Q, int64_t ldq, const float* dQ, int64_t lddq, int64_t B, int d, float tau,
            int dtype, float* dtau, void* ws, size_t ws_bytes, void* cuda_stream) {
    int rc = check_rows(Q, ldq, B, d, dtype);
    if (rc) return rc;
    if ((rc = check_f32(dQ, lddq, d))) return rc;
    if (!dtau) return GC_ERR_NULL;
    if (!(tau > 0.f) || !isfinite(tau)) return GC_ERR_SHAPE;
    if (!ws || ((uintptr_t)ws & 255) != 0 || ws_bytes < gc_dtau_workspace_bytes(B)) return GC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    float* row_dot = static_cast<float*>(ws);
    if (dtype == GC_BF16)
        row_dot_kernel<true><<<grid_for(B), 256, 0, st>>>(Q, ldq, dQ, lddq, B, d, row_dot);
    else
        row_dot_kernel<false><<<grid_for(B), 256, 0, st>>>(Q, ldq, dQ, lddq, B, d, row_dot);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    ordered_sum_kernel<<<1, 1024, 0, st>>>(row_dot, B, -1.f / tau, dtau);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

}  // extern "C"
