// Distance Gradient Cache (Section 5, Eq. 10-13) in tiled form.  The similarity of a pair is a
// distance d_ij = Phi(f(s_i), g(t_j)) that the caller's network computes; the loss is Eq. 1 with
// d_ij / tau as the logit.  The paper stores all B x N values w_ij = dL/dd_ij; here nothing of
// size B x N is held: the caller walks the sub-batch pairs (S^, T^) twice, as its Step 3 does
// anyway, handing over one block of distances at a time:
//
//   pass 1   gc_dist_accumulate  folds a block into the running (max, sum) of its rows and picks
//                                up the positives' distances; gc_dist_finish gives row_lse, loss
//   pass 2   gc_dist_w_block     w_ij = (exp(d_ij / tau - lse_i) - [j == r_i]) / (B tau) for the
//                                block, which Eq. 11 (parameters of Phi) and Eq. 12-13
//                                (representation gradients) consume at once
//
// For the dot product, gc_dist_dot_block forms a block of distances from the representations.
// One warp per block row, lanes strided over its columns, fixed shuffle trees: deterministic.
// HBM-bound (a block is read once per pass).
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {
namespace {

__device__ __forceinline__ float wsum(float v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float wmax(float v) {
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__global__ void __launch_bounds__(256)
dist_begin_kernel(float* __restrict__ run_m, float* __restrict__ run_l, float* __restrict__ pos_d,
                  int64_t B) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < B;
         i += (int64_t)gridDim.x * blockDim.x) {
        run_m[i] = -INFINITY;
        run_l[i] = 0.f;
        pos_d[i] = 0.f;
    }
}

__global__ void __launch_bounds__(256)
dist_accumulate_kernel(const float* __restrict__ D, int64_t ldd, int64_t i0, int64_t bq, int64_t j0,
                       int64_t bn, const int32_t* __restrict__ pos_idx, float inv_tau, int mask_mode,
                       float* __restrict__ run_m, float* __restrict__ run_l,
                       float* __restrict__ pos_d) {
    const int lane = threadIdx.x & 31;
    for (int64_t r = blockIdx.x * 8 + (threadIdx.x >> 5); r < bq; r += (int64_t)gridDim.x * 8) {
        const int64_t i = i0 + r;
        const float* row = D + r * ldd;
        const bool self = (mask_mode == GC_MASK_SELF);
        float bm = -INFINITY;
        for (int64_t c = lane; c < bn; c += 32)
            if (!(self && j0 + c == i)) bm = fmaxf(bm, row[c] * inv_tau);
        bm = wmax(bm);
        const int64_t rel = (int64_t)pos_idx[i] - j0;
        if (lane == 0 && rel >= 0 && rel < bn && !(self && j0 + rel == i)) pos_d[i] = row[rel] * inv_tau;
        if (bm == -INFINITY) continue;                       // nothing allowed in this block
        const float m_old = run_m[i];
        const float m_new = fmaxf(m_old, bm);
        float s = 0.f;
        for (int64_t c = lane; c < bn; c += 32)
            if (!(self && j0 + c == i)) s += expf(row[c] * inv_tau - m_new);
        s = wsum(s);
        if (lane == 0) {
            const float carry = m_old == -INFINITY ? 0.f : run_l[i] * expf(m_old - m_new);
            run_m[i] = m_new;
            run_l[i] = carry + s;
        }
    }
}

// row_lse, the loss (mean of lse_i - d_{i,r_i}/tau, rows summed in a fixed order by one block) and
// the validity of pos_idx
__global__ void __launch_bounds__(1024)
dist_finish_kernel(const float* __restrict__ run_m, const float* __restrict__ run_l,
                   const float* __restrict__ pos_d, const int32_t* __restrict__ pos_idx, int64_t B,
                   int64_t N, int mask_mode, float* __restrict__ row_lse, float* __restrict__ loss,
                   int* __restrict__ dev_status) {
    __shared__ float part[32];
    __shared__ int flag[32];
    float s = 0.f;
    int f = 0;
    for (int64_t i = threadIdx.x; i < B; i += 1024) {
        const float lse = run_m[i] + logf(run_l[i]);
        row_lse[i] = lse;
        const int32_t r = pos_idx[i];
        int bad = 0;
        if (r < 0 || (int64_t)r >= N) bad = GC_DEV_POS_RANGE;
        else if (mask_mode == GC_MASK_SELF && (int64_t)r == i) bad = GC_DEV_POS_MASKED;
        f |= bad;
        s += lse - (bad ? 0.f : pos_d[i]);
    }
    s = wsum(s);
    f = __reduce_or_sync(0xffffffffu, f);
    if ((threadIdx.x & 31) == 0) { part[threadIdx.x >> 5] = s; flag[threadIdx.x >> 5] = f; }
    __syncthreads();
    if (threadIdx.x < 32) {
        const float t = wsum(part[threadIdx.x]);
        const int g = __reduce_or_sync(0xffffffffu, flag[threadIdx.x]);
        if (threadIdx.x == 0) {
            *loss = t / (float)B;
            if (dev_status && g) atomicOr(dev_status, g);
        }
    }
}

__global__ void __launch_bounds__(256)
dist_w_kernel(const float* __restrict__ D, int64_t ldd, int64_t i0, int64_t bq, int64_t j0,
              int64_t bn, const int32_t* __restrict__ pos_idx, const float* __restrict__ row_lse,
              int64_t N, float inv_tau, float scale, int mask_mode, float* __restrict__ W,
              int64_t ldw) {
    const int lane = threadIdx.x & 31;
    for (int64_t r = blockIdx.x * 8 + (threadIdx.x >> 5); r < bq; r += (int64_t)gridDim.x * 8) {
        const int64_t i = i0 + r;
        const float lse = row_lse[i];
        const int32_t pr = pos_idx[i];
        const bool pos_ok = pr >= 0 && (int64_t)pr < N && !(mask_mode == GC_MASK_SELF && (int64_t)pr == i);
        for (int64_t c = lane; c < bn; c += 32) {
            const int64_t j = j0 + c;
            float w = 0.f;
            if (!(mask_mode == GC_MASK_SELF && j == i)) {
                w = expf(D[r * ldd + c] * inv_tau - lse);
                if (pos_ok && j == (int64_t)pr) w -= 1.f;
            }
            W[r * ldw + c] = w * scale;
        }
    }
}

// d_ij = <q_i, p_j> for one block: a warp per row, the row of Q in registers (d <= 1024 per pass),
// lanes over the block's passages
template <bool BF16>
__global__ void __launch_bounds__(256)
dist_dot_kernel(const void* __restrict__ Q, int64_t ldq, const void* __restrict__ P, int64_t ldp,
                int64_t i0, int64_t bq, int64_t j0, int64_t bn, int d, float* __restrict__ D,
                int64_t ldd) {
    const size_t es = BF16 ? 2 : 4;
    // one thread per (row, column) pair of the block; both rows are read with 16-byte loads
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < bq * bn;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / bn, c = e - r * bn;
        const char* q = static_cast<const char*>(Q) + (size_t)(i0 + r) * (size_t)ldq * es;
        const char* p = static_cast<const char*>(P) + (size_t)(j0 + c) * (size_t)ldp * es;
        float acc = 0.f;
        if (BF16) {
            for (int k = 0; k < d; k += 8) {
                const uint4 a = *reinterpret_cast<const uint4*>(q + 2 * k);
                const uint4 b = *reinterpret_cast<const uint4*>(p + 2 * k);
                const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
                const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float2 x = __bfloat1622float2(ah[t]), y = __bfloat1622float2(bh[t]);
                    acc = fmaf(x.x, y.x, acc);
                    acc = fmaf(x.y, y.y, acc);
                }
            }
        } else {
            for (int k = 0; k < d; k += 4) {
                const float4 x = *reinterpret_cast<const float4*>(q + 4 * k);
                const float4 y = *reinterpret_cast<const float4*>(p + 4 * k);
                acc = fmaf(x.x, y.x, acc); acc = fmaf(x.y, y.y, acc);
                acc = fmaf(x.z, y.z, acc); acc = fmaf(x.w, y.w, acc);
            }
        }
        D[r * ldd + c] = acc;
    }
}

int rows_grid(int64_t rows) {
    int64_t blocks = (rows + 7) / 8;
    const int cap = sm_count() * 8;
    return (int)(blocks > cap ? cap : (blocks < 1 ? 1 : blocks));
}

int check_block(int64_t B, int64_t N, int64_t i0, int64_t bq, int64_t j0, int64_t bn, int64_t ld) {
    if (B <= 0 || N <= 0 || bq <= 0 || bn <= 0 || i0 < 0 || j0 < 0 || i0 + bq > B || j0 + bn > N ||
        ld < bn)
        return GC_ERR_SHAPE;
    return GC_OK;
}

}  // namespace
}  // namespace gc

using namespace gc;

extern "C" {

int gc_dist_begin(float* run_m, float* run_l, float* pos_d, int64_t B, void* cuda_stream) {
    if (!run_m || !run_l || !pos_d) return GC_ERR_NULL;
    if (B <= 0) return GC_ERR_SHAPE;
    int64_t blocks = (B + 255) / 256;
    if (blocks > 1024) blocks = 1024;
    dist_begin_kernel<<<(int)blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(run_m, run_l,
                                                                                      pos_d, B);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int gc_dist_accumulate(const float* D_block, int64_t ldd, int64_t i0, int64_t bq, int64_t j0,
                       int64_t bn, const int32_t* pos_idx, int64_t B, int64_t N, float tau,
                       int mask_mode, float* run_m, float* run_l, float* pos_d, void* cuda_stream) {
    if (!D_block || !pos_idx || !run_m || !run_l || !pos_d) return GC_ERR_NULL;
    int rc = check_block(B, N, i0, bq, j0, bn, ldd);
    if (rc) return rc;
    if (!(tau > 0.f) || !isfinite(tau)) return GC_ERR_SHAPE;
    if (mask_mode != GC_MASK_NONE && mask_mode != GC_MASK_SELF) return GC_ERR_MASK;
    dist_accumulate_kernel<<<rows_grid(bq), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        D_block, ldd, i0, bq, j0, bn, pos_idx, 1.f / tau, mask_mode, run_m, run_l, pos_d);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int gc_dist_finish(const float* run_m, const float* run_l, const float* pos_d,
                   const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode, float* row_lse,
                   float* loss, int* dev_status, void* cuda_stream) {
    if (!run_m || !run_l || !pos_d || !pos_idx || !row_lse || !loss) return GC_ERR_NULL;
    if (B <= 0 || N <= 0) return GC_ERR_SHAPE;
    if (mask_mode != GC_MASK_NONE && mask_mode != GC_MASK_SELF) return GC_ERR_MASK;
    dist_finish_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        run_m, run_l, pos_d, pos_idx, B, N, mask_mode, row_lse, loss, dev_status);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int gc_dist_w_block(const float* D_block, int64_t ldd, int64_t i0, int64_t bq, int64_t j0,
                    int64_t bn, const int32_t* pos_idx, const float* row_lse, int64_t B, int64_t N,
                    float tau, int mask_mode, float* W_block, int64_t ldw, void* cuda_stream) {
    if (!D_block || !pos_idx || !row_lse || !W_block) return GC_ERR_NULL;
    int rc = check_block(B, N, i0, bq, j0, bn, ldd);
    if (rc) return rc;
    if (ldw < bn) return GC_ERR_SHAPE;
    if (!(tau > 0.f) || !isfinite(tau)) return GC_ERR_SHAPE;
    if (mask_mode != GC_MASK_NONE && mask_mode != GC_MASK_SELF) return GC_ERR_MASK;
    dist_w_kernel<<<rows_grid(bq), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        D_block, ldd, i0, bq, j0, bn, pos_idx, row_lse, N, 1.f / tau, 1.f / ((float)B * tau), mask_mode,
        W_block, ldw);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

int gc_dist_dot_block(const void* Q, int64_t ldq, const void* P, int64_t ldp, int64_t B, int64_t N,
                      int d, int dtype, int64_t i0, int64_t bq, int64_t j0, int64_t bn,
                      float* D_block, int64_t ldd, void* cuda_stream) {
    if (!Q || !P || !D_block) return GC_ERR_NULL;
    if (dtype != GC_F32 && dtype != GC_BF16) return GC_ERR_DTYPE;
    int rc = check_block(B, N, i0, bq, j0, bn, ldd);
    if (rc) return rc;
    if (d <= 0 || ldq < d || ldp < d) return GC_ERR_SHAPE;
    const int es = dtype == GC_BF16 ? 2 : 4;
    if (((uintptr_t)Q & 15) || ((uintptr_t)P & 15) || (ldq * es) % 16 || (ldp * es) % 16)
        return GC_ERR_ALIGN;
    if (d % 8 != 0) return GC_ERR_LIMIT;
    int64_t blocks = (bq * bn + 255) / 256;
    const int cap = sm_count() * 16;
    if (blocks > cap) blocks = cap;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (dtype == GC_BF16)
        dist_dot_kernel<true><<<(int)blocks, 256, 0, st>>>(Q, ldq, P, ldp, i0, bq, j0, bn, d, D_block, ldd);
    else
        dist_dot_kernel<false><<<(int)blocks, 256, 0, st>>>(Q, ldq, P, ldp, i0, bq, j0, bn, d, D_block, ldd);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

}  // extern "C"
