// Small fixed-order reductions that follow the tile sweeps: merging the per-part running
// maximum / sum into row_lse and the loss (Eq. 1), validating pos_idx, and summing the
// per-part gradient partials.  No atomics on floating-point data: results are reproducible.
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {

namespace {

constexpr int kCombineThreads = 1024;

// pos_idx[i] outside [0, N) or on the masked diagonal: flags for *dev_status, 0 when usable.
__device__ __forceinline__ int pos_flags(int32_t r, int64_t i, int64_t N, int mask_mode) {
    if (r < 0 || (int64_t)r >= N) return GC_DEV_POS_RANGE;
    if (mask_mode == GC_MASK_SELF && (int64_t)r == i) return GC_DEV_POS_MASKED;
    return 0;
}

// One block.  Thread t owns rows t, t + 1024, ...; the loss is summed per thread, then by warp
// shuffles, then over the 32 warp totals in a fixed order.
__global__ void __launch_bounds__(kCombineThreads)
lse_combine_kernel(const float* __restrict__ part_m, const float* __restrict__ part_l,
                   const float* __restrict__ pos_ws, const int32_t* __restrict__ pos_idx,
                   int groups, int64_t B, int64_t N, int mask_mode, float* __restrict__ row_lse,
                   float* __restrict__ pos_logit, float* __restrict__ loss,
                   int* __restrict__ dev_status) {
    __shared__ float warp_sum[kCombineThreads / 32];
    __shared__ int warp_flag[kCombineThreads / 32];
    float local = 0.f;
    int flags = 0;
    for (int64_t i = threadIdx.x; i < B; i += kCombineThreads) {
        float m = -INFINITY;
        for (int g = 0; g < groups; ++g) m = fmaxf(m, part_m[(int64_t)g * B + i]);
        float l = 0.f;
        for (int g = 0; g < groups; ++g) {
            float mg = part_m[(int64_t)g * B + i];
            if (mg > -INFINITY) l += part_l[(int64_t)g * B + i] * expf(mg - m);
        }
        float lse = m + logf(l);
        row_lse[i] = lse;
        int f = pos_flags(pos_idx[i], i, N, mask_mode);
        float pl = f ? 0.f : pos_ws[i];
        if (pos_logit) pos_logit[i] = pl;
        flags |= f;
        local += lse - pl;
    }
    for (int o = 16; o > 0; o >>= 1) {
        local += __shfl_xor_sync(0xffffffffu, local, o);
        flags |= __shfl_xor_sync(0xffffffffu, flags, o);
    }
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { warp_sum[warp] = local; warp_flag[warp] = flags; }
    __syncthreads();
    if (warp == 0) {
        float v = warp_sum[lane];
        int f = warp_flag[lane];
        for (int o = 16; o > 0; o >>= 1) {
            v += __shfl_xor_sync(0xffffffffu, v, o);
            f |= __shfl_xor_sync(0xffffffffu, f, o);
        }
        if (lane == 0) {
            *loss = v / (float)B;
            if (dev_status && f) atomicOr(dev_status, f);
        }
    }
}

__global__ void __launch_bounds__(256)
pos_check_kernel(const int32_t* __restrict__ pos_idx, int64_t B, int64_t N, int mask_mode,
                 int* __restrict__ dev_status) {
    int flags = 0;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < B;
         i += (int64_t)gridDim.x * blockDim.x)
        flags |= pos_flags(pos_idx[i], i, N, mask_mode);
    flags = __reduce_or_sync(0xffffffffu, flags);
    if ((threadIdx.x & 31) == 0 && flags) atomicOr(dev_status, flags);
}

// out[r][k] = scale * sum_g partial[g][r][k], groups summed in index order.  The partial
// buffer has a row pitch of 4 * d4 floats (d rounded up to a multiple of 4).
__global__ void __launch_bounds__(256)
partial_reduce_kernel(const float4* __restrict__ partial, int groups, int64_t rows, int d, int d4,
                      float scale, float* __restrict__ out, int64_t ldo) {
    int64_t total = rows * d4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        float4 s = partial[e];
        for (int g = 1; g < groups; ++g) {
            float4 v = partial[(int64_t)g * total + e];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        int64_t r = e / d4;
        int c = 4 * (int)(e - r * d4);
        float* dst = out + r * ldo + c;
        if (c + 3 < d) {
            *reinterpret_cast<float4*>(dst) =
                make_float4(s.x * scale, s.y * scale, s.z * scale, s.w * scale);
        } else {
            float v[4] = {s.x, s.y, s.z, s.w};
            for (int k = 0; k < 4; ++k)
                if (c + k < d) dst[k] = v[k] * scale;
        }
    }
}

// Finishes the fused forward + dQ sweep (Eq. 5).  partial[g][i][:] = sum_j 2^(s2_ij - m2_g) P_j
// over the part's allowed columns except the positive one; part_m holds m_g in natural-log
// units (slot 2g of the row).  dQ_i = (sum_g partial_g exp(m_g - lse_i) + (p_pos - 1) P_pos)
// / (B tau), with p_pos = exp(S_{i,r_i} - lse_i) and the positive row read exactly.  A row whose
// pos_idx is unusable gets no positive term.
__global__ void __launch_bounds__(256)
fused_dq_finalize_kernel(const float4* __restrict__ partial, int groups,
                         const float* __restrict__ part_m, const float* __restrict__ row_lse,
                         const float* __restrict__ pos_ws, const int32_t* __restrict__ pos_idx,
                         const __nv_bfloat16* __restrict__ P, int64_t ldp, int64_t B, int64_t N,
                         int d4, int mask_mode, float scale, float* __restrict__ out,
                         int64_t ldo) {
    int64_t total = B * d4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        int64_t i = e / d4;
        int c = 4 * (int)(e - i * d4);
        const float lse = row_lse[i];
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int g = 0; g < groups; ++g) {
            const float w = expf(part_m[(int64_t)(2 * g) * B + i] - lse);
            const float4 v = partial[(int64_t)g * total + e];
            acc.x = fmaf(v.x, w, acc.x); acc.y = fmaf(v.y, w, acc.y);
            acc.z = fmaf(v.z, w, acc.z); acc.w = fmaf(v.w, w, acc.w);
        }
        const int32_t r = pos_idx[i];
        if (pos_flags(r, i, N, mask_mode) == 0) {
            const float pm1 = expf(pos_ws[i] - lse) - 1.f;
            const __nv_bfloat16* pr = P + (int64_t)r * ldp + c;
            acc.x = fmaf(pm1, __bfloat162float(pr[0]), acc.x);
            acc.y = fmaf(pm1, __bfloat162float(pr[1]), acc.y);
            acc.z = fmaf(pm1, __bfloat162float(pr[2]), acc.z);
            acc.w = fmaf(pm1, __bfloat162float(pr[3]), acc.w);
        }
        *reinterpret_cast<float4*>(out + i * ldo + c) =
            make_float4(acc.x * scale, acc.y * scale, acc.z * scale, acc.w * scale);
    }
}

}  // namespace

cudaError_t launch_fused_dq_finalize(const float* partial, int groups, const float* part_m,
                                     const float* row_lse, const float* pos_ws,
                                     const int32_t* pos_idx, const void* P, int64_t ldp,
                                     int64_t B, int64_t N, int d, int mask_mode, float scale,
                                     float* out, int64_t ldo, cudaStream_t st) {
    int64_t total = B * (d / 4);
    int64_t blocks = (total + 255) / 256;
    int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    fused_dq_finalize_kernel<<<(int)blocks, 256, 0, st>>>(
        reinterpret_cast<const float4*>(partial), groups, part_m, row_lse, pos_ws, pos_idx,
        static_cast<const __nv_bfloat16*>(P), ldp, B, N, d / 4, mask_mode, scale, out, ldo);
    return cudaGetLastError();
}

cudaError_t launch_lse_combine(const float* part_m, const float* part_l, const float* pos_ws,
                               const int32_t* pos_idx, int groups, int64_t B, int64_t N,
                               int mask_mode, float* row_lse, float* pos_logit, float* loss,
                               int* dev_status, cudaStream_t st) {
    lse_combine_kernel<<<1, kCombineThreads, 0, st>>>(part_m, part_l, pos_ws, pos_idx, groups, B,
                                                      N, mask_mode, row_lse, pos_logit, loss,
                                                      dev_status);
    return cudaGetLastError();
}

cudaError_t launch_pos_check(const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode,
                             int* dev_status, cudaStream_t st) {
    int blocks = (int)((B + 255) / 256);
    if (blocks > 1024) blocks = 1024;
    pos_check_kernel<<<blocks, 256, 0, st>>>(pos_idx, B, N, mask_mode, dev_status);
    return cudaGetLastError();
}

cudaError_t launch_partial_reduce(const float* partial, int groups, int64_t rows, int d,
                                  float scale, float* out, int64_t ldo, cudaStream_t st) {
    int d4 = (d + 3) / 4;
    int64_t total = rows * d4;
    int64_t blocks = (total + 255) / 256;
    int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    partial_reduce_kernel<<<(int)blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(partial),
                                                      groups, rows, d, d4, scale, out, ldo);
    return cudaGetLastError();
}

}  // namespace gc
