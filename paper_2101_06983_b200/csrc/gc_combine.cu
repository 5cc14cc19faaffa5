// Small fixed-order reductions that follow the tile sweeps: merging the per-part running
// maximum / sum into row_lse and the loss (Eq. 1), validating pos_idx, and summing the
// per-part gradient partials.  No atomics on floating-point data: results are reproducible.
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {

namespace {

constexpr int kCombineThreads = 256;
constexpr int kRedPartials = 64;     // float offset of the per-block sums in the scratch

// pos_idx[i] outside [0, N) or on the masked diagonal: flags for *dev_status, 0 when usable.
__device__ __forceinline__ int pos_flags(int32_t r, int64_t i, int64_t N, int mask_mode,
                                         int64_t shift) {
    if (r < 0 || (int64_t)r >= N) return GC_DEV_POS_RANGE;
    if (mask_mode == GC_MASK_SELF && (int64_t)r == i + shift) return GC_DEV_POS_MASKED;
    return 0;
}

// Rows are dealt to the threads of all blocks in a fixed pattern; a block sums its loss terms per
// thread, by warp shuffles and over its warp totals, and leaves the result in red[64 + block].
// The block that draws the last ticket (red[0], cleared by the sweep before this kernel, and put
// back to 0 here) adds the block sums in index order: the loss does not depend on block timing.
__global__ void __launch_bounds__(kCombineThreads)
lse_combine_kernel(const float* __restrict__ part_m, const float* __restrict__ part_l,
                   const float* __restrict__ pos_ws, const int32_t* __restrict__ pos_idx,
                   int groups, int64_t B, int64_t N, int mask_mode, float* __restrict__ row_lse,
                   float* __restrict__ pos_logit, float* __restrict__ loss, float* red,
                   int* __restrict__ dev_status, const Gate gate, int64_t mean_over,
                   int64_t mask_shift) {
    if (gate_closed(gate)) return;
    __shared__ float warp_sum[kCombineThreads / 32];
    __shared__ int warp_flag[kCombineThreads / 32];
    __shared__ int is_last;
    float local = 0.f;
    int flags = 0;
    for (int64_t i = blockIdx.x * (int64_t)kCombineThreads + threadIdx.x; i < B;
         i += (int64_t)gridDim.x * kCombineThreads) {
        const float lse = combined_lse(part_m, part_l, groups, B, i);
        row_lse[i] = lse;
        int f = pos_flags(pos_idx[i], i, N, mask_mode, mask_shift);
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
        float v = lane < kCombineThreads / 32 ? warp_sum[lane] : 0.f;
        int f = lane < kCombineThreads / 32 ? warp_flag[lane] : 0;
        for (int o = 16; o > 0; o >>= 1) {
            v += __shfl_xor_sync(0xffffffffu, v, o);
            f |= __shfl_xor_sync(0xffffffffu, f, o);
        }
        if (lane == 0) {
            if (dev_status && f) atomicOr(dev_status, f);
            red[kRedPartials + blockIdx.x] = v;
            __threadfence();
            is_last = atomicAdd(reinterpret_cast<int*>(red), 1) == (int)gridDim.x - 1;
        }
    }
    __syncthreads();
    if (is_last && warp == 0) {
        __threadfence();
        float v = 0.f;
        for (int b = lane; b < (int)gridDim.x; b += 32) v += __ldcg(red + kRedPartials + b);
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) {
            *loss = v / (float)mean_over;
            *reinterpret_cast<int*>(red) = 0;
        }
    }
}

__global__ void __launch_bounds__(256)
pos_check_kernel(const int32_t* __restrict__ pos_idx, int64_t B, int64_t N, int mask_mode,
                 int* __restrict__ dev_status, int64_t mask_shift) {
    int flags = 0;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < B;
         i += (int64_t)gridDim.x * blockDim.x)
        flags |= pos_flags(pos_idx[i], i, N, mask_mode, mask_shift);
    flags = __reduce_or_sync(0xffffffffu, flags);
    if ((threadIdx.x & 31) == 0 && flags) atomicOr(dev_status, flags);
}

// out[r][k] = scale * sum_g partial[g][r][k], groups summed in index order.  The partial
// buffer has a row pitch of 4 * d4 floats (d rounded up to a multiple of 4).
__global__ void __launch_bounds__(256)
partial_reduce_kernel(const float4* __restrict__ partial, int groups, int64_t rows, int d, int d4,
                      float scale, float* __restrict__ out, int64_t ldo,
                      const Gate gate) {
    if (gate_closed(gate)) return;
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
// pos_idx is unusable gets no positive term.  With row_ref2 (one anchor per row, log2 domain,
// shared by all parts) the weight of every part is 2^(row_ref2_i - lse_i log2 e) instead.
__global__ void __launch_bounds__(256)
fused_dq_finalize_kernel(const float4* __restrict__ partial, int groups,
                         const float* __restrict__ part_m, const float* __restrict__ row_ref2,
                         const float* __restrict__ row_lse,
                         const float* __restrict__ pos_ws, const int32_t* __restrict__ pos_idx,
                         const __nv_bfloat16* __restrict__ P, int64_t ldp, int64_t B, int64_t N,
                         int d4, int mask_mode, float scale, float* __restrict__ out,
                         int64_t ldo, const Gate gate, int64_t mask_shift) {
    if (gate_closed(gate)) return;
    int64_t total = B * d4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        int64_t i = e / d4;
        int c = 4 * (int)(e - i * d4);
        const float lse = row_lse[i];
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int g = 0; g < groups; ++g) {
            const float w = row_ref2 ? exp2f(row_ref2[i] - lse * 1.4426950408889634f)
                                     : expf(part_m[(int64_t)(2 * g) * B + i] - lse);
            const float4 v = partial[(int64_t)g * total + e];
            acc.x = fmaf(v.x, w, acc.x); acc.y = fmaf(v.y, w, acc.y);
            acc.z = fmaf(v.z, w, acc.z); acc.w = fmaf(v.w, w, acc.w);
        }
        const int32_t r = pos_idx[i];
        if (pos_flags(r, i, N, mask_mode, mask_shift) == 0) {
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


// Anchor of the stored weights (log2 domain): the positive logit of each query, the value its
// softmax terms are measured against.  One warp per query, fixed summation order.  Queries
// whose pos_idx is unusable get 0.  Block 0 also clears the range flag of the sweep that follows.
__global__ void __launch_bounds__(256)
pos_anchor_kernel(const __nv_bfloat16* __restrict__ Q, int64_t ldq,
                  const __nv_bfloat16* __restrict__ P, int64_t ldp,
                  const int32_t* __restrict__ pos_idx, int64_t B, int64_t N, int d, int mask_mode,
                  float c1, float* __restrict__ ref2, int* __restrict__ range_flag,
                  int64_t mask_shift) {
    dep_release();      // the sweep that follows may start; it waits for this grid before it reads ref2
    if (blockIdx.x == 0 && threadIdx.x == 0) *range_flag = 0;
    const int lane = threadIdx.x & 31;
    for (int64_t i = blockIdx.x * 8 + (threadIdx.x >> 5); i < B; i += (int64_t)gridDim.x * 8) {
        const int32_t r = pos_idx[i];
        float acc = 0.f;
        if (pos_flags(r, i, N, mask_mode, mask_shift) == 0) {
            const uint4* q = reinterpret_cast<const uint4*>(Q + i * ldq);
            const uint4* pp = reinterpret_cast<const uint4*>(P + (int64_t)r * ldp);
            for (int c = lane; c < d / 8; c += 32) {        // 8 elements per load; d % 8 == 0
                const uint4 qa = q[c], pa = pp[c];
                const __nv_bfloat162* qh = reinterpret_cast<const __nv_bfloat162*>(&qa);
                const __nv_bfloat162* ph = reinterpret_cast<const __nv_bfloat162*>(&pa);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float2 a = __bfloat1622float2(qh[k]), b = __bfloat1622float2(ph[k]);
                    acc = fmaf(a.x, b.x, acc);
                    acc = fmaf(a.y, b.y, acc);
                }
            }
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        }
        if (lane == 0) ref2[i] = acc * c1;
    }
}

// Qs[i, :] = bf16(2^(ref2_i - lse_i log2 e) Q[i, :]): with it W~_ij Qs_i = p_ij Q_i.  d is a
// multiple of 8; Qs has row pitch d.
__global__ void __launch_bounds__(256)
scale_rows_kernel(const __nv_bfloat16* __restrict__ Q, int64_t ldq, int64_t B, int d8,
                  const float* __restrict__ ref2, const float* __restrict__ row_lse,
                  __nv_bfloat16* __restrict__ Qs) {
    const int64_t total = B * d8;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / d8;
        const int c = 8 * (int)(e - i * d8);
        const float a = exp2f(ref2[i] - row_lse[i] * 1.4426950408889634f);
        uint4 raw = *reinterpret_cast<const uint4*>(Q + i * ldq + c);
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 v = __bfloat1622float2(h[k]);
            h[k] = __floats2bfloat162_rn(v.x * a, v.y * a);
        }
        *reinterpret_cast<uint4*>(Qs + i * (int64_t)(8 * d8) + c) = raw;
    }
}

// The positive-column term of Eq. 6-7 in fp32: dP[r_i, :] += scale (p_i,r_i - 1) Q_i for every
// query with a usable pos_idx.  A block owns 32 passages, one per warp, and scans all queries in
// index order (1024 at a time, matches compacted in that order); each warp then walks the matches
// and applies those of its own passage, so the sum of a passage that is the positive of several
// queries is formed in ascending query order, by one warp: reproducible, no atomics.
constexpr int kPosTile = 32;
__global__ void __launch_bounds__(1024)
dp_positive_kernel(const int32_t* __restrict__ pos_idx, int64_t B, int64_t N, int mask_mode,
                   const float* __restrict__ pos_ws, const float* __restrict__ row_lse,
                   const __nv_bfloat16* __restrict__ Q, int64_t ldq, int d, float scale,
                   float* __restrict__ out, int64_t ldo, int64_t mask_shift) {
    __shared__ int list_i[1024];
    __shared__ int list_w[1024];
    __shared__ int warp_count[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t j0 = (int64_t)blockIdx.x * kPosTile;
    for (int64_t base = 0; base < B; base += 1024) {
        const int64_t i = base + threadIdx.x;
        bool match = false;
        int32_t r = 0;
        if (i < B) {
            r = pos_idx[i];
            match = pos_flags(r, i, N, mask_mode, mask_shift) == 0 && r >= j0 && r < j0 + kPosTile;
        }
        const unsigned ballot = __ballot_sync(0xffffffffu, match);
        if (lane == 0) warp_count[warp] = __popc(ballot);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < 32; ++w) {
            const int c = warp_count[w];
            if (w < warp) before += c;
            total += c;
        }
        if (match) {
            const int slot = before + __popc(ballot & ((1u << lane) - 1u));
            list_i[slot] = (int)(i - base);
            list_w[slot] = (int)(r - j0);
        }
        __syncthreads();
        for (int m = 0; m < total; ++m) {
            if (list_w[m] != warp) continue;
            const int64_t qi = base + list_i[m];
            const float coef = scale * (expf(pos_ws[qi] - row_lse[qi]) - 1.f);
            const __nv_bfloat16* q = Q + qi * ldq;
            float* dst = out + (j0 + warp) * ldo;
            for (int c = 4 * lane; c < d; c += 128) {
                const uint2 raw = *reinterpret_cast<const uint2*>(q + c);
                const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                float4 v = *reinterpret_cast<float4*>(dst + c);
                v.x = fmaf(coef, a.x, v.x); v.y = fmaf(coef, a.y, v.y);
                v.z = fmaf(coef, b.x, v.z); v.w = fmaf(coef, b.y, v.w);
                *reinterpret_cast<float4*>(dst + c) = v;
            }
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_pos_anchor(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                              const int32_t* pos_idx, int64_t B, int64_t N, int d, int mask_mode,
                              float c1, float* ref2, int* range_flag, cudaStream_t st,
                              int64_t mask_shift) {
    int64_t blocks = (B + 7) / 8;
    int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    pos_anchor_kernel<<<(int)blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(Q), ldq,
                                                  static_cast<const __nv_bfloat16*>(P), ldp,
                                                  pos_idx, B, N, d, mask_mode, c1, ref2,
                                                  range_flag, mask_shift);
    return cudaGetLastError();
}

cudaError_t launch_scale_rows(const void* Q, int64_t ldq, int64_t B, int d, const float* ref2,
                              const float* row_lse, void* Qs, cudaStream_t st) {
    int64_t total = B * (d / 8);
    int64_t blocks = (total + 255) / 256;
    int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    scale_rows_kernel<<<(int)blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(Q), ldq, B,
                                                  d / 8, ref2, row_lse,
                                                  static_cast<__nv_bfloat16*>(Qs));
    return cudaGetLastError();
}

cudaError_t launch_dp_positive(const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode,
                               const float* pos_ws, const float* row_lse, const void* Q,
                               int64_t ldq, int d, float scale, float* out, int64_t ldo,
                               cudaStream_t st, int64_t mask_shift) {
    const int64_t blocks = (N + kPosTile - 1) / kPosTile;
    dp_positive_kernel<<<(unsigned)blocks, 1024, 0, st>>>(pos_idx, B, N, mask_mode, pos_ws, row_lse,
                                                         static_cast<const __nv_bfloat16*>(Q), ldq,
                                                         d, scale, out, ldo, mask_shift);
    return cudaGetLastError();
}

cudaError_t launch_fused_dq_finalize(const float* partial, int groups, const float* part_m,
                                     const float* row_ref2, const float* row_lse,
                                     const float* pos_ws, const int32_t* pos_idx, const void* P,
                                     int64_t ldp, int64_t B, int64_t N, int d, int mask_mode,
                                     float scale, float* out, int64_t ldo, Gate gate,
                                     cudaStream_t st, int64_t mask_shift) {
    int64_t total = B * (d / 4);
    int64_t blocks = (total + 255) / 256;
    int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    fused_dq_finalize_kernel<<<(int)blocks, 256, 0, st>>>(
        reinterpret_cast<const float4*>(partial), groups, part_m, row_ref2, row_lse, pos_ws,
        pos_idx, static_cast<const __nv_bfloat16*>(P), ldp, B, N, d / 4, mask_mode, scale, out, ldo,
        gate, mask_shift);
    return cudaGetLastError();
}

cudaError_t launch_lse_combine(const float* part_m, const float* part_l, const float* pos_ws,
                               const int32_t* pos_idx, int groups, int64_t B, int64_t N,
                               int mask_mode, float* row_lse, float* pos_logit, float* loss,
                               float* red, int* dev_status, Gate gate, cudaStream_t st,
                               int64_t mean_over, int64_t mask_shift) {
    int64_t blocks = (B + kCombineThreads - 1) / kCombineThreads;
    if (blocks > sm_count()) blocks = sm_count();
    if (blocks > 256) blocks = 256;          // the scratch holds this many block sums
    lse_combine_kernel<<<(int)blocks, kCombineThreads, 0, st>>>(part_m, part_l, pos_ws, pos_idx,
                                                               groups, B, N, mask_mode, row_lse,
                                                               pos_logit, loss, red, dev_status,
                                                               gate, mean_over > 0 ? mean_over : B,
                                                               mask_shift);
    return cudaGetLastError();
}

namespace {
// out[i] = pos_idx[i] - first when that lies in [0, count), else -1 (matches no row).
__global__ void __launch_bounds__(256)
shift_pos_kernel(const int32_t* __restrict__ pos_idx, int64_t B, int64_t first, int64_t count,
                 int32_t* __restrict__ out) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < B;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = (int64_t)pos_idx[i] - first;
        out[i] = (r >= 0 && r < count) ? (int32_t)r : -1;
    }
}
}  // namespace

cudaError_t launch_shift_pos(const int32_t* pos_idx, int64_t B, int64_t first, int64_t count,
                             int32_t* out, cudaStream_t st) {
    int64_t blocks = (B + 255) / 256;
    if (blocks > 4 * sm_count()) blocks = 4 * sm_count();
    shift_pos_kernel<<<(int)blocks, 256, 0, st>>>(pos_idx, B, first, count, out);
    return cudaGetLastError();
}

cudaError_t launch_pos_check(const int32_t* pos_idx, int64_t B, int64_t N, int mask_mode,
                             int* dev_status, cudaStream_t st, int64_t mask_shift) {
    int blocks = (int)((B + 255) / 256);
    if (blocks > 1024) blocks = 1024;
    pos_check_kernel<<<blocks, 256, 0, st>>>(pos_idx, B, N, mask_mode, dev_status, mask_shift);
    return cudaGetLastError();
}

cudaError_t launch_partial_reduce(const float* partial, int groups, int64_t rows, int d,
                                  float scale, float* out, int64_t ldo, Gate gate,
                                  cudaStream_t st) {
    int d4 = (d + 3) / 4;
    int64_t total = rows * d4;
    int64_t blocks = (total + 255) / 256;
    int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    partial_reduce_kernel<<<(int)blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(partial),
                                                      groups, rows, d, d4, scale, out, ldo,
                                                      gate);
    return cudaGetLastError();
}

}  // namespace gc
