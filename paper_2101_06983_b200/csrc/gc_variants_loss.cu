// Two more loss variants of Section 3.3, Step 2, built around gc_build_cache:
//
//   several positives per query   loss_i = lse_i - mean_{r in R_i} S_ir, so
//       G_ij = (p_ij - [j in R_i] / |R_i|) / B.  gc_build_cache runs with the first positive of
//       every query; what differs from Eq. 1 is linear in the positives and is added in fp32:
//         loss += (1/B) sum_i (S_{i r0} - mean_r S_ir)
//         dQ_i += (P_{r0} - mean_r P_r) / (B tau)
//         dP_j += sum_i ([j = r0_i] - [j in R_i] / |R_i|) Q_i / (B tau)
//   two-direction loss   L = (L_row + L_col) / 2 with L_row = Eq. 1 and L_col its mirror image
//       over the same B positive pairs: passage r_i is the anchor and the B queries are its
//       candidates.  L_col is Eq. 1 on (A, Q) with A_i = P_{r_i} and positive i, so a second
//       gc_build_cache gives dL_col/dA and dL_col/dQ; dL_col/dA_i goes to row r_i of dP.
//
// Sums into rows of dP that several queries point at are formed by one warp in ascending query
// order (a block owns 32 passages and scans the list of (query, passage) pairs): no atomics on
// data, reproducible.
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {
namespace {

size_t align256v(size_t v) { return (v + 255) & ~(size_t)255; }

__device__ __forceinline__ float warp_sum_v(float v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
template <bool BF16>
__device__ __forceinline__ float4 load4v(const void* row, int k) {
    if (BF16) {
        const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(row) + k);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        return make_float4(a.x, a.y, b.x, b.y);
    }
    return *reinterpret_cast<const float4*>(static_cast<const float*>(row) + k);
}
template <bool BF16>
__device__ __forceinline__ const void* row_ptr(const void* base, int64_t row, int64_t ld) {
    return BF16 ? static_cast<const void*>(static_cast<const __nv_bfloat16*>(base) + row * ld)
                : static_cast<const void*>(static_cast<const float*>(base) + row * ld);
}

// One thread per query: first positive, the pair list (query of every list entry, its
// coefficient ([first] - 1/|R_i|) scale) and the checks of the list.
__global__ void __launch_bounds__(256)
multi_prepare_kernel(const int32_t* __restrict__ pos_ptr, const int32_t* __restrict__ pos_list,
                     int64_t B, int64_t N, int64_t n_pos, int mask_mode, float scale,
                     int32_t* __restrict__ pos0, int32_t* __restrict__ pair_q,
                     float* __restrict__ pair_c, int* __restrict__ dev_status) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= B) return;
    const int64_t lo = pos_ptr[i], hi = pos_ptr[i + 1];
    int flags = 0;
    if (lo < 0 || hi <= lo || hi > n_pos) {
        pos0[i] = -1;                         // gc_build_cache flags it as out of range
        flags = GC_DEV_POS_RANGE;
    } else {
        pos0[i] = pos_list[lo];
        const float inv = 1.f / (float)(hi - lo);
        for (int64_t e = lo; e < hi; ++e) {
            const int32_t r = pos_list[e];
            if (r < 0 || r >= N) flags |= GC_DEV_POS_RANGE;
            else if (mask_mode == GC_MASK_SELF && r == i) flags |= GC_DEV_POS_MASKED;
            pair_q[e] = (int32_t)i;
            pair_c[e] = ((e == lo ? 1.f : 0.f) - inv) * scale;
        }
    }
    if (flags && dev_status) atomicOr(dev_status, flags);
}

// One warp per query: S_ir for its positives (fp32 dot products), the loss correction
// corr[i] = S_{i r0} - mean_r S_ir and dQ_i += (P_{r0} - mean_r P_r) scale.
template <bool BF16>
__global__ void __launch_bounds__(256)
multi_fix_kernel(const void* __restrict__ Q, int64_t ldq, const void* __restrict__ P, int64_t ldp,
                 const int32_t* __restrict__ pos_ptr, const int32_t* __restrict__ pos_list,
                 int64_t B, int64_t N, int64_t n_pos, int d, float inv_tau, float scale,
                 float* __restrict__ dQ, int64_t lddq, float* __restrict__ corr) {
    const int lane = threadIdx.x & 31;
    const int64_t i = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= B) return;
    const int64_t lo = pos_ptr[i], hi = pos_ptr[i + 1];
    const int n = (int)(hi - lo);
    if (n <= 1 || lo < 0 || hi > n_pos) {          // one positive is Eq. 1 itself; a bad list is flagged
        if (lane == 0) corr[i] = 0.f;
        return;
    }
    const void* q = row_ptr<BF16>(Q, i, ldq);
    const float inv = 1.f / (float)n;
    float s_first = 0.f, s_sum = 0.f;
    for (int64_t e = lo; e < hi; ++e) {
        const int32_t r = pos_list[e];
        float dot = 0.f;
        if (r >= 0 && r < N) {
            const void* pr = row_ptr<BF16>(P, r, ldp);
            for (int k = 4 * lane; k < d; k += 128) {
                const float4 a = load4v<BF16>(q, k), b = load4v<BF16>(pr, k);
                dot += a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
            }
        }
        dot = warp_sum_v(dot) * inv_tau;
        if (e == lo) s_first = dot;
        s_sum += dot;
    }
    if (lane == 0) corr[i] = s_first - s_sum * inv;
    float* out = dQ + i * lddq;
    for (int k = 4 * lane; k < d; k += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int64_t e = lo; e < hi; ++e) {
            const int32_t r = pos_list[e];
            if (r < 0 || r >= N) continue;
            const float4 b = load4v<BF16>(row_ptr<BF16>(P, r, ldp), k);
            const float c = (e == lo ? 1.f : 0.f) - inv;
            acc.x += c * b.x; acc.y += c * b.y; acc.z += c * b.z; acc.w += c * b.w;
        }
        float4 o = *reinterpret_cast<float4*>(out + k);
        o.x += acc.x * scale; o.y += acc.y * scale; o.z += acc.z * scale; o.w += acc.w * scale;
        *reinterpret_cast<float4*>(out + k) = o;
    }
}

// *loss += (1/B) sum_i corr[i], summed by one block in a fixed order.
__global__ void __launch_bounds__(1024)
loss_correction_kernel(const float* __restrict__ corr, int64_t B, float* __restrict__ loss) {
    __shared__ float part[32];
    float v = 0.f;
    for (int64_t i = threadIdx.x; i < B; i += 1024) v += corr[i];
    v = warp_sum_v(v);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x < 32) {
        v = warp_sum_v(part[threadIdx.x]);
        if (threadIdx.x == 0) *loss += v / (float)B;
    }
}

// out[tgt[e], :] += coef[e] * Src[src[e], :] for every pair e with tgt[e] in [0, N), pairs of one
// target applied in ascending e by one warp (a block owns 32 targets and scans all pairs, 1024
// at a time, compacting the matches in order).  src == NULL: the source row of pair e is e.
// Pairs whose source row is outside [0, n_src) are skipped.
constexpr int kScanTile = 32;
template <int SRC>      // 0: fp32 rows, 1: bf16 rows
__global__ void __launch_bounds__(1024)
scatter_scan_kernel(const int32_t* __restrict__ tgt, const int32_t* __restrict__ src,
                    const float* __restrict__ coef, float coef_all, int64_t n_pairs, int64_t N,
                    const void* __restrict__ Src, int64_t lds, int64_t n_src, int d,
                    float* __restrict__ out, int64_t ldo) {
    __shared__ int list_e[1024];
    __shared__ int list_w[1024];
    __shared__ int warp_count[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t j0 = (int64_t)blockIdx.x * kScanTile;
    for (int64_t base = 0; base < n_pairs; base += 1024) {
        const int64_t e = base + threadIdx.x;
        bool match = false;
        int32_t r = 0;
        if (e < n_pairs) {
            r = tgt[e];
            match = r >= 0 && (int64_t)r < N && r >= j0 && r < j0 + kScanTile;
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
            list_e[slot] = (int)(e - base);
            list_w[slot] = (int)(r - j0);
        }
        __syncthreads();
        for (int m = 0; m < total; ++m) {
            if (list_w[m] != warp) continue;
            const int64_t pe = base + list_e[m];
            const int64_t srow = src ? src[pe] : pe;
            if (srow < 0 || srow >= n_src) continue;      // a list entry no query owns
            const float c = coef ? coef[pe] : coef_all;
            float* dst = out + (j0 + warp) * ldo;
            const void* s = SRC ? row_ptr<true>(Src, srow, lds) : row_ptr<false>(Src, srow, lds);
            for (int k = 4 * lane; k < d; k += 128) {
                const float4 a = SRC ? load4v<true>(s, k) : load4v<false>(s, k);
                float4 o = *reinterpret_cast<float4*>(dst + k);
                o.x += c * a.x; o.y += c * a.y; o.z += c * a.z; o.w += c * a.w;
                *reinterpret_cast<float4*>(dst + k) = o;
            }
        }
        __syncthreads();
    }
}

// A[i, :] = P[pos[i], :] (16-byte pieces; an unusable pos gives a zero row) and ident[i] = i.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ P, int64_t ldp16, const int32_t* __restrict__ pos,
                   int64_t B, int64_t N, int d16, uint4* __restrict__ A,
                   int32_t* __restrict__ ident) {
    const int64_t total = B * d16;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / d16;
        const int k = (int)(e - i * d16);
        const int32_t r = pos[i];
        A[e] = (r >= 0 && r < N) ? P[(int64_t)r * ldp16 + k] : make_uint4(0u, 0u, 0u, 0u);
        if (k == 0) ident[i] = (int32_t)i;
    }
}

// dQ = (dQ + dQ2) / 2, dP = dP / 2, loss = (loss + loss2) / 2.
__global__ void __launch_bounds__(256)
two_dir_combine_kernel(float* __restrict__ dQ, int64_t lddq, const float* __restrict__ dQ2,
                       int64_t B, float* __restrict__ dP, int64_t lddp, int64_t N, int d4,
                       float* __restrict__ loss, const float* __restrict__ loss2) {
    const int64_t nq = B * d4, total = nq + N * d4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        if (e < nq) {
            const int64_t i = e / d4;
            const int k = 4 * (int)(e - i * d4);
            float4 a = *reinterpret_cast<float4*>(dQ + i * lddq + k);
            const float4 b = *reinterpret_cast<const float4*>(dQ2 + i * (int64_t)(4 * d4) + k);
            a.x = 0.5f * (a.x + b.x); a.y = 0.5f * (a.y + b.y);
            a.z = 0.5f * (a.z + b.z); a.w = 0.5f * (a.w + b.w);
            *reinterpret_cast<float4*>(dQ + i * lddq + k) = a;
        } else {
            const int64_t f = e - nq;
            const int64_t j = f / d4;
            const int k = 4 * (int)(f - j * d4);
            float4 a = *reinterpret_cast<float4*>(dP + j * lddp + k);
            a.x *= 0.5f; a.y *= 0.5f; a.z *= 0.5f; a.w *= 0.5f;
            *reinterpret_cast<float4*>(dP + j * lddp + k) = a;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) *loss = 0.5f * (*loss + *loss2);
}

int grid_for(int64_t items, int threads) {
    int64_t blocks = (items + threads - 1) / threads;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

bool variant_args_ok(int64_t B, int64_t N, int d, int dtype) {
    return B > 0 && N > 0 && d > 0 && (dtype == GC_F32 || dtype == GC_BF16);
}

struct MultiLayout { size_t pos0, pair_q, pair_c, corr, inner, total; };
MultiLayout multi_layout(int64_t B, int64_t N, int d, int dtype, int64_t n_pos) {
    MultiLayout l{};
    size_t off = 0;
    l.pos0 = off;    off += align256v(sizeof(int32_t) * (size_t)B);
    l.pair_q = off;  off += align256v(sizeof(int32_t) * (size_t)n_pos);
    l.pair_c = off;  off += align256v(sizeof(float) * (size_t)n_pos);
    l.corr = off;    off += align256v(sizeof(float) * (size_t)B);
    l.inner = off;   off += gc_workspace_bytes(GC_OP_BUILD, B, N, d, dtype);
    l.total = off;
    return l;
}

struct TwoDirLayout { size_t A, ident, dA, dQ2, lse2, loss2, inner, total; };
TwoDirLayout two_dir_layout(int64_t B, int64_t N, int d, int dtype) {
    TwoDirLayout l{};
    const size_t es = dtype == GC_BF16 ? 2 : 4;
    size_t off = 0;
    l.A = off;      off += align256v(es * (size_t)B * (size_t)d);
    l.ident = off;  off += align256v(sizeof(int32_t) * (size_t)B);
    l.dA = off;     off += align256v(sizeof(float) * (size_t)B * (size_t)d);
    l.dQ2 = off;    off += align256v(sizeof(float) * (size_t)B * (size_t)d);
    l.lse2 = off;   off += align256v(sizeof(float) * (size_t)B);
    l.loss2 = off;  off += 256;
    const size_t w1 = gc_workspace_bytes(GC_OP_BUILD, B, N, d, dtype);
    const size_t w2 = gc_workspace_bytes(GC_OP_BUILD, B, B, d, dtype);
    l.inner = off;  off += w1 > w2 ? w1 : w2;
    l.total = off;
    return l;
}

}  // namespace
}  // namespace gc

using namespace gc;

extern "C" {

size_t gc_multi_pos_workspace_bytes(int64_t B, int64_t N, int d, int dtype, int64_t n_pos) {
    if (!variant_args_ok(B, N, d, dtype) || n_pos < B || d % 8 != 0) return 0;
    return multi_layout(B, N, d, dtype, n_pos).total;
}

int gc_build_cache_multi_pos(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                             const int32_t* pos_ptr, const int32_t* pos_list, int64_t n_pos,
                             int64_t B, int64_t N, int d, float tau, int mask_mode, int dtype,
                             float* loss, float* row_lse, float* dQ, int64_t lddq, float* dP,
                             int64_t lddp, void* ws, size_t ws_bytes, int* dev_status,
                             void* cuda_stream) {
    if (!Q || !P || !pos_ptr || !pos_list || !loss || !row_lse || !dQ || !dP) return GC_ERR_NULL;
    if (dtype != GC_F32 && dtype != GC_BF16) return GC_ERR_DTYPE;
    if (B <= 0 || N <= 0 || d <= 0 || n_pos < B || n_pos > ((int64_t)1 << 30)) return GC_ERR_SHAPE;
    if (d % 8 != 0) return GC_ERR_LIMIT;
    const MultiLayout l = multi_layout(B, N, d, dtype, n_pos);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < l.total) return GC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* w = static_cast<char*>(ws);
    int32_t* pos0 = reinterpret_cast<int32_t*>(w + l.pos0);
    int32_t* pair_q = reinterpret_cast<int32_t*>(w + l.pair_q);
    float* pair_c = reinterpret_cast<float*>(w + l.pair_c);
    float* corr = reinterpret_cast<float*>(w + l.corr);
    const float scale = 1.f / ((float)B * tau);
    // entries that no query's range covers keep the owner -1 and are skipped
    if (cudaMemsetAsync(pair_q, 0xff, sizeof(int32_t) * (size_t)n_pos, st) != cudaSuccess)
        return GC_ERR_CUDA;
    multi_prepare_kernel<<<(unsigned)((B + 255) / 256), 256, 0, st>>>(
        pos_ptr, pos_list, B, N, n_pos, mask_mode, scale, pos0, pair_q, pair_c, dev_status);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    // Eq. 1 and Eq. 5-7 with the first positive of every query (validates the remaining arguments)
    int rc = gc_build_cache(Q, ldq, P, ldp, pos0, B, N, d, tau, mask_mode, dtype, loss, row_lse,
                            nullptr, dQ, lddq, dP, lddp, w + l.inner, ws_bytes - l.inner, dev_status,
                            cuda_stream);
    if (rc) return rc;
    const int warps_per_block = 8;
    const unsigned blocks = (unsigned)((B + warps_per_block - 1) / warps_per_block);
    if (dtype == GC_BF16)
        multi_fix_kernel<true><<<blocks, 32 * warps_per_block, 0, st>>>(
            Q, ldq, P, ldp, pos_ptr, pos_list, B, N, n_pos, d, 1.f / tau, scale, dQ, lddq, corr);
    else
        multi_fix_kernel<false><<<blocks, 32 * warps_per_block, 0, st>>>(
            Q, ldq, P, ldp, pos_ptr, pos_list, B, N, n_pos, d, 1.f / tau, scale, dQ, lddq, corr);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    loss_correction_kernel<<<1, 1024, 0, st>>>(corr, B, loss);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    const unsigned sblocks = (unsigned)((N + kScanTile - 1) / kScanTile);
    if (dtype == GC_BF16)
        scatter_scan_kernel<1><<<sblocks, 1024, 0, st>>>(pos_list, pair_q, pair_c, 0.f, n_pos, N, Q,
                                                         ldq, B, d, dP, lddp);
    else
        scatter_scan_kernel<0><<<sblocks, 1024, 0, st>>>(pos_list, pair_q, pair_c, 0.f, n_pos, N, Q,
                                                         ldq, B, d, dP, lddp);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

size_t gc_two_direction_workspace_bytes(int64_t B, int64_t N, int d, int dtype) {
    if (!variant_args_ok(B, N, d, dtype) || d % 8 != 0) return 0;
    return two_dir_layout(B, N, d, dtype).total;
}

int gc_build_cache_two_direction(const void* Q, int64_t ldq, const void* P, int64_t ldp,
                                 const int32_t* pos_idx, int64_t B, int64_t N, int d, float tau,
                                 int dtype, float* loss, float* row_lse, float* dQ, int64_t lddq,
                                 float* dP, int64_t lddp, void* ws, size_t ws_bytes,
                                 int* dev_status, void* cuda_stream) {
    if (!Q || !P || !pos_idx || !loss || !row_lse || !dQ || !dP) return GC_ERR_NULL;
    if (dtype != GC_F32 && dtype != GC_BF16) return GC_ERR_DTYPE;
    if (B <= 0 || N <= 0 || d <= 0) return GC_ERR_SHAPE;
    if (d % 8 != 0) return GC_ERR_LIMIT;
    const TwoDirLayout l = two_dir_layout(B, N, d, dtype);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < l.total) return GC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* w = static_cast<char*>(ws);
    const int es = dtype == GC_BF16 ? 2 : 4;
    // row direction: Eq. 1 as it stands (validates the arguments)
    int rc = gc_build_cache(Q, ldq, P, ldp, pos_idx, B, N, d, tau, GC_MASK_NONE, dtype, loss,
                            row_lse, nullptr, dQ, lddq, dP, lddp, w + l.inner, ws_bytes - l.inner,
                            dev_status, cuda_stream);
    if (rc) return rc;
    // column direction: anchors A_i = P[r_i], candidates Q, positive i
    void* A = w + l.A;
    int32_t* ident = reinterpret_cast<int32_t*>(w + l.ident);
    float* dA = reinterpret_cast<float*>(w + l.dA);
    float* dQ2 = reinterpret_cast<float*>(w + l.dQ2);
    float* lse2 = reinterpret_cast<float*>(w + l.lse2);
    float* loss2 = reinterpret_cast<float*>(w + l.loss2);
    const int d16 = d * es / 16;
    gather_rows_kernel<<<grid_for(B * d16, 256), 256, 0, st>>>(
        static_cast<const uint4*>(P), ldp * es / 16, pos_idx, B, N, d16, static_cast<uint4*>(A),
        ident);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    rc = gc_build_cache(A, d, Q, ldq, ident, B, B, d, tau, GC_MASK_NONE, dtype, loss2, lse2, nullptr,
                        dA, d, dQ2, d, w + l.inner, ws_bytes - l.inner, dev_status, cuda_stream);
    if (rc) return rc;
    two_dir_combine_kernel<<<grid_for((B + N) * (d / 4), 256), 256, 0, st>>>(
        dQ, lddq, dQ2, B, dP, lddp, N, d / 4, loss, loss2);
    if (cudaGetLastError() != cudaSuccess) return GC_ERR_CUDA;
    // dP[r_i] += dA_i / 2, in query order
    scatter_scan_kernel<0><<<(unsigned)((N + kScanTile - 1) / kScanTile), 1024, 0, st>>>(
        pos_idx, nullptr, nullptr, 0.5f, B, N, dA, d, B, d, dP, lddp);
    return cudaGetLastError() == cudaSuccess ? GC_OK : GC_ERR_CUDA;
}

}  // extern "C"
