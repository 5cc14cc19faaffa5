// fp32 FMA tile kernels: the plan for fp32 inputs (where one bf16 tensor-core pass cannot meet
// the 1e-4 gradient bound) and for shapes the tensor-core plan does not cover.  Same two-sweep
// structure as the tensor-core plan: a forward sweep with an online row maximum / sum, and a
// sweep that recomputes S tiles, forms the softmax-minus-onehot weights in registers and
// accumulates them against the streamed rows.  S never leaves the chip.
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {

namespace {

constexpr int TX = 64;        // stationary rows per block
constexpr int TY = 64;        // streamed rows per step
constexpr int TK = 32;        // width of one staged k chunk of the logits product
constexpr int TR = 16;        // streamed rows staged per pass of the accumulation product
constexpr int TD = 128;       // accumulator columns per block in the sweep
constexpr int PADX = TX + 4;  // row pitch of the k-major staging tiles (keeps float4 alignment)
constexpr int THREADS = 256;

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) {
    return __bfloat162float(v);
}

// Thread t fetches 8 consecutive k values (columns k0 + 8 (t % 4) ..) of row row0 + t / 4 into
// registers as float, zero outside the matrix: one or two 16-byte loads on the fast path.
template <typename T>
__device__ __forceinline__ void fetch8(const T* __restrict__ M, int64_t ld, int64_t rows, int d,
                                       int64_t row0, int k0, float (&v)[8]) {
    const int64_t row = row0 + (threadIdx.x >> 2);
    const int k = k0 + (threadIdx.x & 3) * 8;
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = 0.f;
    if (row >= rows || k >= d) return;
    const T* src = M + row * ld + k;
    if (k + 8 <= d) {
        if (sizeof(T) == 4) {
            const float4 a = *reinterpret_cast<const float4*>(src);
            const float4 b = *reinterpret_cast<const float4*>(src + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
            v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
            const uint4 u = *reinterpret_cast<const uint4*>(src);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                v[2 * e] = __uint_as_float(w[e] << 16);              // bf16 -> fp32 is a shift
                v[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
            }
        }
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (k + e < d) v[e] = to_float<T>(src[e]);
    }
}

__device__ __forceinline__ void put8(const float (&v)[8], float (*dst)[PADX]) {
    const int r = threadIdx.x >> 2, kq = (threadIdx.x & 3) * 8;
#pragma unroll
    for (int e = 0; e < 8; ++e) dst[kq + e][r] = v[e];
}

// acc[a][b] = sum_k X[x0 + 4 ty + a][k] * Y[y0 + 4 tx + b][k] over the full width d.  The next
// 32-wide k chunk is fetched into registers while the current one is multiplied.
template <typename T>
__device__ __forceinline__ void logits_tile(const T* __restrict__ X, int64_t ldx, int64_t nx,
                                            const T* __restrict__ Y, int64_t ldy, int64_t ny,
                                            int d, int64_t x0, int64_t y0, float (*Xs)[PADX],
                                            float (*Ys)[PADX], float acc[4][4]) {
    int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    float xr[8], yr[8];
    fetch8<T>(X, ldx, nx, d, x0, 0, xr);
    fetch8<T>(Y, ldy, ny, d, y0, 0, yr);
    for (int k0 = 0; k0 < d; k0 += TK) {
        __syncthreads();                      // the previous chunk has been consumed
        put8(xr, Xs);
        put8(yr, Ys);
        __syncthreads();
        if (k0 + TK < d) {
            fetch8<T>(X, ldx, nx, d, x0, k0 + TK, xr);
            fetch8<T>(Y, ldy, ny, d, y0, k0 + TK, yr);
        }
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            float4 xv = *reinterpret_cast<const float4*>(&Xs[k][ty * 4]);
            float4 yv = *reinterpret_cast<const float4*>(&Ys[k][tx * 4]);
            float xa[4] = {xv.x, xv.y, xv.z, xv.w};
            float yb[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(xa[a], yb[b], acc[a][b]);
        }
    }
}

// The contiguous range of streamed steps owned by part g of `groups`.
__device__ __forceinline__ void part_range(int64_t steps, int groups, int g, int64_t* lo,
                                           int64_t* hi) {
    int64_t base = steps / groups, rem = steps % groups;
    *lo = g * base + (g < rem ? g : rem);
    *hi = *lo + base + (g < rem ? 1 : 0);
}

// Forward sweep (Eq. 1): block (bx, g) owns 64 queries and part g of the passages.
template <typename T>
__global__ void __launch_bounds__(THREADS) simt_fwd_kernel(FwdArgs a) {
    __shared__ __align__(16) float Xs[TK][PADX];
    __shared__ __align__(16) float Ys[TK][PADX];
    const Problem& p = a.p;
    const T* Q = static_cast<const T*>(p.Q);
    const T* P = static_cast<const T*>(p.P);
    int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    int64_t i0 = (int64_t)blockIdx.x * TX;
    int g = blockIdx.y;
    float inv_tau = 1.f / p.tau;
    // the ticket word of the loss reduction that follows this sweep
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0 && a.red)
        *reinterpret_cast<int*>(a.red) = 0;

    float m[4], l[4];
    int32_t pos[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        m[r] = -INFINITY;
        l[r] = 0.f;
        int64_t i = i0 + ty * 4 + r;
        pos[r] = (i < p.B) ? p.pos_idx[i] : -1;
    }
    int64_t steps = (p.N + TY - 1) / TY, lo, hi;
    part_range(steps, a.groups, g, &lo, &hi);
    for (int64_t s = lo; s < hi; ++s) {
        int64_t j0 = s * TY;
        float acc[4][4];
        logits_tile<T>(Q, p.ldq, p.B, P, p.ldp, p.N, p.d, i0, j0, Xs, Ys, acc);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            int64_t i = i0 + ty * 4 + r;
            float v[4];
            float tile_max = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int64_t j = j0 + tx * 4 + c;
                bool ok = (j < p.N) && !(p.mask_mode == GC_MASK_SELF && i + p.mask_shift == j);
                v[c] = ok ? acc[r][c] * inv_tau : -INFINITY;
                tile_max = fmaxf(tile_max, v[c]);
                if (ok && i < p.B && j == (int64_t)pos[r]) a.pos_logit[i] = v[c];
            }
            if (tile_max > -INFINITY) {
                float m_new = fmaxf(m[r], tile_max);
                float sum = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) sum += expf(v[c] - m_new);   // exp(-inf) = 0
                l[r] = l[r] * expf(m[r] - m_new) + sum;
                m[r] = m_new;
            }
        }
    }
    // merge the 16 threads that share a row (lanes differ in tx only within a half warp)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) {
            float mo = __shfl_xor_sync(0xffffffffu, m[r], o);
            float lo_ = __shfl_xor_sync(0xffffffffu, l[r], o);
            float mn = fmaxf(m[r], mo);
            float la = (m[r] > -INFINITY) ? l[r] * expf(m[r] - mn) : 0.f;
            float lb = (mo > -INFINITY) ? lo_ * expf(mo - mn) : 0.f;
            m[r] = mn;
            l[r] = la + lb;
        }
        int64_t i = i0 + ty * 4 + r;
        if (tx == 0 && i < p.B) {
            a.part_m[(int64_t)g * p.B + i] = m[r];
            a.part_l[(int64_t)g * p.B + i] = l[r];
        }
    }
}

// Gradient sweep (Eq. 5 or Eq. 6-7): block (bx, by, g) owns 64 stationary rows, accumulator
// columns [128 by, 128 by + 128) and part g of the streamed rows.
template <typename T>
__global__ void __launch_bounds__(THREADS) simt_sweep_kernel(SweepArgs a) {
    __shared__ __align__(16) float Xs[TK][PADX];
    __shared__ __align__(16) float Ys[TK][PADX];
    __shared__ float Ws[TX][TY + 1];
    __shared__ __align__(16) float Yd[TR][TD];
    const T* X = static_cast<const T*>(a.X);
    const T* Y = static_cast<const T*>(a.Y);
    int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
    int64_t x0 = (int64_t)blockIdx.x * TX;
    int c0 = blockIdx.y * TD;
    int g = blockIdx.z;
    const bool dq = (a.mode == SWEEP_DQ);

    // per-row constants of the stationary side (query index == x in the dQ sweep)
    float lse_x[4];
    int32_t pos_x[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        int64_t x = x0 + ty * 4 + r;
        lse_x[r] = (dq && x < a.nx) ? a.row_lse[x] : 0.f;
        pos_x[r] = (dq && x < a.nx) ? a.pos_idx[x] : -1;
    }
    float out[4][8];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) out[r][c] = 0.f;

    int64_t steps = (a.ny + TY - 1) / TY, lo, hi;
    part_range(steps, a.groups, g, &lo, &hi);
    for (int64_t s = lo; s < hi; ++s) {
        int64_t y0 = s * TY;
        float acc[4][4];
        logits_tile<T>(X, a.ldx, a.nx, Y, a.ldy, a.ny, a.d, x0, y0, Xs, Ys, acc);
        float lse_y[4];
        int32_t pos_y[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            int64_t y = y0 + tx * 4 + c;
            lse_y[c] = (!dq && y < a.ny) ? a.row_lse[y] : 0.f;
            pos_y[c] = (!dq && y < a.ny) ? a.pos_idx[y] : -1;
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            int64_t x = x0 + ty * 4 + r;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int64_t y = y0 + tx * 4 + c;
                float w = 0.f;
                bool live = (x < a.nx) && (y < a.ny) && !(a.mask_mode == GC_MASK_SELF && x + a.mask_delta == y);
                if (live) {
                    float lse = dq ? lse_x[r] : lse_y[c];
                    bool hit = dq ? (y == (int64_t)pos_x[r]) : (x == (int64_t)pos_y[c]);
                    w = expf(acc[r][c] * a.inv_tau - lse) - (hit ? 1.f : 0.f);
                }
                Ws[ty * 4 + r][tx * 4 + c] = w;
            }
        }
        // out[x][c0 + 8 tx ..] += sum_y Ws[x][y] * Y[y0 + y][c0 + 8 tx ..]
        for (int yb = 0; yb < TY; yb += TR) {
            __syncthreads();   // Ws complete (first pass) / Yd free (later passes)
            {
                int r = threadIdx.x >> 4;              // 16 rows x 16 threads of 8 columns
                int cq = (threadIdx.x & 15) * 8;
                int64_t y = y0 + yb + r;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    int col = c0 + cq + e;
                    Yd[r][cq + e] = (y < a.ny && col < a.d) ? to_float<T>(Y[y * a.ldy + col]) : 0.f;
                }
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < TR; ++k) {
                float4 y0v = *reinterpret_cast<const float4*>(&Yd[k][tx * 8]);
                float4 y1v = *reinterpret_cast<const float4*>(&Yd[k][tx * 8 + 4]);
                float yv[8] = {y0v.x, y0v.y, y0v.z, y0v.w, y1v.x, y1v.y, y1v.z, y1v.w};
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    float w = Ws[ty * 4 + r][yb + k];
#pragma unroll
                    for (int c = 0; c < 8; ++c) out[r][c] = fmaf(w, yv[c], out[r][c]);
                }
            }
        }
    }
    // write: final values (scaled) or this part's unscaled partial
    const bool final_out = (a.groups == 1);
    int dpad = (a.d + 3) & ~3;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        int64_t x = x0 + ty * 4 + r;
        if (x >= a.nx) continue;
        float* dst = final_out ? a.out + x * a.ldo
                               : a.partial + ((int64_t)g * a.nx + x) * dpad;
        float sc = final_out ? a.out_scale : 1.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            int col = c0 + tx * 8 + c;
            if (col < (final_out ? a.d : dpad)) dst[col] = (col < a.d) ? out[r][c] * sc : 0.f;
        }
    }
}

}  // namespace

int simt_fwd_groups(int64_t B, int64_t N) {
    int64_t tiles = (B + TX - 1) / TX, steps = (N + TY - 1) / TY;
    int64_t want = (2LL * sm_count() + tiles - 1) / tiles;
    int64_t g = want < 1 ? 1 : want;
    if (g > steps) g = steps;
    if (g > 32) g = 32;
    return (int)g;
}

int simt_sweep_groups(int64_t nx, int64_t ny, int d) {
    int64_t units = ((nx + TX - 1) / TX) * ((d + TD - 1) / TD), steps = (ny + TY - 1) / TY;
    int64_t want = (2LL * sm_count() + units - 1) / units;
    int64_t g = want < 1 ? 1 : want;
    if (g > steps) g = steps;
    if (g > 8) g = 8;
    return (int)g;
}

cudaError_t simt_launch_fwd(const FwdArgs& a, cudaStream_t st) {
    dim3 grid((unsigned)((a.p.B + TX - 1) / TX), (unsigned)a.groups);
    if (a.p.dtype == GC_BF16)
        simt_fwd_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(a);
    else
        simt_fwd_kernel<float><<<grid, THREADS, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t simt_launch_sweep(const SweepArgs& a, cudaStream_t st) {
    dim3 grid((unsigned)((a.nx + TX - 1) / TX), (unsigned)((a.d + TD - 1) / TD),
              (unsigned)a.groups);
    if (a.dtype == GC_BF16)
        simt_sweep_kernel<__nv_bfloat16><<<grid, THREADS, 0, st>>>(a);
    else
        simt_sweep_kernel<float><<<grid, THREADS, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace gc
