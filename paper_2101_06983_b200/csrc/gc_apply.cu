// Step 3 of Gradient Cache for a linear encoder f(s) = W s (Section 3.3, Eq. 8; Eq. 9 for g):
// the representation gradients of one sub-batch, read from the cache, times the sub-batch's
// encoder inputs,
//
//     dW[a][b] (+)= sum_i U[i][a] X[i][b]          U: rows x d fp32 (cache slice), X: rows x d_in bf16
//
// in ONE launch, reading U and X once as they are.  The cache is fp32 and the tensor cores take
// bf16, so every u is used as two bf16 terms, hi = rn(u) and lo = rn(u - hi), whose sum misses u
// by at most 2^-17 |u|; both terms accumulate into the same fp32 accumulator.
//
// A CTA owns a tile of 128 output rows (columns of U) x up to 384 output columns (columns of X)
// and one part of the contraction range (the rows of the sub-batch).  Per step of 32 rows:
//   producer warp   one bulk tensor load of the fp32 U block (32 x 128) and of the X block
//                   (32 x 384, an MN-major B operand as it lies in memory);
//   4 converter warps  read the fp32 block from shared memory, form hi and lo and write them as
//                   two MN-major A operands in the 128-byte swizzle the tensor core expects;
//   MMA warp        up to 8 instructions (two steps of 16 rows, hi and lo, columns 0..255 and
//                   256..383 of the tile).
// The parts of a tile's contraction range are the CTAs of one thread-block cluster (1, 2, 4 or 8):
// every CTA owns a slice of the tile's rows, the CTAs send the rows of their accumulators to the
// owners' shared memory, and an owner adds the parts in rank order and writes (or adds to) dW.  Nothing goes through a workspace, there are no atomics on
// data, the result is deterministic, and every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include "tc_common.cuh"

namespace gc {

namespace {

constexpr int AK = 32;                         // contraction rows per pipeline step
constexpr int ATM = 128;                       // output rows per CTA = MMA M
constexpr int ATN = 384;                       // output columns per CTA (at most): MMAs of N <= 256
constexpr int A_NS = 4;                        // load stages
constexpr int A_NA = 2;                        // converted-operand stages
constexpr uint32_t BLOCK_BYTES = AK * 128;     // 32 rows of 128 bytes: one box, one operand atom
constexpr uint32_t U_STAGE = 4 * BLOCK_BYTES;  // 128 fp32 columns = 4 boxes of 32
constexpr uint32_t X_STAGE = 6 * BLOCK_BYTES;  // 384 bf16 columns = 6 boxes of 64
constexpr uint32_t LD_STAGE = U_STAGE + X_STAGE;
constexpr uint32_t A_HALF = 2 * BLOCK_BYTES;   // hi (or lo) of 128 output rows x 32
constexpr uint32_t A_STAGE = 2 * A_HALF;
constexpr int CONV_WARPS = 4;
constexpr int APPLY_PROD_WARP = CONV_WARPS;
constexpr int APPLY_MMA_WARP = CONV_WARPS + 1;
constexpr int APPLY_THREADS = 32 * (CONV_WARPS + 2);
constexpr int APPLY_TMEM_COLS = 512;
constexpr size_t APPLY_DYN_SMEM = 1024 + (size_t)A_NS * LD_STAGE + (size_t)A_NA * A_STAGE;
constexpr int MAX_SPLITS = 8;                  // portable cluster size

static_assert((size_t)ATM * ATN * 4 <= (size_t)A_NS * LD_STAGE + (size_t)A_NA * A_STAGE,
              "the accumulator copy fits the pipeline's shared memory");

static_assert(APPLY_DYN_SMEM <= SMEM_LIMIT - SMEM_STATIC_RESERVE, "shared memory budget");

struct ApplyParams {
    int64_t rows;
    int d, d_in;
    int tiles_n;              // tiles along d_in
    int splits;               // parts of the contraction range = cluster size
    float* dW;
    int64_t lddw;
    int accumulate;
    int* dev_status;
};

struct ApplyBars {
    uint64_t full[A_NS];
    uint64_t empty[A_NS];
    uint64_t a_full[A_NA];
    uint64_t a_empty[A_NA];
    uint64_t acc_full;
};

__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void st_cluster128(uint32_t cluster_addr, uint32_t a, uint32_t b,
                                              uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(cluster_addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c,
                                       uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// (x, y) -> packed bf16 pair hi and the packed pair of the rounded remainders
__device__ __forceinline__ void split2(float x, float y, uint32_t* hi, uint32_t* lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    const uint32_t hb = *reinterpret_cast<const uint32_t*>(&h);
    const float hx = __uint_as_float(hb << 16), hy = __uint_as_float(hb & 0xffff0000u);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x - hx, y - hy);
    *hi = hb;
    *lo = *reinterpret_cast<const uint32_t*>(&l);
}

__global__ void __launch_bounds__(APPLY_THREADS, 1)
apply_kernel(const __grid_constant__ CUtensorMap mapU, const __grid_constant__ CUtensorMap mapX,
             const ApplyParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) ApplyBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;

    // work item: (row tile, column tile, part of the contraction range); the parts of a tile are
    // the CTAs of one cluster
    const int split = (int)cluster_ctarank();
    const int tile = (int)(blockIdx.x / (unsigned)p.splits);
    const int m0 = (tile / p.tiles_n) * ATM;
    const int n0 = (tile % p.tiles_n) * ATN;
    const int n_cols = min(ATN, p.d_in - n0);          // a multiple of 64
    int64_t lo, hi;
    part_range((p.rows + AK - 1) / AK, p.splits, split, &lo, &hi);
    const int T = (int)(hi - lo);

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t ld_smem = base;
    const uint32_t a_smem = base + A_NS * LD_STAGE;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < A_NS; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        for (int s = 0; s < A_NA; ++s) {
            mbar_init(smem_u32(&bars.a_full[s]), CONV_WARPS);
            mbar_init(smem_u32(&bars.a_empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.acc_full), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == APPLY_MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)APPLY_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    bool acc_ok = false;

    if (warp == APPLY_PROD_WARP) {
        // ------------------------------ loads -----------------------------------------------------
        // Columns past d (of U) or rows past the sub-batch read as zeros and add nothing.
        const int atoms = n_cols / 64;
        int stage = 0;
        uint32_t phase = 0;
        for (int t = 0; t < T; ++t) {
            if (!mbar_wait(smem_u32(&bars.empty[stage]), phase ^ 1u, abort_flag)) break;
            const uint32_t full = smem_u32(&bars.full[stage]);
            const uint32_t dst = ld_smem + stage * LD_STAGE;
            const int k0 = (int)(lo + t) * AK;
            if (elect_one()) {
                mbar_expect_tx(full, U_STAGE + (uint32_t)atoms * BLOCK_BYTES);
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    tma_load_2d(dst + b * BLOCK_BYTES, &mapU, m0 + 32 * b, k0, full);
                for (int b = 0; b < atoms; ++b)
                    tma_load_2d(dst + U_STAGE + b * BLOCK_BYTES, &mapX, n0 + 64 * b, k0, full);
            }
            if (++stage == A_NS) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == APPLY_MMA_WARP) {
        // ------------------------------ MMA issuer ------------------------------------------------
        const int n1 = min(256, n_cols), n2 = n_cols - n1;        // n2 = 0, 64 or 128
        const uint32_t idesc1 = instr_desc(n1, true, ATM, true);
        const uint32_t idesc2 = instr_desc(n2 > 0 ? n2 : 64, true, ATM, true);
        constexpr uint32_t B2 = (4 * BLOCK_BYTES) >> 4;           // columns 256.. of the X block
        int s = 0, a = 0;
        uint32_t ps = 0, pa = 0;
        bool ok = true;
        for (int t = 0; t < T; ++t) {
            ok = mbar_wait(smem_u32(&bars.full[s]), ps, abort_flag) &&
                 mbar_wait(smem_u32(&bars.a_full[a]), pa, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t hi_lo = desc_lo(a_smem + a * A_STAGE, BLOCK_BYTES);
            const uint32_t lo_lo = desc_lo(a_smem + a * A_STAGE + A_HALF, BLOCK_BYTES);
            const uint32_t b_lo = desc_lo(ld_smem + s * LD_STAGE + U_STAGE, BLOCK_BYTES);
            if (elect_one()) {
#pragma unroll
                for (int k = 0; k < AK / 16; ++k) {      // 16 rows of an MN-major operand: 2 KB
                    const uint32_t ah = hi_lo + k * 128, al = lo_lo + k * 128, b = b_lo + k * 128;
                    if (t == 0 && k == 0) mma_ss<false, false>(tmem, ah, b, idesc1);
                    else                  mma_ss<true, false>(tmem, ah, b, idesc1);
                    mma_ss<true, false>(tmem, al, b, idesc1);
                    if (n2 > 0) {
                        if (t == 0 && k == 0) mma_ss<false, false>(tmem + 256, ah, b + B2, idesc2);
                        else                  mma_ss<true, false>(tmem + 256, ah, b + B2, idesc2);
                        mma_ss<true, false>(tmem + 256, al, b + B2, idesc2);
                    }
                }
                tc_commit(smem_u32(&bars.empty[s]));
                tc_commit(smem_u32(&bars.a_empty[a]));
            }
            if (++s == A_NS) { s = 0; ps ^= 1u; }
            if (++a == A_NA) { a = 0; pa ^= 1u; }
        }
        if (ok && elect_one()) tc_commit(smem_u32(&bars.acc_full));
    } else {
        // ------------------------------ converter warps -------------------------------------------
        // Item = 8 consecutive output rows m (one 16-byte piece of bf16) of contraction row k.
        // Eight neighbouring threads share k and cover one 128-byte operand row, so their stores
        // fall on distinct banks; their fp32 sources are two boxes, and the halves of a thread's
        // 32 bytes are fetched in opposite order in the two boxes so that the loads do too.
        const int tid = threadIdx.x;
        int s = 0, a = 0;
        uint32_t ps = 0, pa = 0;
        for (int t = 0; t < T; ++t) {
            if (!mbar_wait(smem_u32(&bars.full[s]), ps, abort_flag)) break;
            if (!mbar_wait(smem_u32(&bars.a_empty[a]), pa ^ 1u, abort_flag)) break;
            const uint32_t u_base = ld_smem + s * LD_STAGE;
            const uint32_t hi_base = a_smem + a * A_STAGE, lo_base = hi_base + A_HALF;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int id = tid + 128 * i;
                const int j = id & 7, atom = (id >> 3) & 1, k = id >> 4;
                const int sw = k & 7;
                const int odd = j >> 2;
                const int c = 2 * (j & 3);
                const uint32_t row = u_base + (uint32_t)(2 * atom + odd) * BLOCK_BYTES + k * 128;
                const float4 A = lds128(row + (uint32_t)(((c ^ odd) ^ sw) << 4));
                const float4 B = lds128(row + (uint32_t)(((c ^ odd ^ 1) ^ sw) << 4));
                const float4 f0 = odd ? B : A, f1 = odd ? A : B;
                uint32_t h[4], l[4];
                split2(f0.x, f0.y, &h[0], &l[0]);
                split2(f0.z, f0.w, &h[1], &l[1]);
                split2(f1.x, f1.y, &h[2], &l[2]);
                split2(f1.z, f1.w, &h[3], &l[3]);
                const uint32_t off = (uint32_t)atom * BLOCK_BYTES + k * 128 + ((j ^ sw) << 4);
                sts128(hi_base + off, h[0], h[1], h[2], h[3]);
                sts128(lo_base + off, l[0], l[1], l[2], l[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the MMAs
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.a_full[a]));
            if (++s == A_NS) { s = 0; ps ^= 1u; }
            if (++a == A_NA) { a = 0; pa ^= 1u; }
        }
        acc_ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);   // all MMAs have completed
    }

    // ------------------------------ sum over the parts -------------------------------------------
    // Rank g of the cluster owns rows [g, g + 1) * 128 / splits of the tile.  Once every CTA's
    // pipeline buffers are free (first cluster barrier) each CTA sends the rows of its accumulator
    // to their owners' shared memory, slot [sender][float4 piece q][row]; after the second barrier
    // an owner adds the senders' slots in rank order and writes (or adds to) dW.
    const int rows_per = ATM / p.splits;
    tc_fence_before();
    cluster_sync_all();            // every CTA gets here, aborted or not
    if (warp < CONV_WARPS && acc_ok) {
        tc_fence_after();
        const int r = threadIdx.x;                              // warp w reads lanes 32 w ..
        const int owner = r / rows_per, r_local = r - owner * rows_per;
        const uint32_t dst = mapa_u32(base, (uint32_t)owner) +
                             (uint32_t)((split * (ATN / 4)) * rows_per + r_local) * 16;
        const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
        for (int cb = 0; cb < n_cols / 32; ++cb) {
            uint32_t v[32];
            tmem_ld32(taddr + cb * 32, v);
            tmem_ld_wait();
#pragma unroll
            for (int q = 0; q < 8; ++q)
                st_cluster128(dst + (uint32_t)((cb * 8 + q) * rows_per) * 16, v[4 * q], v[4 * q + 1],
                              v[4 * q + 2], v[4 * q + 3]);
        }
    }
    tc_fence_before();
    cluster_sync_all();            // the slots of this CTA are complete
    if (!*abort_flag) {
        const int items = (n_cols / 4) * rows_per;
        for (int idx = threadIdx.x; idx < items; idx += APPLY_THREADS) {
            const int q = idx / rows_per;
            const int r_local = idx - q * rows_per;
            const int r = split * rows_per + r_local;
            if (m0 + r >= p.d) continue;
            const uint32_t src = base + (uint32_t)(q * rows_per + r_local) * 16;
            float4* dst = reinterpret_cast<float4*>(p.dW + (int64_t)(m0 + r) * p.lddw + n0 + 4 * q);
            float4 v[MAX_SPLITS];
#pragma unroll
            for (int g = 0; g < MAX_SPLITS; ++g)
                if (g < p.splits) v[g] = lds128(src + (uint32_t)(g * (ATN / 4) * rows_per) * 16);
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p.accumulate) sum = *dst;
#pragma unroll
            for (int g = 0; g < MAX_SPLITS; ++g)
                if (g < p.splits) { sum.x += v[g].x; sum.y += v[g].y; sum.z += v[g].z; sum.w += v[g].w; }
            *dst = sum;
        }
    }

    // ------------------------------ teardown ------------------------------------------------------
    __syncthreads();
    if (*abort_flag) {
        // let bulk copies still in flight land before the shared memory is released
        uint64_t t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, GC_DEV_WAIT_LIMIT);
        __syncthreads();
    }
    if (warp == APPLY_MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)APPLY_TMEM_COLS) : "memory");
    }
}

struct ApplyPlan {
    int tiles_m, tiles_n, splits;
};

// Parts of the contraction range = cluster size: the largest of 8, 4, 2, 1 whose clusters can
// all be resident at once (a cluster of c CTAs needs c free SMs in one GPC: about SMs / 9
// clusters of 8, SMs / 4.5 of 4, SMs / 2 of 2) with at least four steps per part.
ApplyPlan make_apply_plan(int64_t rows, int d, int d_in) {
    ApplyPlan pl{};
    pl.tiles_m = (d + ATM - 1) / ATM;
    pl.tiles_n = (d_in + ATN - 1) / ATN;
    const int64_t tiles = (int64_t)pl.tiles_m * pl.tiles_n;
    const int64_t steps = (rows + AK - 1) / AK;
    const int sms = sm_count();
    int c = 1;
    if (tiles <= sms / 2 && steps >= 8) c = 2;
    if (tiles * 2 <= sms * 4 / 9 && steps >= 16) c = 4;
    if (tiles * 9 <= sms && steps >= 32) c = 8;
    pl.splits = c;
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
    return 256;       // nothing is staged in global memory; the call accepts any such buffer
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
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < 256) return GC_ERR_WORKSPACE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return GC_ERR_CUDA;
    }
    if (major != 10) return GC_ERR_ARCH;
    if (dev < 0 || dev >= 64) return GC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    CUtensorMap mu, mx;
    if (!make_map_f32(&mu, U, rows, d, ldu, AK) || !make_map(&mx, X, rows, d_in, ldx, AK))
        return GC_ERR_CUDA;
    ApplyParams p{};
    p.rows = rows; p.d = d; p.d_in = d_in;
    p.tiles_n = pl.tiles_n; p.splits = pl.splits;
    p.dW = dW; p.lddw = lddw; p.accumulate = accumulate ? 1 : 0;
    p.dev_status = dev_status;

    static bool configured_on[64] = {false};      // the attribute belongs to (kernel, device)
    if (!configured_on[dev]) {
        if (cudaFuncSetAttribute(apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)APPLY_DYN_SMEM) != cudaSuccess) {
            cudaGetLastError();
            return GC_ERR_CUDA;
        }
        configured_on[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((int64_t)pl.tiles_m * pl.tiles_n * pl.splits));
    cfg.blockDim = dim3(APPLY_THREADS);
    cfg.dynamicSmemBytes = APPLY_DYN_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)pl.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, apply_kernel, mu, mx, p);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return GC_ERR_CUDA;
    }
    return GC_OK;
}

}  // extern "C"
