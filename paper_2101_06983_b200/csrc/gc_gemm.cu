// The two products that follow a forward sweep which stored the bf16 weights W~ [B x N]
// (W~_ij = 2^(s2_ij - ref2_i), 0 at masked pairs and at the positive column):
//
//   dQ part (Eq. 5):    acc[i, :] = sum_j W~_ij P_j        A = W~   (K-major),  B = P
//   dP part (Eq. 6-7):  acc[j, :] = sum_i W~_ij Q'_i       A = W~^T (MN-major), B = Q'
//
// with Q'_i = 2^(ref2_i - lse2_i) Q_i, so that W~_ij Q'_i = p_ij Q_i.  Both are plain GEMMs: no
// logits are recomputed.  The per-row factor of dQ and the positive-column terms of both
// gradients are applied in fp32 by the kernels that follow.
//
// One kernel template: 128 output rows per CTA (CTA pairs issue M = 256 MMAs and split every B
// item, as in the sweeps), up to 384 output columns per CTA in tensor memory, the contraction in
// steps of 128.  A and B travel through separate mbarrier rings: an A stage holds the two 64-wide
// chunks of a step side by side (an MN-major operand addresses them through one descriptor), a B
// stage holds one 128-column group of the step.  Warp 0 loads A, warp 1 loads B, warp 2 issues
// the MMAs, warps 3..10 run the epilogue.  Every wait is bounded.
#include "tc_common.cuh"

namespace gc {

namespace {

constexpr int GEMM_KSTEP = 128;
constexpr int MAX_A_STAGES = 4;
constexpr int MAX_B_STAGES = 10;
constexpr uint32_t A_STAGE_BYTES = 2 * CHUNK_BYTES;

struct GemmParams {
    int64_t m_rows;           // output rows
    int64_t k_len;            // contraction length
    int kc;                   // output columns / 64
    int dparts, dpc;          // column parts and chunks per part
    int groups;               // the contraction range is split into this many parts
    int na, nb;               // ring depths
    int final_out;            // 1: write out_scale * acc to the output, 0: plane g of the partials
    float out_scale;
    int* dev_status;
};

struct GemmBars {
    uint64_t a_full[MAX_A_STAGES];
    uint64_t a_empty[MAX_A_STAGES];
    uint64_t b_full[MAX_B_STAGES];
    uint64_t b_empty[MAX_B_STAGES];
    uint64_t acc_full;
};

template <bool A_MN, bool PAIR>
__global__ void __launch_bounds__(NTHREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
            const __grid_constant__ CUtensorMap mapO, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) GemmBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const bool leader = (rank == 0);
    constexpr uint32_t NCTA = PAIR ? 2u : 1u;
    constexpr uint32_t B_STAGE_BYTES = PAIR ? CHUNK_BYTES : 2 * CHUNK_BYTES;

    // work item: (row tile, column part, part of the contraction range)
    int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int g = unit % p.groups;
    unit /= p.groups;
    const int dp = unit % p.dparts;
    const int64_t xt = PAIR ? 2 * (int64_t)(unit / p.dparts) + rank : unit / p.dparts;
    const int64_t x0 = xt * XROWS;
    const int c_begin = dp * p.dpc;
    const int c_count = min(p.dpc, p.kc - c_begin);
    const int ngroups = (c_count + 1) / 2;          // 128-column groups of this part
    int64_t lo, hi;
    part_range((p.k_len + GEMM_KSTEP - 1) / GEMM_KSTEP, p.groups, g, &lo, &hi);
    const int T = (int)(hi - lo);

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_smem = base;
    const uint32_t b_smem = base + (uint32_t)p.na * A_STAGE_BYTES;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < MAX_A_STAGES; ++s) {
            mbar_init(smem_u32(&bars.a_full[s]), 1);
            mbar_init(smem_u32(&bars.a_empty[s]), 1);
        }
        for (int s = 0; s < MAX_B_STAGES; ++s) {
            mbar_init(smem_u32(&bars.b_full[s]), 1);
            mbar_init(smem_u32(&bars.b_empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.acc_full), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();     // both CTAs' barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    auto in_leader = [&](uint32_t local) -> uint32_t { return PAIR ? mapa_u32(local, 0) : local; };
    auto tma = [&](uint32_t dst, const CUtensorMap* map, int64_t col, int64_t r, uint32_t bar) {
        if (PAIR) tma_load_2d_pair(dst, map, (int)col, (int)r, bar);
        else      tma_load_2d(dst, map, (int)col, (int)r, bar);
    };

    if (warp == 0) {
        // ------------------------------ A loads ---------------------------------------------------
        // K-major A (rows = output rows, 64 contraction columns per chunk) or MN-major A (rows =
        // contraction rows, 64 output rows per chunk): the source box is 64 columns x 128 rows
        // either way, only the roles of the coordinates change.
        int stage = 0;
        uint32_t phase = 0;
        for (int t = 0; t < T; ++t) {
            if (!mbar_wait(smem_u32(&bars.a_empty[stage]), phase ^ 1u, abort_flag)) break;
            const uint32_t full = smem_u32(&bars.a_full[stage]);
            const uint32_t full_bar = in_leader(full);
            const uint32_t dst = a_smem + stage * A_STAGE_BYTES;
            const int64_t k0 = (lo + t) * GEMM_KSTEP;
            if (elect_one()) {
                if (leader) mbar_expect_tx(full, NCTA * A_STAGE_BYTES);
                for (int c = 0; c < 2; ++c) {
                    if (A_MN) tma(dst + c * CHUNK_BYTES, &mapA, x0 + 64 * c, k0, full_bar);
                    else      tma(dst + c * CHUNK_BYTES, &mapA, k0 + 64 * c, x0, full_bar);
                }
            }
            if (++stage == p.na) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == 1) {
        // ------------------------------ B loads ---------------------------------------------------
        // One item per 128-column group: 128 contraction rows x (64 columns of this rank when
        // paired, else both 64-column chunks).  A chunk past the last column reads as zeros.
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int t = 0; t < T && ok; ++t) {
            const int64_t k0 = (lo + t) * GEMM_KSTEP;
            for (int n = 0; n < ngroups; ++n) {
                if (!mbar_wait(smem_u32(&bars.b_empty[stage]), phase ^ 1u, abort_flag)) {
                    ok = false;
                    break;
                }
                const uint32_t full = smem_u32(&bars.b_full[stage]);
                const uint32_t full_bar = in_leader(full);
                const uint32_t dst = b_smem + stage * B_STAGE_BYTES;
                if (elect_one()) {
                    if (PAIR) {
                        if (leader) mbar_expect_tx(full, 2 * CHUNK_BYTES);
                        tma(dst, &mapB, (int64_t)(c_begin + 2 * n + (int)rank) * 64, k0, full_bar);
                    } else {
                        const int cnt = min(2, c_count - 2 * n);
                        mbar_expect_tx(full, (uint32_t)cnt * CHUNK_BYTES);
                        for (int i = 0; i < cnt; ++i)
                            tma(dst + i * CHUNK_BYTES, &mapB, (int64_t)(c_begin + 2 * n + i) * 64, k0,
                                full_bar);
                    }
                }
                if (++stage == p.nb) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------ MMA issuer ------------------------------------------------
        if (leader) {
            constexpr int MROWS = PAIR ? 2 * XROWS : XROWS;
            const uint32_t idesc128 = instr_desc(128, true, MROWS, A_MN);
            const uint32_t idesc64 = instr_desc(64, true, MROWS, A_MN);
            auto commit = [&](uint32_t bar) {
                if (PAIR) tc_commit_pair(bar);
                else      tc_commit(bar);
            };
            constexpr uint32_t CH_LO = CHUNK_BYTES >> 4;
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            bool ok = true;
            for (int t = 0; t < T && ok; ++t) {
                ok = mbar_wait(smem_u32(&bars.a_full[sa]), pa, abort_flag);
                if (!ok) break;
                tc_fence_after();
                // MN-major: the two 64-row atoms of A are one chunk apart
                const uint32_t a_lo = desc_lo(a_smem + sa * A_STAGE_BYTES, A_MN ? CHUNK_BYTES : 0);
                for (int n = 0; n < ngroups; ++n) {
                    ok = mbar_wait(smem_u32(&bars.b_full[sb]), pb, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t b_lo = desc_lo(b_smem + sb * B_STAGE_BYTES, CHUNK_BYTES);
                    const uint32_t d_tmem = tmem + n * 128;
                    const bool wide = PAIR || c_count - 2 * n >= 2;
                    const uint32_t idesc = wide ? idesc128 : idesc64;
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < GEMM_KSTEP / 16; ++k) {
                            const uint32_t a_k = A_MN ? a_lo + k * 128
                                                      : a_lo + (k / 4) * CH_LO + (k % 4) * 2;
                            if (k == 0 && t == 0) mma_ss<false, PAIR>(d_tmem, a_k, b_lo, idesc);
                            else                  mma_ss<true, PAIR>(d_tmem, a_k, b_lo + k * 128, idesc);
                        }
                        commit(smem_u32(&bars.b_empty[sb]));
                        if (n == ngroups - 1) commit(smem_u32(&bars.a_empty[sa]));
                    }
                    if (++sb == p.nb) { sb = 0; pb ^= 1u; }
                }
                if (++sa == p.na) { sa = 0; pa ^= 1u; }
            }
            if (ok && elect_one()) commit(smem_u32(&bars.acc_full));
        }
    } else {
        // ------------------------------ epilogue warps --------------------------------------------
        const int q = warp & 3;                        // tensor-memory lane quarter of this warp
        const int half = (warp - (NPROD + 1)) >> 2;    // alternate 32-column blocks
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        bool ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
        if (ok) {
            tc_fence_after();
            // every MMA and every load has completed: the dynamic shared memory is free
            const bool final_out = (p.final_out != 0);
            const uint32_t slot = base + (uint32_t)(warp - (NPROD + 1)) * 8192u;
            store_acc_blocks(tmem + lane_addr, c_count * 2, half, slot,
                             final_out ? p.out_scale : 1.f, lane, &mapO, c_begin * 64,
                             (int)x0 + q * 32, final_out ? 0 : g);
        }
    }

    // ------------------------------ teardown ------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // let bulk copies still in flight land before the shared memory is released
        uint64_t t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, GC_DEV_WAIT_LIMIT);
        __syncthreads();
    }
    if (PAIR) cluster_sync_all();   // the peer's MMAs, loads and arrivals no longer touch this CTA
    if (warp == MMA_WARP) {
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                         ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                         ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <bool A_MN, bool PAIR>
cudaError_t launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mo,
                        GemmParams p, int64_t ctas, cudaStream_t st) {
    constexpr size_t b_stage = PAIR ? CHUNK_BYTES : 2 * CHUNK_BYTES;
    p.na = 3;
    size_t avail = SMEM_LIMIT - SMEM_STATIC_RESERVE - 1024 - (size_t)p.na * A_STAGE_BYTES;
    int nb = (int)(avail / b_stage);
    if (nb > MAX_B_STAGES) nb = MAX_B_STAGES;
    p.nb = nb;
    const size_t dynamic_bytes = 1024 + (size_t)p.na * A_STAGE_BYTES + (size_t)nb * b_stage;
    // the attribute belongs to the (kernel, device) pair
    static bool configured_on[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    bool& configured = configured_on[dev];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<A_MN, PAIR>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(SMEM_LIMIT - SMEM_STATIC_RESERVE));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    if (!PAIR) {
        gemm_kernel<A_MN, false><<<(unsigned)ctas, NTHREADS, dynamic_bytes, st>>>(ma, mb, mo, p);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = dynamic_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_kernel<A_MN, PAIR>, ma, mb, mo, p);
}

}  // namespace

int gemm_groups(int64_t m_rows, int64_t k_len, int d) {
    const int kc = d / 64;
    int64_t tiles = (m_rows + XROWS - 1) / XROWS;
    if (m_rows > XROWS) tiles = (tiles + 1) / 2 * 2;
    int64_t units = tiles * parts_for(kc);
    int64_t steps = (k_len + GEMM_KSTEP - 1) / GEMM_KSTEP;
    int64_t g = sm_count() / units;
    if (g < 1) g = 1;
    if (g > steps) g = steps;
    if (g > 8) g = 8;
    return (int)g;
}

// acc = A B with A = weights [B x N] (transpose == 0: output rows are queries, the contraction
// runs over passages) or its transpose (output rows are passages, contraction over queries) and
// V = the [k_len x d] bf16 matrix of the other side.  With groups == 1 and an output pointer:
// out = out_scale * acc; otherwise partial[g] = the unscaled sum over part g of the contraction
// range.
cudaError_t launch_weight_gemm(const void* weights, int64_t ldw, int64_t B, int64_t N, int transpose,
                               const void* V, int64_t ldv, int d, int groups, float out_scale,
                               float* out, int64_t ldo, float* partial, int* dev_status,
                               cudaStream_t st) {
    const int64_t m_rows = transpose ? N : B, k_len = transpose ? B : N;
    CUtensorMap ma, mb, mo;
    if (!make_map(&ma, weights, B, (int)N, ldw, 128) || !make_map(&mb, V, k_len, d, ldv, 128))
        return cudaErrorInvalidValue;
    const bool final_out = groups == 1 && out != nullptr;
    const bool ok_map = final_out ? make_out_map(&mo, out, m_rows, d, ldo, 1)
                                  : make_out_map(&mo, partial, m_rows, d, d, groups);
    if (!ok_map) return cudaErrorInvalidValue;
    GemmParams p{};
    p.final_out = final_out ? 1 : 0;
    p.m_rows = m_rows; p.k_len = k_len;
    p.kc = d / 64; p.dparts = parts_for(p.kc); p.dpc = chunks_per_part(p.kc);
    p.groups = groups;
    p.out_scale = out_scale;
    p.dev_status = dev_status;
    const bool pair = m_rows > XROWS;
    int64_t tiles = (m_rows + XROWS - 1) / XROWS;
    if (pair) tiles = (tiles + 1) / 2 * 2;
    const int64_t ctas = tiles * p.dparts * groups;
    if (transpose)
        return pair ? launch_gemm<true, true>(ma, mb, mo, p, ctas, st)
                    : launch_gemm<true, false>(ma, mb, mo, p, ctas, st);
    return pair ? launch_gemm<false, true>(ma, mb, mo, p, ctas, st)
                : launch_gemm<false, false>(ma, mb, mo, p, ctas, st);
}

}  // namespace gc
