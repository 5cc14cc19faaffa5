// One-launch plan for batches of a single tile: B <= 128 queries, N <= 256 passages (bf16) or
// N <= 128 (fp32), d a multiple of 8.  Loss (Eq. 1) and the representation gradients (Eq. 5-7)
// of such a batch are a few hundred MFLOP: several dependent launches cost more than the work.
//
// CTA c owns columns [64 c, 64 c + 64) of dQ and dP; the CTAs do not talk to one another.  Every
// CTA forms the whole logit tile S = Q P^T (tcgen05, fp32 in tensor memory) from 64-column slices
// of Q and P that a producer warp streams through shared memory, the softmax warps turn it into
// the weights W_ij = p_ij - [j = r_i] (0 at masked pairs, rows past B and columns past N), kept
// in shared memory as bf16 MMA operands, and two more products give the CTA's columns,
//     dQ[:, slice] = W P[:, slice] / (B tau),     dP[:, slice] = W^T Q[:, slice] / (B tau),
// with the slice of P (of Q) read as the MN-major B operand where the bulk tensor load left it.
// CTA 0 also writes loss, row_lse, pos_logit and the pos_idx flags.
//
// fp32 inputs run on the same tensor cores: converter warps split every value into three bf16
// terms x = t1 + t2 + t3 (each the rounding of what the previous ones left, so the sum is exact
// to 2^-24 |x|) as it arrives, S takes the six products t1 t1', t1 t2', t1 t3', t2 t1', t2 t2',
// t3 t1' in fp32 accumulation, the weights are kept as two terms and the gradient products take
// w1 t1 + w1 t2 + w2 t1.  Every mbarrier wait is bounded.
#include "tc_common.cuh"

namespace gc {

namespace {

constexpr int SM_WORKERS = 8;                    // converter / softmax / epilogue warps
constexpr int SM_PROD_WARP = 0;
constexpr int SM_MMA_WARP = 1;
constexpr int SM_FIRST_WORKER = 2;
constexpr int SM_THREADS = 32 * (SM_FIRST_WORKER + SM_WORKERS);
constexpr uint32_t TILE = 16384;                 // 128 rows x 128 bytes
constexpr int SM_STAGES = 3;
constexpr uint32_t BF_STAGE = 3 * TILE;          // Q slice + P slice (two row tiles)
constexpr uint32_t F32_STAGE = 2 * TILE;         // 32 fp32 columns of Q and of P
constexpr uint32_t BF_W_OFF = SM_STAGES * BF_STAGE;          // four weight chunks behind the ring
constexpr uint32_t F32_TERM_OFF = SM_STAGES * F32_STAGE;     // q1 q2 q3 p1 p2 p3 behind the ring
constexpr size_t SM_DYN_SMEM = 1024 + (size_t)SM_STAGES * BF_STAGE + 4 * TILE;
constexpr uint32_t COL_S = 0, COL_DQ = 256, COL_DP = 320;    // tensor-memory columns

static_assert(SM_DYN_SMEM <= SMEM_LIMIT - SMEM_STATIC_RESERVE, "shared memory budget");
static_assert(F32_TERM_OFF + 6 * TILE <= SM_STAGES * BF_STAGE + 4 * TILE, "fp32 layout fits");

struct SmallParams {
    int B, N, d;
    int op;                   // GC_OP_FWD, GC_OP_BWD, GC_OP_BUILD
    int mask_mode;
    int mask_shift;           // masked pair: j == i + mask_shift
    float scale2;             // log2(e) / tau
    float out_scale;          // 1 / (B tau)
    float inv_mean;           // 1 / B
    const int32_t* pos_idx;
    const float* row_lse_in;  // GC_OP_BWD
    float* loss;
    float* row_lse;
    float* pos_logit;         // may be NULL
    float* dQ;
    int64_t lddq;
    float* dP;
    int64_t lddp;
    int* dev_status;
};

struct SmallBars {
    uint64_t full[SM_STAGES];
    uint64_t empty[SM_STAGES];
    uint64_t term_full[2];
    uint64_t term_empty[2];
    uint64_t s_full;
    uint64_t w_full;
    uint64_t acc_full;
};

__device__ __forceinline__ float4 lds128f(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128u(uint32_t addr, const uint32_t (&w)[4]) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float x, float y) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float lo_f(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float hi_f(uint32_t packed) {
    return __uint_as_float(packed & 0xffff0000u);
}
// (x, y) -> three packed bf16 pairs whose sum is (x, y) to 2^-24
__device__ __forceinline__ void split3(float x, float y, uint32_t* t1, uint32_t* t2, uint32_t* t3) {
    const uint32_t a = pack_bf16(x, y);
    const float rx = x - lo_f(a), ry = y - hi_f(a);
    const uint32_t b = pack_bf16(rx, ry);
    *t1 = a;
    *t2 = b;
    *t3 = pack_bf16(rx - lo_f(b), ry - hi_f(b));
}
// All worker threads take a decision together (named barrier 1).
__device__ __forceinline__ bool workers_all(bool mine) {
    uint32_t all;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "barrier.cta.red.and.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(all) : "r"(mine ? 1u : 0u), "n"(32 * SM_WORKERS) : "memory");
    return all != 0;
}
__device__ __forceinline__ void workers_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(32 * SM_WORKERS) : "memory");
}

template <bool F32>
__global__ void __launch_bounds__(SM_THREADS, 1)
small_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapP,
             const SmallParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) SmallBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float x_max[2][128], x_sum[2][128];     // exchange between the two column halves
    __shared__ float loss_part[4];
    volatile int* abort_flag = &abort_s;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;
    const int slice = blockIdx.x;
    const bool do_grad = p.op != GC_OP_FWD;
    // steps of the S loop: 64 columns (bf16) or 32 columns (fp32, an even number of them so that
    // a slice's first half always lands in the first half of the term tiles; a step past d reads
    // zeros); then the CTA's own slice
    const int s_steps = F32 ? 2 * ((p.d + 63) / 64) : (p.d + 63) / 64;
    const int g_steps = do_grad ? (F32 ? 2 : 1) : 0;
    const int n_pad = (p.N + 15) & ~15;
    const int ptiles = p.N > 128 ? 2 : 1;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t STAGE = F32 ? F32_STAGE : BF_STAGE;
    const uint32_t w_smem = F32 ? base : base + BF_W_OFF;      // fp32: over the drained ring
    const uint32_t term_smem = base + F32_TERM_OFF;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < SM_STAGES; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), F32 ? SM_WORKERS : 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bars.term_full[s]), SM_WORKERS);
            mbar_init(smem_u32(&bars.term_empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.s_full), 1);
        mbar_init(smem_u32(&bars.w_full), SM_WORKERS);
        mbar_init(smem_u32(&bars.acc_full), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == SM_MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    if (warp == SM_PROD_WARP) {
        // ------------------------------ loads -----------------------------------------------------
        // Rows past B (N) and columns past d read as zeros.
        int stage = 0;
        uint32_t phase = 0;
        for (int t = 0; t < s_steps + g_steps; ++t) {
            if (!mbar_wait(smem_u32(&bars.empty[stage]), phase ^ 1u, abort_flag)) break;
            const uint32_t full = smem_u32(&bars.full[stage]);
            const uint32_t dst = base + stage * STAGE;
            int col;
            if (F32) col = t < s_steps ? 32 * t : 64 * slice + 32 * (t - s_steps);
            else     col = t < s_steps ? 64 * t : 64 * slice;
            if (elect_one()) {
                if (F32) {
                    mbar_expect_tx(full, 2 * TILE);
                    tma_load_2d(dst, &mapQ, col, 0, full);
                    tma_load_2d(dst + TILE, &mapP, col, 0, full);
                } else {
                    mbar_expect_tx(full, (uint32_t)(1 + ptiles) * TILE);
                    tma_load_2d(dst, &mapQ, col, 0, full);
                    tma_load_2d(dst + TILE, &mapP, col, 0, full);
                    if (ptiles == 2) tma_load_2d(dst + 2 * TILE, &mapP, col, 128, full);
                }
            }
            if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == SM_MMA_WARP) {
        // ------------------------------ MMA issuer ------------------------------------------------
        const uint32_t idesc_s = instr_desc(n_pad, false, XROWS, false);
        const uint32_t idesc_dq = instr_desc(64, true, XROWS, false);    // A = W, K-major
        const uint32_t idesc_dp = instr_desc(64, true, XROWS, true);     // A = W^T: MN-major
        const int nchunks = (p.N + 63) / 64;
        bool ok = true;
        uint32_t q_tile = 0, p_tile = 0;       // the CTA's own slices as MN-major B operands
        if (F32) {
            for (int t = 0; t < s_steps && ok; ++t) {
                const int h = t & 1;
                ok = mbar_wait(smem_u32(&bars.term_full[h]), (uint32_t)(t >> 1) & 1u, abort_flag);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        const uint32_t k = (uint32_t)(2 * (2 * h + kk));     // 32 bytes per K = 16
                        const uint32_t q1 = desc_lo(term_smem, 0) + k;
                        const uint32_t p1 = desc_lo(term_smem + 3 * TILE, 0) + k;
                        constexpr uint32_t T = TILE >> 4;
                        if (t == 0 && kk == 0) mma_ss<false, false>(tmem + COL_S, q1, p1, idesc_s);
                        else                   mma_ss<true, false>(tmem + COL_S, q1, p1, idesc_s);
                        mma_ss<true, false>(tmem + COL_S, q1, p1 + T, idesc_s);
                        mma_ss<true, false>(tmem + COL_S, q1 + T, p1, idesc_s);
                        mma_ss<true, false>(tmem + COL_S, q1 + T, p1 + T, idesc_s);
                        mma_ss<true, false>(tmem + COL_S, q1, p1 + 2 * T, idesc_s);
                        mma_ss<true, false>(tmem + COL_S, q1 + 2 * T, p1, idesc_s);
                    }
                    tc_commit(smem_u32(&bars.term_empty[h]));
                }
            }
            if (ok && elect_one()) tc_commit(smem_u32(&bars.s_full));
            for (int t = s_steps; t < s_steps + g_steps && ok; ++t)
                ok = mbar_wait(smem_u32(&bars.term_full[t & 1]), (uint32_t)(t >> 1) & 1u, abort_flag);
            q_tile = term_smem;
            p_tile = term_smem + 3 * TILE;
        } else {
            int stage = 0;
            uint32_t phase = 0;
            for (int t = 0; t < s_steps && ok; ++t) {
                ok = mbar_wait(smem_u32(&bars.full[stage]), phase, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a = desc_lo(base + stage * STAGE, 0);
                const uint32_t b = desc_lo(base + stage * STAGE + TILE, 0);
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        if (t == 0 && kk == 0) mma_ss<false, false>(tmem + COL_S, a, b, idesc_s);
                        else mma_ss<true, false>(tmem + COL_S, a + 2 * kk, b + 2 * kk, idesc_s);
                    }
                    tc_commit(smem_u32(&bars.empty[stage]));
                }
                if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (ok && elect_one()) tc_commit(smem_u32(&bars.s_full));
            if (ok && do_grad) {
                ok = mbar_wait(smem_u32(&bars.full[stage]), phase, abort_flag);
                q_tile = base + stage * STAGE;
                p_tile = q_tile + TILE;
            }
        }
        if (ok && do_grad) ok = mbar_wait(smem_u32(&bars.w_full), 0, abort_flag);
        if (ok && do_grad) {
            tc_fence_after();
            if (elect_one()) {
                // products (weight term, operand term): fp32 inputs take w1 t1, w1 t2, w2 t1
                constexpr int NPROD_G = F32 ? 3 : 1;
                constexpr uint32_t T = TILE >> 4;
                const uint32_t w_term[3] = {0u, 0u, 2 * T};        // lo weights: 2 chunks further
                const uint32_t o_term[3] = {0u, T, 0u};
                // dQ slice: contraction over passages, 64 per weight chunk
                bool first = true;
                for (int c = 0; c < nchunks; ++c) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
                        for (int pr = 0; pr < NPROD_G; ++pr) {
                            const uint32_t a = desc_lo(w_smem + c * TILE, 0) + w_term[pr] + 2 * kk;
                            const uint32_t b = desc_lo(p_tile + c * (TILE / 2), 0) + o_term[pr] + 128 * kk;
                            if (first) mma_ss<false, false>(tmem + COL_DQ, a, b, idesc_dq);
                            else       mma_ss<true, false>(tmem + COL_DQ, a, b, idesc_dq);
                            first = false;
                        }
                    }
                }
                // dP slice: contraction over the 128 query rows; 128 passages per block
                for (int blk = 0; blk < ptiles; ++blk) {
                    first = true;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
                        for (int pr = 0; pr < NPROD_G; ++pr) {
                            const uint32_t a = desc_lo(w_smem + 2 * blk * TILE, TILE) + w_term[pr] + 128 * kk;
                            const uint32_t b = desc_lo(q_tile, 0) + o_term[pr] + 128 * kk;
                            if (first) mma_ss<false, false>(tmem + COL_DP + 64 * blk, a, b, idesc_dp);
                            else       mma_ss<true, false>(tmem + COL_DP + 64 * blk, a, b, idesc_dp);
                            first = false;
                        }
                    }
                }
                tc_commit(smem_u32(&bars.acc_full));
            }
        }
    } else {
        // ------------------------------ workers ---------------------------------------------------
        const int wt = threadIdx.x - 32 * SM_FIRST_WORKER;      // 0 .. 255
        const int q = warp & 3;                                  // tensor-memory lane quarter
        const int half = (warp - SM_FIRST_WORKER) >> 2;          // column half of S / of a slice
        const int i = 32 * q + lane;                             // row of S, of dQ, of a dP block
        const uint32_t lane_addr = (uint32_t)(32 * q) << 16;
        bool ok = true;
        if (F32) {
            // fp32 -> three bf16 terms.  Item = 8 consecutive columns of one row (two 16-byte
            // pieces in, one piece per term out).  Eight neighbouring threads take four items of
            // row r and four of row r + 4, the second row fetching its two pieces in the opposite
            // order: loads and stores both fall on distinct banks.
            int stage = 0;
            uint32_t phase = 0;
            for (int t = 0; t < s_steps + g_steps; ++t) {
                const int h = t & 1;
                ok = mbar_wait(smem_u32(&bars.full[stage]), phase, abort_flag) &&
                     mbar_wait(smem_u32(&bars.term_empty[h]), ((uint32_t)(t >> 1) & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                const uint32_t src0 = base + stage * STAGE;
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int id = wt + 256 * it;
                    const int cp = id & 3, rr = (id >> 2) & 1, b = (id >> 3) & 3, a = (id >> 5) & 15;
                    const int mat = id >> 9;
                    const int r = 8 * a + b + 4 * rr, sw = r & 7;
                    const uint32_t src = src0 + mat * TILE + r * 128;
                    const int first = (2 * cp) ^ rr;
                    const float4 A = lds128f(src + (uint32_t)((first ^ sw) << 4));
                    const float4 Bv = lds128f(src + (uint32_t)(((first ^ 1) ^ sw) << 4));
                    const float4 f0 = rr ? Bv : A, f1 = rr ? A : Bv;
                    uint32_t t1[4], t2[4], t3[4];
                    split3(f0.x, f0.y, &t1[0], &t2[0], &t3[0]);
                    split3(f0.z, f0.w, &t1[1], &t2[1], &t3[1]);
                    split3(f1.x, f1.y, &t1[2], &t2[2], &t3[2]);
                    split3(f1.z, f1.w, &t1[3], &t2[3], &t3[3]);
                    const uint32_t dst = term_smem + (uint32_t)(3 * mat) * TILE + r * 128 +
                                         (uint32_t)(((4 * h + cp) ^ sw) << 4);
                    sts128u(dst, t1);
                    sts128u(dst + TILE, t2);
                    sts128u(dst + 2 * TILE, t3);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&bars.term_full[h]));
                    mbar_arrive(smem_u32(&bars.empty[stage]));
                }
                if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        ok = ok && mbar_wait(smem_u32(&bars.s_full), 0, abort_flag);
        if (workers_all(ok)) {
            tc_fence_after();
            // ------------------------------ softmax of row i over this half's columns -------------
            const int ncols = F32 ? 128 : 256;
            const int j0 = half * (ncols / 2);                    // fp32: 0 or 64; bf16: 0 or 128
            const int nblk = ncols / 64;                          // blocks of 32 columns per half
            const int32_t r_i = i < p.B ? p.pos_idx[i] : -1;
            int flags = 0;
            if (i < p.B) {
                if (r_i < 0 || r_i >= p.N) flags = GC_DEV_POS_RANGE;
                else if (p.mask_mode == GC_MASK_SELF && r_i == i + p.mask_shift) flags = GC_DEV_POS_MASKED;
            }
            const int pos = flags ? -1 : r_i;
            const int masked = p.mask_mode == GC_MASK_SELF ? i + p.mask_shift : -1;
            float lse2, pos2 = 0.f;
            if (p.op == GC_OP_BWD) {
                lse2 = i < p.B ? p.row_lse_in[i] * 1.4426950408889634f : 0.f;
            } else {
                float m = -INFINITY;
                for (int cb = 0; cb < nblk; ++cb) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + COL_S + j0 + 32 * cb, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int j = j0 + 32 * cb + e;
                        const float s2 = __uint_as_float(v[e]) * p.scale2;
                        if (j == pos) pos2 = s2;
                        if (j < p.N && j != masked) m = fmaxf(m, s2);
                    }
                }
                x_max[half][i] = m;
                x_sum[half][i] = pos2;
                workers_sync();
                m = fmaxf(x_max[0][i], x_max[1][i]);
                pos2 = x_sum[0][i] + x_sum[1][i];                 // the other half holds 0
                workers_sync();
                float sum = 0.f;
                for (int cb = 0; cb < nblk; ++cb) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + COL_S + j0 + 32 * cb, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int j = j0 + 32 * cb + e;
                        const float s2 = __uint_as_float(v[e]) * p.scale2;
                        if (j < p.N && j != masked) sum += exp2f(s2 - m);
                    }
                }
                x_sum[half][i] = sum;
                workers_sync();
                sum = x_sum[0][i] + x_sum[1][i];
                lse2 = m + log2f(sum);
            }
            // ------------------------------ outputs of the forward (CTA 0) ------------------------
            if (slice == 0) {
                const float ln2 = 0.6931471805599453f;
                float term = 0.f;
                if (half == 0 && i < p.B) {
                    if (p.op != GC_OP_BWD) {
                        p.row_lse[i] = lse2 * ln2;
                        if (p.pos_logit) p.pos_logit[i] = pos2 * ln2;
                        term = (lse2 - pos2) * ln2;
                    }
                    if (flags && p.dev_status) atomicOr(p.dev_status, flags);
                }
                if (p.op != GC_OP_BWD) {
                    for (int o = 16; o > 0; o >>= 1) term += __shfl_xor_sync(0xffffffffu, term, o);
                    if (half == 0 && lane == 0) loss_part[q] = term;
                    workers_sync();
                    if (wt == 0)
                        *p.loss = (((loss_part[0] + loss_part[1]) + loss_part[2]) + loss_part[3]) *
                                  p.inv_mean;
                }
            }
            if (do_grad) {
                // ------------------------------ weights as MMA operands ---------------------------
                // chunk c = 64 columns; element (i, j) in 16-byte piece ((j % 64) / 8) ^ (i % 8) of
                // row i: a K-major A operand for dQ and, read by columns, an MN-major one for dP
                for (int cb = 0; cb < nblk; ++cb) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + COL_S + j0 + 32 * cb, v);
                    tmem_ld_wait();
                    float w[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int j = j0 + 32 * cb + e;
                        float x = 0.f;
                        if (i < p.B && j < p.N && j != masked) {
                            x = exp2f(__uint_as_float(v[e]) * p.scale2 - lse2);
                            if (j == pos) x -= 1.f;
                        }
                        w[e] = x;
                    }
                    const int jb = j0 + 32 * cb;                  // 4 pieces of 8 columns
                    const uint32_t row = w_smem + (uint32_t)(jb >> 6) * TILE + i * 128;
#pragma unroll
                    for (int pc = 0; pc < 4; ++pc) {
                        const int piece = ((jb & 63) >> 3) + pc;
                        const uint32_t dst = row + (uint32_t)((piece ^ (i & 7)) << 4);
                        uint32_t hi[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) hi[e] = pack_bf16(w[8 * pc + 2 * e], w[8 * pc + 2 * e + 1]);
                        sts128u(dst, hi);
                        if (F32) {
                            uint32_t lo[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                lo[e] = pack_bf16(w[8 * pc + 2 * e] - lo_f(hi[e]),
                                                  w[8 * pc + 2 * e + 1] - hi_f(hi[e]));
                            sts128u(dst + 2 * TILE, lo);
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.w_full));
                // ------------------------------ gradients out -------------------------------------
                if (mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag)) {
                    tc_fence_after();
                    const int col = 64 * slice + 32 * half;
                    for (int blk = 0; blk < 1 + ptiles; ++blk) {       // dQ, dP rows 0.., dP rows 128..
                        const int rows = blk == 0 ? p.B : p.N - 128 * (blk - 1);
                        float* out = blk == 0 ? p.dQ + (int64_t)i * p.lddq
                                              : p.dP + (int64_t)(128 * (blk - 1) + i) * p.lddp;
                        uint32_t v[32];
                        tmem_ld32(tmem + lane_addr + (blk == 0 ? COL_DQ : COL_DP + 64 * (blk - 1)) +
                                      32 * half, v);
                        tmem_ld_wait();
                        if (i < rows && (blk == 0 ? p.dQ : p.dP) != nullptr) {
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (col + 4 * e < p.d)
                                    *reinterpret_cast<float4*>(out + col + 4 * e) = make_float4(
                                        __uint_as_float(v[4 * e]) * p.out_scale,
                                        __uint_as_float(v[4 * e + 1]) * p.out_scale,
                                        __uint_as_float(v[4 * e + 2]) * p.out_scale,
                                        __uint_as_float(v[4 * e + 3]) * p.out_scale);
                        }
                    }
                }
            }
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
    if (warp == SM_MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <bool F32>
cudaError_t launch_small_t(const CUtensorMap& mq, const CUtensorMap& mp, const SmallParams& p,
                           unsigned ctas, cudaStream_t st) {
    static bool configured_on[64] = {false};      // the attribute belongs to (kernel, device)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured_on[dev]) {
        cudaError_t e = cudaFuncSetAttribute(small_kernel<F32>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)SM_DYN_SMEM);
        if (e != cudaSuccess) return e;
        configured_on[dev] = true;
    }
    small_kernel<F32><<<ctas, SM_THREADS, SM_DYN_SMEM, st>>>(mq, mp, p);
    return cudaGetLastError();
}

}  // namespace

bool small_applicable(int64_t B, int64_t N, int d, int dtype) {
    if (B > 128 || d % 8 != 0 || d > 1024) return false;
    return dtype == GC_BF16 ? N <= 256 : N <= 128;
}

// op: GC_OP_FWD (loss, row_lse, pos_logit), GC_OP_BWD (dQ, dP from row_lse_in) or GC_OP_BUILD.
cudaError_t launch_small(int op, const Problem& pr, const float* row_lse_in, float* loss,
                         float* row_lse, float* pos_logit, float* dQ, int64_t lddq, float* dP,
                         int64_t lddp, int* dev_status, cudaStream_t st) {
    const bool f32 = pr.dtype == GC_F32;
    CUtensorMap mq, mp;
    const bool ok = f32 ? make_map_f32(&mq, pr.Q, pr.B, pr.d, pr.ldq, 128) &&
                              make_map_f32(&mp, pr.P, pr.N, pr.d, pr.ldp, 128)
                        : make_map(&mq, pr.Q, pr.B, pr.d, pr.ldq, 128) &&
                              make_map(&mp, pr.P, pr.N, pr.d, pr.ldp, 128);
    if (!ok) return cudaErrorInvalidValue;
    SmallParams p{};
    p.B = (int)pr.B; p.N = (int)pr.N; p.d = pr.d;
    p.op = op;
    p.mask_mode = pr.mask_mode;
    p.mask_shift = (int)pr.mask_shift;
    p.scale2 = 1.4426950408889634f / pr.tau;
    const float batch = (float)(pr.b_total > 0 ? pr.b_total : pr.B);
    p.out_scale = 1.f / (batch * pr.tau);
    p.inv_mean = 1.f / batch;
    p.pos_idx = pr.pos_idx;
    p.row_lse_in = row_lse_in;
    p.loss = loss; p.row_lse = row_lse; p.pos_logit = pos_logit;
    p.dQ = dQ; p.lddq = lddq; p.dP = dP; p.lddp = lddp;
    p.dev_status = dev_status;
    const unsigned ctas = op == GC_OP_FWD ? 1u : (unsigned)((pr.d + 63) / 64);
    return f32 ? launch_small_t<true>(mq, mp, p, ctas, st) : launch_small_t<false>(mq, mp, p, ctas, st);
}

}  // namespace gc
