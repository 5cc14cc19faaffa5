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
// terms x = t1 + t2 + t3 (each the upper 16 bits of what the previous ones left, so the sum is
// exact) as it arrives, S takes the six products t1 t1', t1 t2', t1 t3', t2 t1', t2 t2', t3 t1'
// in fp32 accumulation (spread over three accumulators, see the MMA warp), the weights are kept
// as two terms and the gradient products take w1 (t1 + t2 + t3) + w2 (t1 + t2).  Every mbarrier
// wait is bounded.
#include <stdlib.h>
#include <string.h>

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
constexpr uint32_t COL_S2 = 384;     // fp32 inputs: the small products of S (128 columns)

static_assert(SM_DYN_SMEM <= SMEM_LIMIT - SMEM_STATIC_RESERVE, "shared memory budget");
static_assert(F32_TERM_OFF + 6 * TILE <= SM_STAGES * BF_STAGE + 4 * TILE, "fp32 layout fits");

struct SmallParams {
    int B, N, d;
    int op;                   // GC_OP_FWD, GC_OP_BWD, GC_OP_BUILD
    int mask_mode;
    int mask_shift;           // masked pair: j == i + mask_shift
    float scale2;             // log2(e) / tau
    float inv_tau;
    float out_scale;          // 1 / (B tau)
    float inv_mean;           // 1 / B
    const int32_t* pos_idx;
    const float* row_lse_in;  // GC_OP_BWD
    // Several tiles (grid y = query tiles of 128, grid z = passage tiles): the forward writes one
    // (max, sum) slot per passage tile and row, slot t at [t * B + i] (natural-log units), and the
    // positive's logit, for the combine kernel that follows; the gradients of a tile pair go to
    // plane (passage tile) of the dQ partials and plane (query tile) of the dP partials.
    int tiled;
    int plane_q, plane_p;     // the gradient of that side goes to a plane of partials
    float out_scale_q, out_scale_p;
    float* part_m;
    float* part_l;
    float* pos_ws;
    int* zero_me;             // block ticket of the loss reduction that follows: cleared here
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
// 32 columns of this thread's row of S; fp32 inputs keep S as the sum of three accumulators.
template <bool F32>
__device__ __forceinline__ void load_s(uint32_t trow, int jb, float (&s)[32]) {
    uint32_t v[32];
    tmem_ld32(trow + COL_S + jb, v);
    tmem_ld_wait();
#pragma unroll
    for (int e = 0; e < 32; ++e) s[e] = __uint_as_float(v[e]);
    if (F32) {
        uint32_t u[32];
        tmem_ld32(trow + COL_S + 128 + jb, v);
        tmem_ld32(trow + COL_S2 + jb, u);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; ++e) s[e] = (s[e] + __uint_as_float(v[e])) + __uint_as_float(u[e]);
    }
}
__device__ __forceinline__ void workers_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(32 * SM_WORKERS) : "memory");
}

template <bool F32>
__global__ void __launch_bounds__(SM_THREADS, 1)
small_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapP,
             const __grid_constant__ CUtensorMap mapDQ, const __grid_constant__ CUtensorMap mapDP,
             const SmallParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) SmallBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float x_max[2][128], x_sum[2][128], x_pos[2][128];   // exchange between the column halves
    __shared__ float loss_part[4];
    volatile int* abort_flag = &abort_s;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;
    const int slice = blockIdx.x;
    const bool do_grad = p.op != GC_OP_FWD;
    // this CTA's tile pair: rows x0 .. of Q, rows y0 .. of P; B_ and N_ are the rows it holds
    constexpr int YT = F32 ? 128 : 256;
    const int x0 = 128 * (int)blockIdx.y, y0 = YT * (int)blockIdx.z;
    const int B_ = min(128, p.B - x0), N_ = min(YT, p.N - y0);
    // steps of the S loop: 64 columns (bf16) or 32 columns (fp32, an even number of them so that
    // a slice's first half always lands in the first half of the term tiles; a step past d reads
    // zeros); then the CTA's own slice
    const int s_steps = F32 ? 2 * ((p.d + 63) / 64) : (p.d + 63) / 64;
    const int g_steps = do_grad ? (F32 ? 2 : 1) : 0;
    const int n_pad = (N_ + 15) & ~15;
    const int ptiles = N_ > 128 ? 2 : 1;

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
                    tma_load_2d(dst, &mapQ, col, x0, full);
                    tma_load_2d(dst + TILE, &mapP, col, y0, full);
                } else {
                    mbar_expect_tx(full, (uint32_t)(1 + ptiles) * TILE);
                    tma_load_2d(dst, &mapQ, col, x0, full);
                    tma_load_2d(dst + TILE, &mapP, col, y0, full);
                    if (ptiles == 2) tma_load_2d(dst + 2 * TILE, &mapP, col, y0 + 128, full);
                }
            }
            if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == SM_MMA_WARP) {
        // ------------------------------ MMA issuer ------------------------------------------------
        const uint32_t idesc_s = instr_desc(n_pad, false, XROWS, false);
        const uint32_t idesc_dq = instr_desc(64, true, XROWS, false);    // A = W, K-major
        const uint32_t idesc_dp = instr_desc(64, true, XROWS, true);     // A = W^T: MN-major
        const int nchunks = (N_ + 63) / 64;
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
                        // The accumulator adds with truncation: the leading product alternates
                        // between two accumulators and the five small ones have a third, so that
                        // each takes few additions of its own magnitude; the softmax warps sum
                        // the three in fp32.
                        const uint32_t lead = tmem + COL_S + 128 * kk, rest = tmem + COL_S2;
                        if (t == 0) mma_ss<false, false>(lead, q1, p1, idesc_s);
                        else        mma_ss<true, false>(lead, q1, p1, idesc_s);
                        if (t == 0 && kk == 0) mma_ss<false, false>(rest, q1, p1 + T, idesc_s);
                        else                   mma_ss<true, false>(rest, q1, p1 + T, idesc_s);
                        mma_ss<true, false>(rest, q1 + T, p1, idesc_s);
                        mma_ss<true, false>(rest, q1 + T, p1 + T, idesc_s);
                        mma_ss<true, false>(rest, q1, p1 + 2 * T, idesc_s);
                        mma_ss<true, false>(rest, q1 + 2 * T, p1, idesc_s);
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
                // products (weight term, operand term): fp32 inputs take w1 t1, w1 t2, w1 t3, w2 t1,
                // w2 t2 (the terms are truncations: dropping t3 would leave a one-sided 2^-16)
                constexpr int NPROD_G = F32 ? 5 : 1;
                constexpr uint32_t T = TILE >> 4;
                const uint32_t w_term[5] = {0u, 0u, 0u, 2 * T, 2 * T};   // lo weights: 2 chunks further
                const uint32_t o_term[5] = {0u, T, 2 * T, 0u, T};
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
            // fp32 -> three bf16 terms by truncation (t1 = the upper 16 bits of x, t2 those of
            // x - t1, t3 those of what is left: x = t1 + t2 + t3 exactly).  Item = 8 consecutive
            // columns of one row (two 16-byte pieces in, one piece per term out).  Eight
            // neighbouring threads take four items of row r and four of row r + 4, the second
            // row fetching its two pieces in the opposite order: loads and stores both fall on
            // distinct banks.  Rows past B (N) are skipped: the term tiles start out as zeros.
            for (int e = wt; e < (int)(6 * TILE / 16); e += 32 * SM_WORKERS) {
                const uint32_t z[4] = {0u, 0u, 0u, 0u};
                sts128u(term_smem + 16 * e, z);
            }
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
                    if (r >= (mat ? N_ : B_)) continue;
                    const uint32_t src = src0 + mat * TILE + r * 128;
                    const int first = (2 * cp) ^ rr;
                    const float4 A = lds128f(src + (uint32_t)((first ^ sw) << 4));
                    const float4 Bv = lds128f(src + (uint32_t)(((first ^ 1) ^ sw) << 4));
                    const float4 f0 = rr ? Bv : A, f1 = rr ? A : Bv;
                    const float x[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
                    uint32_t t1[4], t2[4], t3[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t a0 = __float_as_uint(x[2 * e]), a1 = __float_as_uint(x[2 * e + 1]);
                        const float r0 = x[2 * e] - __uint_as_float(a0 & 0xffff0000u);
                        const float r1 = x[2 * e + 1] - __uint_as_float(a1 & 0xffff0000u);
                        const uint32_t b0 = __float_as_uint(r0), b1 = __float_as_uint(r1);
                        const float s0 = r0 - __uint_as_float(b0 & 0xffff0000u);
                        const float s1 = r1 - __uint_as_float(b1 & 0xffff0000u);
                        t1[e] = __byte_perm(a0, a1, 0x7632);      // the two upper halves
                        t2[e] = __byte_perm(b0, b1, 0x7632);
                        t3[e] = __byte_perm(__float_as_uint(s0), __float_as_uint(s1), 0x7632);
                    }
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
            // One pass over the row keeps a running (max, sum); the special columns of a block of
            // 32 (past N, the masked pair, the positive) are patched after the plain arithmetic.
            const int ncols = F32 ? 128 : 256;
            const int j0 = half * (ncols / 2);                    // fp32: 0 or 64; bf16: 0 or 128
            const int nblk = ncols / 64;                          // blocks of 32 columns per half
            // columns are counted within the tile: the positive and the masked pair of row i fall
            // into it or not
            const int32_t r_i = i < B_ ? p.pos_idx[x0 + i] : -1;
            int flags = 0;
            if (i < B_) {
                if (r_i < 0 || r_i >= p.N) flags = GC_DEV_POS_RANGE;
                else if (p.mask_mode == GC_MASK_SELF && r_i == x0 + i + p.mask_shift) flags = GC_DEV_POS_MASKED;
            }
            const int pos = (flags || r_i < y0 || r_i >= y0 + N_) ? -1 : r_i - y0;
            const int masked = p.mask_mode == GC_MASK_SELF ? x0 + i + p.mask_shift - y0 : -1;
            float lse2, pos2 = 0.f, lse_nat = 0.f, m_row = 0.f, lnsum_row = 0.f;
            if (p.op == GC_OP_BWD) {
                lse2 = p.row_lse_in[i < B_ ? x0 + i : 0] * 1.4426950408889634f;
            } else {
                // The running maximum is kept in units of <q, p> (unscaled), so that the row's
                // logsumexp and its positive logit come out of the same product with 1/tau:
                // lse_i - S_{i,r_i} is exactly 0 when the positive is the only column.
                float m = -INFINITY, sum = 0.f, lnsum = 0.f;
                for (int cb = 0; cb < nblk; ++cb) {
                    const int jb = j0 + 32 * cb;
                    if (jb >= N_) break;
                    float sr[32];
                    load_s<F32>(tmem + lane_addr, jb, sr);
                    if ((unsigned)(pos - jb) < 32u) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) if (e == pos - jb) pos2 = sr[e];
                    }
                    if ((unsigned)(masked - jb) < 32u) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) if (e == masked - jb) sr[e] = -INFINITY;
                    }
                    if (jb + 32 > N_) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) if (jb + e >= N_) sr[e] = -INFINITY;
                    }
                    float bm = sr[0];
#pragma unroll
                    for (int e = 1; e < 32; ++e) bm = fmaxf(bm, sr[e]);
                    const float mn = fmaxf(m, bm);
                    const float ref = mn == -INFINITY ? 0.f : mn;
                    float part = 0.f;      // (s - max) first: the largest term is exactly 2^0
#pragma unroll
                    for (int e = 0; e < 32; ++e) part += ex2((sr[e] - ref) * p.scale2);
                    sum = sum * ex2((m - ref) * p.scale2) + part;
                    m = mn;
                }
                x_max[half][i] = m;
                x_sum[half][i] = sum;
                x_pos[half][i] = pos2;
                workers_sync();
                const float m0 = x_max[0][i], m1 = x_max[1][i];
                m = fmaxf(m0, m1);
                const float mref = m == -INFINITY ? 0.f : m;                // all columns masked
                sum = x_sum[0][i] * ex2((m0 - mref) * p.scale2) +
                      x_sum[1][i] * ex2((m1 - mref) * p.scale2);
                pos2 = x_pos[0][i] + x_pos[1][i];                 // the other half holds 0
                const float lg = log2f(sum);          // once per row: the accurate one
                lse2 = m * p.scale2 + lg;
                lnsum = lg * 0.6931471805599453f;
                if (p.tiled) {
                    // one slot per passage tile; the combine kernel merges them
                    if (half == 0 && i < B_) {
                        p.part_m[(int64_t)blockIdx.z * p.B + x0 + i] = m * p.inv_tau;
                        p.part_l[(int64_t)blockIdx.z * p.B + x0 + i] = sum;
                        if (pos >= 0) p.pos_ws[x0 + i] = pos2 * p.inv_tau;
                    }
                    if (blockIdx.y == 0 && blockIdx.z == 0 && wt == 0 && p.zero_me) *p.zero_me = 0;
                }
                lse_nat = m * p.inv_tau + lnsum;
                m_row = m;
                lnsum_row = lnsum;
            }
            // ------------------------------ outputs of the forward (CTA 0) ------------------------
            if (slice == 0 && !p.tiled) {
                float term = 0.f;
                if (half == 0 && i < B_) {
                    if (p.op != GC_OP_BWD) {
                        const float pl = pos2 * p.inv_tau;
                        p.row_lse[i] = lse_nat;
                        if (p.pos_logit) p.pos_logit[i] = pl;
                        term = (m_row - pos2) * p.inv_tau + lnsum_row;   // no cancellation of two roundings
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
                // row i: a K-major A operand for dQ and, read by columns, an MN-major one for dP.
                // Rows past B get lse = +inf: all their weights are 0.
                const float neg_lse = i < B_ ? -lse2 : -INFINITY;
                const int pos_w = i < B_ ? pos : -1;
                for (int cb = 0; cb < nblk; ++cb) {
                    const int jb = j0 + 32 * cb;                  // 4 pieces of 8 columns
                    float w[32];
                    if (jb < N_) {
                        load_s<F32>(tmem + lane_addr, jb, w);
#pragma unroll
                        for (int e = 0; e < 32; ++e) w[e] = ex2(fmaf(w[e], p.scale2, neg_lse));
                        if ((unsigned)(masked - jb) < 32u) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) if (e == masked - jb) w[e] = 0.f;
                        }
                        if ((unsigned)(pos_w - jb) < 32u) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) if (e == pos_w - jb) w[e] -= 1.f;
                        }
                        if (jb + 32 > N_) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) if (jb + e >= N_) w[e] = 0.f;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) w[e] = 0.f;
                    }
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
                // A warp's 32 x 32 block goes through a 4 KB buffer (two per warp, over the
                // drained pipeline buffers) and leaves with one bulk tensor store, which clips it
                // at the matrix's last row and column.
                if (mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag)) {
                    tc_fence_after();
                    const int col = 64 * slice + 32 * half;
                    const uint32_t slot = base + (uint32_t)(warp - SM_FIRST_WORKER) * 8192u;
                    int n = 0;
                    for (int blk = 0; blk < 1 + ptiles; ++blk) {       // dQ, dP rows 0.., dP rows 128..
                        const int rows = blk == 0 ? p.B : p.N;
                        const int row0 = (blk == 0 ? x0 : y0 + 128 * (blk - 1)) + 32 * q;
                        const bool have = blk == 0 ? p.dQ != nullptr : p.dP != nullptr;
                        if (!have || row0 >= rows || col >= p.d) continue;
                        uint32_t v[32];
                        tmem_ld32(tmem + lane_addr + (blk == 0 ? COL_DQ : COL_DP + 64 * (blk - 1)) +
                                      32 * half, v);
                        if (n >= 2) {   // the store issued two blocks ago has read this buffer
                            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                            __syncwarp();
                        }
                        tmem_ld_wait();
                        const uint32_t buf = slot + (uint32_t)(n & 1) * 4096u;
                        stage_block(buf, v, blk == 0 ? p.out_scale_q : p.out_scale_p, lane);
                        __syncwarp();
                        // several tiles: plane = the tile of the other side (unscaled partials)
                        if (lane == 0)
                            tma_store_3d(blk == 0 ? &mapDQ : &mapDP, buf, col, row0,
                                         blk == 0 ? (p.plane_q ? (int)blockIdx.z : 0)
                                                  : (p.plane_p ? (int)blockIdx.y : 0));
                        ++n;
                    }
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                    __syncwarp();
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
cudaError_t launch_small_t(const CUtensorMap& mq, const CUtensorMap& mp, const CUtensorMap& mdq,
                           const CUtensorMap& mdp, const SmallParams& p, dim3 grid,
                           cudaStream_t st) {
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
    small_kernel<F32><<<grid, SM_THREADS, SM_DYN_SMEM, st>>>(mq, mp, mdq, mdp, p);
    return cudaGetLastError();
}

}  // namespace

// GRADCACHE_PLAN=sweeps in the environment (read at every call) keeps every problem on the sweep
// kernels (or the FMA tiles): a diagnostic switch, so that small shapes can still exercise the
// kernels that large ones run.
static bool small_plans_enabled() {
    const char* e = getenv("GRADCACHE_PLAN");
    return !(e && strcmp(e, "sweeps") == 0);
}

bool small_applicable(int64_t B, int64_t N, int d, int dtype) {
    if (!small_plans_enabled()) return false;
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
    // gradient outputs as [1][rows][d] for the epilogue's bulk tensor stores; a missing output
    // (gc_loss_fwd; gc_loss_bwd with one of the two) gets a map of the other, never written
    CUtensorMap mdq = mq, mdp = mp;
    if (dQ && !make_out_map(&mdq, dQ, pr.B, pr.d, lddq, 1)) return cudaErrorInvalidValue;
    if (dP && !make_out_map(&mdp, dP, pr.N, pr.d, lddp, 1)) return cudaErrorInvalidValue;
    SmallParams p{};
    p.B = (int)pr.B; p.N = (int)pr.N; p.d = pr.d;
    p.op = op;
    p.mask_mode = pr.mask_mode;
    p.mask_shift = (int)pr.mask_shift;
    p.scale2 = 1.4426950408889634f / pr.tau;
    p.inv_tau = 1.f / pr.tau;
    const float batch = (float)(pr.b_total > 0 ? pr.b_total : pr.B);
    p.out_scale = 1.f / (batch * pr.tau);
    p.out_scale_q = p.out_scale_p = p.out_scale;
    p.inv_mean = 1.f / batch;
    p.pos_idx = pr.pos_idx;
    p.row_lse_in = row_lse_in;
    p.loss = loss; p.row_lse = row_lse; p.pos_logit = pos_logit;
    p.dQ = dQ; p.lddq = lddq; p.dP = dP; p.lddp = lddp;
    p.dev_status = dev_status;
    const dim3 grid(op == GC_OP_FWD ? 1u : (unsigned)((pr.d + 63) / 64));
    return f32 ? launch_small_t<true>(mq, mp, mdq, mdp, p, grid, st)
               : launch_small_t<false>(mq, mp, mdq, mdp, p, grid, st);
}

// Batches of a few tiles (query tiles of 128 x passage tiles of 128 for fp32, of 256 for bf16) run
// the same kernel once per tile pair and column slice: the forward launch leaves one (max, sum)
// slot per passage tile and row for the combine kernel, the gradient launch (row_lse given)
// writes every tile pair's slices as planes of partial sums that a reduce kernel adds in index
// order.  Every CTA of a tile pair forms that pair's logits, so the work grows with d / 64: a plan
// for batches where launches, not arithmetic, set the time.  fp32: whatever its partial planes
// allow (what serves fp32 otherwise is the FMA-tile plan, which is slower at every size); bf16: while the gradient launch is at most two
// waves of CTAs (measured: 37-42 us against 58-71 us for the sweeps at 300 x 520 x 640 or
// 1000 x 1000 x 128, 48-51 us against 68-70 us at 385 x 900 x 768 or 512 x 1024 x 768 with 192
// CTAs; at 1030 x 1300 x 768, 648 CTAs, 87 us against 69 us: there the sweeps are faster).
bool small_tiled_applicable(int64_t B, int64_t N, int d, int dtype) {
    if (!small_plans_enabled()) return false;
    if (d % 8 != 0 || d > 4096 || small_applicable(B, N, d, dtype)) return false;
    const int64_t xt = small_tiles_x(B), yt = small_tiles_y(N, dtype);
    const int64_t ctas = xt * yt * ((d + 63) / 64);
    if (dtype == GC_F32) {
        // as long as the planes of partial sums stay within 2 GiB: the alternative for fp32 is
        // the FMA-tile plan, which this plan outruns about five times at every size measured
        const double plane_bytes = ((double)yt * (double)B + (double)xt * (double)N) * d * 4.0;
        return xt <= 65535 && yt <= 65535 && plane_bytes <= 2147483648.0;
    }
    return dtype == GC_BF16 && xt * yt <= 64 && ctas <= 2 * sm_count();
}
int small_tiles_x(int64_t B) { return (int)((B + 127) / 128); }
int small_tiles_y(int64_t N, int dtype) {
    return dtype == GC_F32 ? (int)((N + 127) / 128) : (int)((N + 255) / 256);
}
namespace {
bool small_in_maps(const Problem& pr, CUtensorMap* mq, CUtensorMap* mp) {
    return pr.dtype == GC_F32 ? make_map_f32(mq, pr.Q, pr.B, pr.d, pr.ldq, 128) &&
                                    make_map_f32(mp, pr.P, pr.N, pr.d, pr.ldp, 128)
                              : make_map(mq, pr.Q, pr.B, pr.d, pr.ldq, 128) &&
                                    make_map(mp, pr.P, pr.N, pr.d, pr.ldp, 128);
}
}  // namespace

// Forward of the tiled plan: slots part_m / part_l [tiles_y][B], pos_ws [B]; `red` is the scratch
// of the combine kernel that follows.
cudaError_t launch_small_tiled_fwd(const Problem& pr, float* part_m, float* part_l, float* pos_ws,
                                   float* red, int* dev_status, cudaStream_t st) {
    CUtensorMap mq, mp;
    if (!small_in_maps(pr, &mq, &mp)) return cudaErrorInvalidValue;
    SmallParams p{};
    p.B = (int)pr.B; p.N = (int)pr.N; p.d = pr.d;
    p.op = GC_OP_FWD;
    p.mask_mode = pr.mask_mode;
    p.mask_shift = (int)pr.mask_shift;
    p.scale2 = 1.4426950408889634f / pr.tau;
    p.inv_tau = 1.f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.tiled = 1;
    p.part_m = part_m; p.part_l = part_l; p.pos_ws = pos_ws;
    p.zero_me = reinterpret_cast<int*>(red);
    p.dev_status = dev_status;
    const dim3 grid(1u, (unsigned)small_tiles_x(pr.B), (unsigned)small_tiles_y(pr.N, pr.dtype));
    return pr.dtype == GC_F32 ? launch_small_t<true>(mq, mp, mq, mp, p, grid, st)
                              : launch_small_t<false>(mq, mp, mq, mp, p, grid, st);
}

// Gradients of the tiled plan from row_lse.  With one passage tile dQ is final (scaled) in dQ,
// otherwise plane t of partial_q [tiles_y][B][d] holds passage tile t's unscaled share; likewise
// dP / partial_p [tiles_x][N][d].  Either output may be NULL.
cudaError_t launch_small_tiled_bwd(const Problem& pr, const float* row_lse, float* dQ, int64_t lddq,
                                   float* partial_q, float* dP, int64_t lddp, float* partial_p,
                                   int* dev_status, cudaStream_t st) {
    const int xt = small_tiles_x(pr.B), yt = small_tiles_y(pr.N, pr.dtype);
    CUtensorMap mq, mp;
    if (!small_in_maps(pr, &mq, &mp)) return cudaErrorInvalidValue;
    CUtensorMap mdq = mq, mdp = mp;
    if (dQ) {
        const bool ok = yt == 1 ? make_out_map(&mdq, dQ, pr.B, pr.d, lddq, 1)
                                : make_out_map(&mdq, partial_q, pr.B, pr.d, pr.d, yt);
        if (!ok) return cudaErrorInvalidValue;
    }
    if (dP) {
        const bool ok = xt == 1 ? make_out_map(&mdp, dP, pr.N, pr.d, lddp, 1)
                                : make_out_map(&mdp, partial_p, pr.N, pr.d, pr.d, xt);
        if (!ok) return cudaErrorInvalidValue;
    }
    SmallParams p{};
    p.B = (int)pr.B; p.N = (int)pr.N; p.d = pr.d;
    p.op = GC_OP_BWD;
    p.mask_mode = pr.mask_mode;
    p.mask_shift = (int)pr.mask_shift;
    p.scale2 = 1.4426950408889634f / pr.tau;
    p.inv_tau = 1.f / pr.tau;
    const float batch = (float)(pr.b_total > 0 ? pr.b_total : pr.B);
    p.out_scale = 1.f / (batch * pr.tau);          // planes are scaled by the reduce kernel
    p.out_scale_q = yt == 1 ? p.out_scale : 1.f;
    p.out_scale_p = xt == 1 ? p.out_scale : 1.f;
    p.pos_idx = pr.pos_idx;
    p.row_lse_in = row_lse;
    p.dQ = dQ; p.lddq = lddq; p.dP = dP; p.lddp = lddp;
    p.tiled = 1;
    p.plane_q = yt > 1; p.plane_p = xt > 1;
    p.dev_status = dev_status;
    const dim3 grid((unsigned)((pr.d + 63) / 64), (unsigned)xt, (unsigned)yt);
    return pr.dtype == GC_F32 ? launch_small_t<true>(mq, mp, mdq, mdp, p, grid, st)
                              : launch_small_t<false>(mq, mp, mdq, mdp, p, grid, st);
}

}  // namespace gc
