// Gradient sweeps for narrow rows (bf16, d = 64 or 128), where a 128 x 128 tile of logits costs
// the tensor pipe about as many cycles (S = X Y^T plus acc += W Y: 1024 at d = 128) as its
// exponentials cost the special-function units, so neither may wait for the other.
//
//   DQ  (Eq. 5)    x = 128 queries,  y streams passages: W = exp(S - lse_x) - onehot, acc += W Y
//   DP  (Eq. 6-7)  x = 128 passages, y streams queries:  W = exp(S - lse_y) - onehot, acc += W Y
//   DA  (Eq. 1+5)  forward fused into the dQ sweep with a scale fixed before the sweep: W =
//                  2^(s2 - ref2_x), ref2_x = the row's positive logit, positive column left out,
//                  row sums kept per part; row sums beyond 2^100 raise a flag that hands the call
//                  to the sweeps that track the maximum.
//
// Tensor memory holds the accumulator (128 columns), two W tiles (2 x 64 columns, packed bf16:
// the A operand of the accumulation MMAs) and two S tiles (2 x 128 columns, fp32) side by side,
// so an S tile is free again as soon as its logits have been read, two tiles ahead of the
// accumulation that consumes the weights made from them: the MMA warp issues S(t), then
// acc(t - 2).  Two groups of eight softmax warps take the even and the odd tiles; each group owns
// one S tile and one W tile.  A streamed tile Y (128 x d) is loaded once and serves both MMAs:
// K-major for S, MN-major for the accumulation.  (Measured alternatives at 8192 x 8192 x 128,
// this layout 0.100 ms per call: W in two shared-memory buffers 0.108-0.110, also with a third
// S tile or with X as a tensor-memory operand; 16-column pieces with the next piece's load in
// flight 0.103.)
//
// Warp roles (576 threads): warp 0 = TMA producer (in DP it also writes, per streamed tile, the
// 128 column constants -lse2_y and the tile row of pos_y to shared memory), warp 1 = MMA issuer
// and tensor-memory allocator, warps 2..17 = softmax / epilogue: per group two warps per
// tensor-memory lane quarter, each owning half of the tile's columns, one thread per tile row.
// Every wait is bounded: on a timeout the CTA raises GC_DEV_WAIT_LIMIT, drains and exits.
#include "tc_common.cuh"

namespace gc {

namespace {

enum { NMODE_DQ = 0, NMODE_DP = 1, NMODE_DA = 2 };

constexpr int NW_STAGES = 5;                 // streamed tiles in flight
constexpr int NW_SOFT = 16;                  // softmax warps: two groups of eight
constexpr int NW_THREADS = 32 * (2 + NW_SOFT);
constexpr uint32_t NCOL_ACC = 0, NCOL_W = 128, NCOL_S = 256;
constexpr int NW_SBUF = 2;                   // S tiles in tensor memory

struct NarrowParams {
    int64_t nx, ny;
    int64_t nq;               // number of queries B (pitch of the forward slots)
    int kc;                   // d / 64: 1 or 2
    int groups;               // parts of the streamed range
    int mask_mode;
    int64_t mask_delta;       // GC_MASK_SELF drops the pair (x, y) with y == x + mask_delta
    float c1;                 // log2(e) / tau
    float inv_tau;
    float out_scale;
    const float* row_lse;
    const int32_t* pos_idx;
    float* part_m;
    float* part_l;
    float* pos_logit;
    const float* row_ref;     // DA: per-query anchor of the weights, log2 domain
    int* range_flag;          // DA: set to 1 when a row sum leaves the range the anchor allows
    int* dev_status;
    Gate gate;                // closed: the kernel returns at once
    int* zero_me;             // DA: the ticket word of the reduction that follows
};

struct NBars {
    uint64_t x_full;
    uint64_t y_full[NW_STAGES];
    uint64_t y_empty[NW_STAGES];
    uint64_t c_full[NW_STAGES];   // DP: the column constants of the stage are written
    uint64_t s_full[NW_SBUF];
    uint64_t s_free[NW_SBUF];     // a group has read the S tile
    uint64_t w_full[2];
    uint64_t w_empty[2];          // the accumulation MMAs that read W tile b have completed
    uint64_t acc_full;
};

template <int MODE>
__global__ void __launch_bounds__(NW_THREADS, 1)
narrow_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
              const __grid_constant__ CUtensorMap mapO, const NarrowParams p) {
    // All shared memory is dynamic: X and the ring (1024-byte aligned for the
    // 128-byte swizzle), then the barriers and the DP column constants.  With no static shared
    // memory the dynamic region starts on a 1024-byte boundary, so no slack is set aside for
    // alignment; a CTA that finds it otherwise
    // reports through dev_status instead of running.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t stage_bytes = (uint32_t)p.kc * CHUNK_BYTES;   // one tile of X or of Y
    const uint32_t data_bytes = (1 + NW_STAGES) * stage_bytes;
    NBars& bars = *reinterpret_cast<NBars*>(smem_raw + data_bytes);
    uint32_t& tmem_base_s = *reinterpret_cast<uint32_t*>(smem_raw + data_bytes + 192);
    int& abort_s = *reinterpret_cast<int*>(smem_raw + data_bytes + 196);
    // DP: -lse2 of the streamed queries, and the tile row of their positives (-1: not in this tile)
    float (*col_nlse)[128] = reinterpret_cast<float (*)[128]>(smem_raw + data_bytes + 256);
    int8_t (*col_rel)[128] =
        reinterpret_cast<int8_t (*)[128]>(smem_raw + data_bytes + 256 + NW_STAGES * 512);
    volatile int* abort_flag = &abort_s;
    if (gate_closed(p.gate)) return;            // same answer in every CTA
    if (MODE == NMODE_DA && blockIdx.x == 0 && threadIdx.x == 0 && p.zero_me) *p.zero_me = 0;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;
    const int g = (int)(blockIdx.x % (unsigned)p.groups);
    const int64_t x0 = (int64_t)(blockIdx.x / (unsigned)p.groups) * XROWS;
    int64_t lo, hi;
    part_range((p.ny + 127) / 128, p.groups, g, &lo, &hi);
    const int T = (int)(hi - lo);

    const uint32_t base = smem_u32(smem_raw);
    if (base & 1023u) {
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, GC_DEV_WAIT_LIMIT);
        return;
    }
    const uint32_t x_smem = base;
    const uint32_t y_smem = base + stage_bytes;               // the ring

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bars.x_full), 1);
        for (int s = 0; s < NW_STAGES; ++s) {
            mbar_init(smem_u32(&bars.y_full[s]), 1);
            mbar_init(smem_u32(&bars.y_empty[s]), 1);
            mbar_init(smem_u32(&bars.c_full[s]), 1);
        }
        for (int b = 0; b < NW_SBUF; ++b) {
            mbar_init(smem_u32(&bars.s_full[b]), 1);
            mbar_init(smem_u32(&bars.s_free[b]), NW_SOFT / 2);   // one arrival per warp of a group
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars.w_full[b]), NW_SOFT / 2);
            mbar_init(smem_u32(&bars.w_empty[b]), 1);
        }
        mbar_init(smem_u32(&bars.acc_full), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;

    if (warp == 0) {
        // ------------------------------ TMA producer --------------------------------------------
        // all 32 lanes run the loop; one elected lane issues the loads
        if (elect_one()) {
            mbar_expect_tx(smem_u32(&bars.x_full), stage_bytes);
            for (int c = 0; c < p.kc; ++c)
                tma_load_2d(x_smem + c * CHUNK_BYTES, &mapX, c * 64, (int)x0,
                            smem_u32(&bars.x_full));
        }
        int stage = 0;
        uint32_t phase = 0;
        for (int t = 0; t < T; ++t) {
            if (!mbar_wait(smem_u32(&bars.y_empty[stage]), phase ^ 1u, abort_flag)) break;
            const int64_t y0 = (lo + t) * 128;
            if (elect_one()) {
                const uint32_t full = smem_u32(&bars.y_full[stage]);
                mbar_expect_tx(full, stage_bytes);
                for (int c = 0; c < p.kc; ++c)
                    tma_load_2d(y_smem + stage * stage_bytes + c * CHUNK_BYTES, &mapY, c * 64,
                                (int)y0, full);
            }
            if (MODE == NMODE_DP) {   // the column constants of the tile: four per lane
                float nl[4];
                int rel[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int64_t y = y0 + lane + 32 * k;
                    float lse_y = INFINITY;
                    int32_t pos_y = -1;
                    if (y < p.ny) {
                        lse_y = p.row_lse[y];
                        pos_y = p.pos_idx[y];
                    }
                    nl[k] = -lse_y * 1.4426950408889634f;
                    const int64_t r = (int64_t)pos_y - x0;
                    rel[k] = (pos_y >= 0 && r >= 0 && r < XROWS) ? (int)r : -1;
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    col_nlse[stage][lane + 32 * k] = nl[k];
                    col_rel[stage][lane + 32 * k] = (int8_t)rel[k];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.c_full[stage]));
            }
            if (++stage == NW_STAGES) { stage = 0; phase ^= 1u; }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ----------------------------------------------
        // all 32 lanes run the loop; one elected lane issues the MMAs and commits
        const uint32_t idesc_s = instr_desc(128, false);
        const uint32_t idesc_acc = instr_desc(64 * p.kc, true);
        const uint32_t x_lo = desc_lo(x_smem, 0);
        const uint32_t ring_lo = desc_lo(y_smem, CHUNK_BYTES);   // LBO: next 64-column chunk
        constexpr uint32_t CH_LO = CHUNK_BYTES >> 4;
        const uint32_t stage_lo = stage_bytes >> 4;
        bool ok = mbar_wait(smem_u32(&bars.x_full), 0, abort_flag);
        tc_fence_after();
        int s_stage = 0, a_stage = 0, s_buf = 0;   // S tile t lives in buffer t % NW_SBUF
        uint32_t s_phase = 0, s_par = 0;           // (t / NW_SBUF) & 1
        for (int t = 0; t < T + 2 && ok; ++t) {
            if (t < T) {
                ok = mbar_wait(smem_u32(&bars.y_full[s_stage]), s_phase, abort_flag);
                if (!ok) break;
                if (t >= NW_SBUF) {   // its group has read S(t - 2) out of this tile
                    ok = mbar_wait(smem_u32(&bars.s_free[s_buf]), s_par ^ 1u, abort_flag);
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem + NCOL_S + s_buf * 128;
                const uint32_t yb = ring_lo + s_stage * stage_lo;
                if (elect_one()) {
                    mma_ss<false, false>(d_tmem, x_lo, yb, idesc_s);
                    mma_ss<true, false>(d_tmem, x_lo + 2, yb + 2, idesc_s);
                    mma_ss<true, false>(d_tmem, x_lo + 4, yb + 4, idesc_s);
                    mma_ss<true, false>(d_tmem, x_lo + 6, yb + 6, idesc_s);
                    if (p.kc == 2) {
                        mma_ss<true, false>(d_tmem, x_lo + CH_LO, yb + CH_LO, idesc_s);
                        mma_ss<true, false>(d_tmem, x_lo + CH_LO + 2, yb + CH_LO + 2, idesc_s);
                        mma_ss<true, false>(d_tmem, x_lo + CH_LO + 4, yb + CH_LO + 4, idesc_s);
                        mma_ss<true, false>(d_tmem, x_lo + CH_LO + 6, yb + CH_LO + 6, idesc_s);
                    }
                    tc_commit(smem_u32(&bars.s_full[s_buf]));
                }
                if (++s_buf == NW_SBUF) { s_buf = 0; s_par ^= 1u; }
                if (++s_stage == NW_STAGES) { s_stage = 0; s_phase ^= 1u; }
            }
            if (t >= 2) {
                const int u = t - 2, b = u & 1;
                ok = mbar_wait(smem_u32(&bars.w_full[b]), (u >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t w_tmem = tmem + NCOL_W + b * 64;
                const uint32_t yb = ring_lo + a_stage * stage_lo;
                if (elect_one()) {
                    // k-step k: streamed rows 16 k .. 16 k + 15 = W columns 8 k .. 8 k + 7
                    if (u == 0) mma_ts<false, false>(tmem + NCOL_ACC, w_tmem, yb, idesc_acc);
                    else        mma_ts<true, false>(tmem + NCOL_ACC, w_tmem, yb, idesc_acc);
#pragma unroll
                    for (int k = 1; k < 8; ++k)
                        mma_ts<true, false>(tmem + NCOL_ACC, w_tmem + k * 8, yb + k * 128,
                                            idesc_acc);
                    tc_commit(smem_u32(&bars.y_empty[a_stage]));
                    tc_commit(smem_u32(&bars.w_empty[b]));
                }
                if (++a_stage == NW_STAGES) a_stage = 0;
            }
        }
        if (ok && elect_one()) tc_commit(smem_u32(&bars.acc_full));
    } else {
        // ------------------------------ softmax / epilogue warps --------------------------------
        const int sw = warp - 2;                       // 0..15
        const int grp = sw >> 3;                       // tiles grp, grp + 2, ...; S and W tile grp
        const int q = warp & 3;                        // tensor-memory lane quarter of this warp
        const int half = (sw & 7) >> 2;                // which half of the tile's columns
        const int row = q * 32 + lane;
        const int64_t x = x0 + row;
        const int64_t xm = x + p.mask_delta;           // the streamed index masked for this row
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const bool self_mask = (p.mask_mode == GC_MASK_SELF);
        const uint32_t wbuf = tmem + lane_addr + NCOL_W + grp * 64;
        bool ok = true;
        float lse2_x = 0.f, l_sum = 0.f;
        int32_t pos_x = -1;
        // DA may have been launched ahead of the anchor kernel's completion
        if (MODE == NMODE_DA) dep_wait();
        if (MODE != NMODE_DP && x < p.nx) {
            lse2_x = (MODE == NMODE_DA) ? p.row_ref[x] : p.row_lse[x] * 1.4426950408889634f;
            pos_x = p.pos_idx[x];
        }
        const uint64_t c1_2 = pack2(p.c1, p.c1), nref_2 = pack2(-lse2_x, -lse2_x);
        // The arithmetic of one block of NE = 32 columns: logits v of columns c0 .. c0 + 31 of the
        // tile at y0 -> packed bf16 weights.
        auto weights = [&](const uint32_t (&v)[32], int c0, int64_t y0, int stage,
                           uint32_t (&packed)[16]) {
            constexpr int NE = 32;
            const int64_t yb = y0 + c0;
            float w[NE];
            if (MODE == NMODE_DP) {
                const float4* nl = reinterpret_cast<const float4*>(&col_nlse[stage][c0]);
#pragma unroll
                for (int c = 0; c < NE; c += 4) {
                    const float4 n4 = nl[c >> 2];   // same address in every lane: broadcast
                    float e0, e1, e2, e3;
                    unpack2(fma2(pack2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), c1_2,
                                 pack2(n4.x, n4.y)), e0, e1);
                    unpack2(fma2(pack2(__uint_as_float(v[c + 2]), __uint_as_float(v[c + 3])),
                                 c1_2, pack2(n4.z, n4.w)), e2, e3);
                    w[c] = ex2(e0);                 // rows past ny: ex2(-inf) = 0
                    w[c + 1] = ex2(e1);
                    w[c + 2] = ex2(e2);
                    w[c + 3] = ex2(e3);
                }
                // one-hot: column c's query has its positive at row pos - x0 of this tile
                const int rel_row = col_rel[stage][c0 + (lane & (NE - 1))];
                const bool mine = lane < NE && rel_row >= q * 32 && rel_row < q * 32 + 32;
                unsigned hits = __ballot_sync(0xffffffffu, mine);
                if (__popc(hits) > 3) {
                    // many positives in this block (the tile where streamed queries meet their
                    // own positives): every column in turn, three instructions each
#pragma unroll
                    for (int c = 0; c < NE; ++c)
                        if (__shfl_sync(0xffffffffu, rel_row, c) == row) w[c] -= 1.f;
                } else {
                    while (hits) {
                        const int col = __ffs(hits) - 1;
                        hits &= hits - 1;
                        const int target = __shfl_sync(0xffffffffu, rel_row, col) - q * 32;
                        if (lane == target) {
#pragma unroll
                            for (int c = 0; c < NE; ++c)
                                if (c == col) w[c] -= 1.f;
                        }
                    }
                }
            } else {
                if (MODE == NMODE_DA) {
                    const bool has_pos = pos_x >= yb && pos_x < yb + NE && pos_x < p.ny &&
                                         !(self_mask && xm == pos_x);
                    if (has_pos) {
                        const int rel = (int)(pos_x - yb);
                        float sp = 0.f;
#pragma unroll
                        for (int c = 0; c < NE; ++c)
                            if (c == rel) sp = __uint_as_float(v[c]);
                        p.pos_logit[x] = sp * p.inv_tau;
                    }
                }
                // exponents two at a time (one issue slot per pair)
#pragma unroll
                for (int c = 0; c < NE; c += 2) {
                    float e0, e1;
                    unpack2(fma2(pack2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])), c1_2,
                                 nref_2), e0, e1);
                    w[c] = ex2(e0);
                    w[c + 1] = ex2(e1);
                }
                if (MODE == NMODE_DQ && pos_x >= yb && pos_x < yb + NE) {
                    const int rel = (int)(pos_x - yb);
#pragma unroll
                    for (int c = 0; c < NE; ++c)
                        if (c == rel) w[c] -= 1.f;
                }
                if (yb + NE > p.ny) {
#pragma unroll
                    for (int c = 0; c < NE; ++c)
                        if (yb + c >= p.ny) w[c] = 0.f;
                }
            }
            if (self_mask && xm >= yb && xm < yb + NE) {
                const int rel = (int)(xm - yb);
#pragma unroll
                for (int c = 0; c < NE; ++c)
                    if (c == rel) w[c] = 0.f;
            }
            if (MODE == NMODE_DA) {
                // the weights are positive, so the row sum bounds the largest of them
                uint64_t sa = pack2(w[0], w[1]), sb = pack2(w[2], w[3]);
#pragma unroll
                for (int c = 4; c < NE; c += 4) {
                    sa = add2(sa, pack2(w[c], w[c + 1]));
                    sb = add2(sb, pack2(w[c + 2], w[c + 3]));
                }
                float s0, s1;
                unpack2(add2(sa, sb), s0, s1);
                l_sum += s0 + s1;
                if (pos_x >= yb && pos_x < yb + NE) {      // positive: fp32, in the finalize
                    const int rel = (int)(pos_x - yb);
#pragma unroll
                    for (int c = 0; c < NE; ++c)
                        if (c == rel) w[c] = 0.f;
                }
            }
#pragma unroll
            for (int r = 0; r < NE / 2; ++r) {
                __nv_bfloat162 h = __floats2bfloat162_rn(w[2 * r], w[2 * r + 1]);
                packed[r] = *reinterpret_cast<uint32_t*>(&h);
            }
        };
        // A warp takes its 64 columns of a tile as two blocks of 32 in a loop that is not
        // unrolled (the body is long: unrolled, its first pass runs at instruction-fetch speed).
        const int col0 = half * 64;
        for (int t = grp; t < T && ok; t += 2) {
            const int n = t >> 1;                      // tiles this group has finished
            const int stage = t % NW_STAGES;
            const int64_t y0 = (lo + t) * 128;
            if (MODE == NMODE_DP) {
                ok = mbar_wait(smem_u32(&bars.c_full[stage]), (uint32_t)(t / NW_STAGES) & 1u,
                               abort_flag);
                if (!ok) break;
            }
            const int sb = t % NW_SBUF;
            ok = mbar_wait(smem_u32(&bars.s_full[sb]), (uint32_t)(t / NW_SBUF) & 1u, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sbuf = tmem + lane_addr + NCOL_S + sb * 128;
#pragma unroll 1
            for (int j = 0; j < 2; ++j) {
                uint32_t v[32], pk[16];
                tmem_ld32(sbuf + col0 + 32 * j, v);
                tmem_ld_wait();
                if (j == 1) {   // the S tile may be overwritten
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.s_free[sb]));
                }
                weights(v, col0 + 32 * j, y0, stage, pk);
                if (j == 0 && n >= 1) {   // acc(t - 2) has read this W tile
                    ok = mbar_wait(smem_u32(&bars.w_empty[grp]), (n - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                }
                tmem_st16(wbuf + (col0 >> 1) + 16 * j, pk);
            }
            if (!ok) break;
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.w_full[grp]));
        }
        if (MODE == NMODE_DA && ok && x < p.nx) {
            // one (scale, sum) slot per row, part of the streamed range, softmax group and
            // column half
            const int64_t slot = (int64_t)((2 * g + grp) * 2 + half) * p.nq + x;
            p.part_m[slot] = lse2_x * 0.69314718055994531f;
            p.part_l[slot] = l_sum;
            // sums beyond 2^100 (or not finite) cannot be accumulated safely
            if (!(l_sum <= 1.2676506e30f)) *p.range_flag = 1;
        }
        // epilogue: one 32 x 32 block of the accumulator per warp (lane quarter q, columns 32 cb)
        if (ok) ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
        const int cb = 2 * grp + half;
        if (ok && cb < 2 * p.kc) {
            tc_fence_after();
            // every MMA and every load has completed: the ring is free
            const bool final_out = (p.groups == 1) && MODE != NMODE_DA;
            const uint32_t buf = y_smem + (uint32_t)sw * 4096u;
            uint32_t v[32];
            tmem_ld32(tmem + lane_addr + NCOL_ACC + cb * 32, v);
            tmem_ld_wait();
            stage_block(buf, v, final_out ? p.out_scale : 1.f, lane);
            __syncwarp();
            if (lane == 0) {
                tma_store_3d(&mapO, buf, cb * 32, (int)x0 + q * 32, final_out ? 0 : g);
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            }
            __syncwarp();
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
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <int MODE>
cudaError_t launch_narrow(const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& mo,
                          const NarrowParams& p, cudaStream_t st, bool overlap_prev) {
    // data, then 256 bytes of barriers and NW_STAGES x (512 + 128) bytes of column constants
    size_t dynamic_bytes = (size_t)(1 + NW_STAGES) * p.kc * CHUNK_BYTES + 256 +
                           NW_STAGES * 640;
    // keep one CTA per SM (each CTA allocates all 512 tensor-memory columns)
    if (dynamic_bytes < 120 * 1024) dynamic_bytes = 120 * 1024;
    // the attribute belongs to the (kernel, device) pair
    static bool configured_on[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured_on[dev]) {
        cudaError_t e = cudaFuncSetAttribute(narrow_kernel<MODE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)((1 + NW_STAGES) * 2 * CHUNK_BYTES + 256 + NW_STAGES * 640));
        if (e != cudaSuccess) return e;
        configured_on[dev] = true;
    }
    const int64_t ctas = ((p.nx + XROWS - 1) / XROWS) * p.groups;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(NW_THREADS);
    cfg.dynamicSmemBytes = dynamic_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, narrow_kernel<MODE>, mx, my, mo, p);
}

}  // namespace

bool narrow_applicable(int d, int dtype) { return dtype == GC_BF16 && (d == 64 || d == 128); }

// Forward fused into the dQ sweep with row_ref (log2 domain) as each row's fixed scale: writes
// (scale, sum) slots [4 groups][B] (scale = row_ref in natural-log units), pos_logit and the
// unscaled accumulators partial[groups][B][d] of sum_j 2^(s2_ij - ref_i) P_j over all allowed
// columns but the positive one; raises *range_flag when a row sum exceeds 2^100.
cudaError_t narrow_launch_anchored_dq(const FwdArgs& a, float* partial, int groups,
                                      const float* row_ref, int* range_flag, cudaStream_t st,
                                      bool overlap_prev) {
    const Problem& pr = a.p;
    CUtensorMap mx, my, mo;
    if (!make_map(&mx, pr.Q, pr.B, pr.d, pr.ldq, XROWS) ||
        !make_map(&my, pr.P, pr.N, pr.d, pr.ldp, 128) ||
        !make_out_map(&mo, partial, pr.B, pr.d, pr.d, groups))
        return cudaErrorInvalidValue;
    NarrowParams p{};
    p.nx = pr.B; p.ny = pr.N; p.nq = pr.B;
    p.kc = pr.d / 64; p.groups = groups;
    p.mask_mode = pr.mask_mode;
    p.mask_delta = pr.mask_shift;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.row_ref = row_ref;
    p.range_flag = range_flag;
    p.zero_me = reinterpret_cast<int*>(a.red);
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    return launch_narrow<NMODE_DA>(mx, my, mo, p, st, overlap_prev);
}

cudaError_t narrow_launch_sweep(const SweepArgs& a, cudaStream_t st) {
    CUtensorMap mx, my, mo;
    if (!make_map(&mx, a.X, a.nx, a.d, a.ldx, XROWS) || !make_map(&my, a.Y, a.ny, a.d, a.ldy, 128))
        return cudaErrorInvalidValue;
    const bool ok_map = a.groups == 1 ? make_out_map(&mo, a.out, a.nx, a.d, a.ldo, 1)
                                      : make_out_map(&mo, a.partial, a.nx, a.d, a.d, a.groups);
    if (!ok_map) return cudaErrorInvalidValue;
    NarrowParams p{};
    p.nx = a.nx; p.ny = a.ny; p.nq = 0;
    p.kc = a.d / 64; p.groups = a.groups;
    p.mask_mode = a.mask_mode;
    p.mask_delta = a.mask_delta;
    p.inv_tau = a.inv_tau;
    p.c1 = 1.4426950408889634f * a.inv_tau;
    p.out_scale = a.out_scale;
    p.row_lse = a.row_lse; p.pos_idx = a.pos_idx;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    if (a.mode == SWEEP_DQ) return launch_narrow<NMODE_DQ>(mx, my, mo, p, st, false);
    return launch_narrow<NMODE_DP>(mx, my, mo, p, st, false);
}

}  // namespace gc
