// Gradient sweeps for rows too wide for one accumulator (two column parts of at most 384
// columns): clusters of four CTAs that compute every logit tile once.
//
// The plain sweep gives each 384-column part of the accumulator its own CTA, and each of them
// recomputes the same S tiles.  Here the two CTA pairs of a cluster own the SAME two x tiles and
// one half of the columns each:
//
//     rank 0: x tile A, columns [0, d/2)      rank 2: x tile A, columns [d/2, d)
//     rank 1: x tile B, columns [0, d/2)      rank 3: x tile B, columns [d/2, d)
//
// Pair p = rank / 2 issues M = 256 MMAs over its two CTAs exactly as the paired sweep does.  The
// pairs take turns: pair (t mod 2) computes S(t) and its weights W(t) for both x tiles, writes W
// to its own shared memory and copies it to the CTA that holds the same x tile in the other pair
// (rank ^ 2) through distributed shared memory.  Every pair then runs acc(t) += W(t) Y(t) on its
// own column half for every t.  Per y tile a cluster therefore executes one S tile pair and two
// accumulation tile pairs instead of two and two, and streams X only on its duty tiles.
//
// Order of the tensor work of pair p (duty tiles p, p + 2, ...):
//     S(p); then for j = 0, 1, ...: S(2j + 2 + p), acc(2j), acc(2j + 1)
// so the weights of a round are one S phase old when they are needed and two W buffers (tile
// parity) suffice.  Every wait is bounded; DQ and DP modes take row_lse as an input, FA is the
// forward fused into the dQ sweep with the positive logit as the fixed scale of each row.
#include "tc_common.cuh"

namespace gc {

namespace {

enum { QMODE_DQ = 1, QMODE_DP = 2, QMODE_FA = 3 };

struct QuadParams {
    int64_t nx, ny;
    int64_t nq;               // number of queries B (pitch of the forward slot arrays)
    int nslots;               // DP: forward slots per query to merge (0: read row_lse)
    int kc;                   // d / 64
    int dpc;                  // chunks per column half
    int groups;
    int nstage;
    int mask_mode;
    float c1;                 // log2(e) / tau
    float inv_tau;
    float out_scale;
    const float* row_lse;
    const int32_t* pos_idx;
    const float* row_ref;     // FA: anchor of each query's weights, log2 domain
    float* part_m;            // FA: [4 groups][B] slots (scale, natural log), written
    float* part_l;            // FA: [4 groups][B] slots (sum), written
    const float* slot_m;      // DP with nslots > 0: the slots a forward sweep wrote
    const float* slot_l;
    float* pos_logit;         // FA
    int* range_flag;          // FA
    int* dev_status;
    int64_t mask_delta;       // GC_MASK_SELF drops the pair (x, y) with y == x + mask_delta
    Gate gate;
    int* zero_me;
};

constexpr int Q_XRES = 0;     // X chunks that stay resident (a deeper ring serves better)

struct QBars {
    uint64_t x_full;
    uint64_t y_full[MAX_STAGES];
    uint64_t y_empty[MAX_STAGES];
    // A remote arrive with cluster-scope release costs the arriving warp well over a thousand
    // cycles, so the softmax warps only ever arrive on barriers of their own CTA; the MMA warp of
    // the pair's second CTA, otherwise idle, forwards each completed phase to the leader.
    uint64_t s_full;           // S tile of the duty pair complete (both CTAs of the pair)
    uint64_t s_read;           // this CTA's 8 softmax warps have read the S tile
    uint64_t s_read_peer;      // leader: forwarded s_read of the second CTA
    uint64_t w_done;           // this CTA's 8 softmax warps have written their part of W
    uint64_t w_done_peer;      // leader: forwarded w_done of the second CTA
    uint64_t w_recv;           // the other pair's W has landed here (1 arrival + 32 KB)
    uint64_t w_peer;           // leader: forwarded w_recv of the second CTA
    uint64_t w_empty[2][2];    // [W buffer][consuming pair], committed to all four CTAs
    uint64_t acc_full;
};

__device__ __forceinline__ void tc_commit_mask(uint32_t bar, uint16_t mask) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
        "[%0], %1;"
        ::"r"(bar), "h"(mask) : "memory");
}
// arrive on a barrier of another CTA and add to the bytes it expects
__device__ __forceinline__ void mbar_arrive_expect_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;"
                 ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// shared memory of this CTA -> shared memory of another CTA of the cluster, counted on a barrier
// of the destination CTA
__device__ __forceinline__ void dsmem_copy(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes,
                                           uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst_cluster), "r"(src_cta), "r"(bytes), "r"(bar_cluster) : "memory");
}

template <int MODE>
__global__ void __launch_bounds__(NTHREADS, 1)
quad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
            const __grid_constant__ CUtensorMap mapYh, const __grid_constant__ CUtensorMap mapO,
            const QuadParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) QBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;
    if (gate_closed(p.gate)) return;            // same answer in every CTA
    if (MODE == QMODE_FA && blockIdx.x == 0 && threadIdx.x == 0 && p.zero_me) *p.zero_me = 0;

    constexpr int SN = 128;
    constexpr uint32_t S_COL0 = TMEM_COLS - SN;
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;

    const uint32_t rank = cluster_ctarank();        // 0..3
    const int pr = (int)(rank >> 1);                // pair = column half = duty parity
    const int side = (int)(rank & 1);               // which of the two x tiles
    const bool leader = (side == 0);
    const uint32_t leader_rank = rank & ~1u;
    const uint16_t pair_mask = (uint16_t)(3u << (2 * pr));

    int unit = (int)(blockIdx.x >> 2);
    const int g = unit % p.groups;
    unit /= p.groups;
    const int64_t xt = 2 * (int64_t)unit + side;
    const int64_t x0 = xt * XROWS;
    const int c_begin = pr * p.dpc;
    const int c_count = min(p.dpc, p.kc - c_begin);
    const int na = (c_count + 1) / 2;               // accumulation items (two chunks each)

    int64_t lo, hi;
    part_range((p.ny + SN - 1) / SN, p.groups, g, &lo, &hi);
    const int T = (int)(hi - lo);
    const int nd = (T - pr + 1) / 2;                // duty tiles of this pair: pr, pr + 2, ...
    const int rounds = (T + 1) / 2;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t x_smem = base;
    const uint32_t w_smem = base + Q_XRES * X_CHUNK_BYTES;      // two 32 KB W buffers (tile parity)
    const uint32_t y_smem = w_smem + 2u * 32768u;               // the ring, 16 KB stages
    const int xres = min(Q_XRES, p.kc);

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bars.x_full), 1);
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(smem_u32(&bars.y_full[s]), 1);
            mbar_init(smem_u32(&bars.y_empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.s_full), 1);
        mbar_init(smem_u32(&bars.s_read), NSOFT);
        mbar_init(smem_u32(&bars.s_read_peer), 1);
        mbar_init(smem_u32(&bars.w_done), NSOFT);
        mbar_init(smem_u32(&bars.w_done_peer), 1);
        mbar_init(smem_u32(&bars.w_recv), 1);
        mbar_init(smem_u32(&bars.w_peer), 1);
        for (int b = 0; b < 2; ++b)
            for (int q = 0; q < 2; ++q) mbar_init(smem_u32(&bars.w_empty[b][q]), 1);
        mbar_init(smem_u32(&bars.acc_full), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();               // all four CTAs' barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    auto in_leader = [&](uint32_t local) -> uint32_t { return mapa_u32(local, leader_rank); };

    // The tensor work of this pair, in issue order: op(kind, index) with kind 0 = S of duty tile
    // 2 index + pr, kind 1 = accumulation of tile index.  Producer and MMA issuer walk it alike.
    auto for_each_op = [&](auto&& op) {
        if (0 < nd) op(0, 0);
        for (int j = 0; j < rounds; ++j) {
            if (j + 1 < nd) op(0, j + 1);
            if (2 * j < T) op(1, 2 * j);
            if (2 * j + 1 < T) op(1, 2 * j + 1);
        }
    };

    if (warp < NPROD) {
        // ------------------------------ TMA producers -----------------------------------------
        const uint32_t x_full_bar = in_leader(smem_u32(&bars.x_full));
        if (warp == 0 && leader && elect_one())
            mbar_expect_tx(smem_u32(&bars.x_full), 2u * (uint32_t)xres * X_CHUNK_BYTES);
        for (int c = warp; c < xres; c += NPROD)
            if (elect_one())
                tma_load_2d_pair(x_smem + c * X_CHUNK_BYTES, &mapX, c * 64, (int)x0, x_full_bar);
        int next = 0;
        uint32_t next_phase = 0;
        bool ok = true;
        auto acquire = [&]() -> int {
            const int stage = next;
            const uint32_t phase = next_phase;
            if (++next == p.nstage) { next = 0; next_phase ^= 1u; }
            if (!ok || (stage & (NPROD - 1)) != warp) return -1;
            if (!mbar_wait(smem_u32(&bars.y_empty[stage]), phase ^ 1u, abort_flag)) {
                ok = false;
                return -1;
            }
            return stage;
        };
        // kind 0: this CTA's 64 rows of two Y chunks (S phase); kind 1: one X chunk of its 128
        // rows; kind 2: the Y chunk of its side for one accumulation item
        auto load_item = [&](int kind, int chunk0, int64_t row) {
            const int stage = acquire();
            if (stage < 0) return;
            const uint32_t full = smem_u32(&bars.y_full[stage]);
            const uint32_t full_bar = in_leader(full);
            const uint32_t dst = y_smem + stage * CHUNK_BYTES;
            if (elect_one()) {
                if (leader) mbar_expect_tx(full, 2 * CHUNK_BYTES);
                if (kind == 0) {
                    for (int i = 0; i < 2; ++i)
                        tma_load_2d_pair(dst + i * (CHUNK_BYTES / 2), &mapYh, (chunk0 + i) * 64,
                                         (int)(row + 64 * side), full_bar);
                } else if (kind == 1) {
                    tma_load_2d_pair(dst, &mapX, chunk0 * 64, (int)x0, full_bar);
                } else {
                    tma_load_2d_pair(dst, &mapY, (chunk0 + side) * 64, (int)row, full_bar);
                }
            }
        };
        for_each_op([&](int kind, int idx) {
            if (kind == 0) {
                const int64_t row = (lo + 2 * idx + pr) * SN;
                for (int c = 0; c < p.kc; c += 2) {
                    load_item(0, c, row);
                    for (int j = 0; j < 2; ++j)
                        if (c + j >= xres) load_item(1, c + j, x0);
                }
            } else {
                const int64_t row = (lo + idx) * SN;
                for (int a = 0; a < na; ++a) load_item(2, c_begin + 2 * a, row);
            }
        });
    } else if (warp == MMA_WARP) {
        if (leader) {
            // ------------------------------ MMA issuer ------------------------------------------
            const uint32_t idesc_s = instr_desc(SN, false, 2 * XROWS);
            const uint32_t idesc_acc = instr_desc(128, true, 2 * XROWS);
            constexpr uint32_t YCH_LO = (CHUNK_BYTES / 2) >> 4;
            constexpr uint32_t CH_LO = CHUNK_BYTES >> 4;
            const uint32_t x_lo = desc_lo(x_smem, 0);
            const uint32_t ring_lo = desc_lo(y_smem, CHUNK_BYTES);
            int next = 0;
            uint32_t next_phase = 0;
            bool ok = mbar_wait(smem_u32(&bars.x_full), 0, abort_flag);
            tc_fence_after();
            auto next_stage = [&]() -> int {
                const int stage = next;
                const uint32_t phase = next_phase;
                if (++next == p.nstage) { next = 0; next_phase ^= 1u; }
                if (!mbar_wait(smem_u32(&bars.y_full[stage]), phase, abort_flag)) {
                    ok = false;
                    return -1;
                }
                return stage;
            };
            for_each_op([&](int kind, int idx) {
                if (!ok) return;
                if (kind == 0) {
                    if (idx >= 1) {     // the softmax warps have read the previous duty tile
                        ok = mbar_wait(smem_u32(&bars.s_read), (idx - 1) & 1, abort_flag) &&
                             mbar_wait(smem_u32(&bars.s_read_peer), (idx - 1) & 1, abort_flag);
                        if (!ok) return;
                        tc_fence_after();
                    }
                    const uint32_t d_tmem = tmem + S_COL0;
                    for (int c = 0; c < p.kc && ok; c += 2) {
                        const int ys = next_stage();
                        if (!ok) return;
                        const uint32_t yb = ring_lo + ys * CH_LO;
                        for (int j = 0; j < 2 && ok; ++j) {
                            int xs = -1;
                            uint32_t xa = x_lo + (c + j) * CH_LO;
                            if (c + j >= xres) {
                                xs = next_stage();
                                if (!ok) return;
                                xa = ring_lo + xs * CH_LO;
                            }
                            const uint32_t yj = yb + j * YCH_LO;
                            if (elect_one()) {
                                if (c + j == 0) mma_ss<false, true>(d_tmem, xa, yj, idesc_s);
                                else            mma_ss<true, true>(d_tmem, xa, yj, idesc_s);
                                mma_ss<true, true>(d_tmem, xa + 2, yj + 2, idesc_s);
                                mma_ss<true, true>(d_tmem, xa + 4, yj + 4, idesc_s);
                                mma_ss<true, true>(d_tmem, xa + 6, yj + 6, idesc_s);
                                if (xs >= 0) tc_commit_mask(smem_u32(&bars.y_empty[xs]), pair_mask);
                                if (j == 1) tc_commit_mask(smem_u32(&bars.y_empty[ys]), pair_mask);
                            }
                        }
                    }
                    if (ok && elect_one()) tc_commit_mask(smem_u32(&bars.s_full), pair_mask);
                } else {
                    const int u = idx, b = u & 1, round = u >> 1;
                    if (b == pr) {
                        ok = mbar_wait(smem_u32(&bars.w_done), round & 1, abort_flag) &&
                             mbar_wait(smem_u32(&bars.w_done_peer), round & 1, abort_flag);
                    } else {
                        ok = mbar_wait(smem_u32(&bars.w_recv), round & 1, abort_flag) &&
                             mbar_wait(smem_u32(&bars.w_peer), round & 1, abort_flag);
                    }
                    if (!ok) return;
                    tc_fence_after();
                    const uint32_t w_lo = desc_lo(w_smem + b * 32768u, 0);   // K-major A operand
                    for (int a = 0; a < na && ok; ++a) {
                        const int ys = next_stage();
                        if (!ok) return;
                        const uint32_t yb = ring_lo + ys * CH_LO;
                        const uint32_t d_tmem = tmem + a * 128;
                        if (elect_one()) {
                            if (u == 0) mma_ss<false, true>(d_tmem, w_lo, yb, idesc_acc);
                            else        mma_ss<true, true>(d_tmem, w_lo, yb, idesc_acc);
#pragma unroll
                            for (int k = 1; k < SN / 16; ++k)
                                mma_ss<true, true>(d_tmem, w_lo + (k / 4) * CH_LO + (k % 4) * 2,
                                                   yb + k * 128, idesc_acc);
                            tc_commit_mask(smem_u32(&bars.y_empty[ys]), pair_mask);
                            // the W buffer may be rewritten, by either pair's softmax warps
                            if (a == na - 1)
                                tc_commit_mask(smem_u32(&bars.w_empty[b][pr]), (uint16_t)0xF);
                        }
                    }
                }
            });
            if (ok && elect_one()) tc_commit_mask(smem_u32(&bars.acc_full), pair_mask);
        } else {
            // Forwarder: the second CTA's completed phases (S tile read, W written, received W
            // landed) become single arrivals on the leader's barriers.  The three sequences are
            // polled together so that none waits behind another.
            const uint32_t fs = in_leader(smem_u32(&bars.s_read_peer));
            const uint32_t fw = in_leader(smem_u32(&bars.w_done_peer));
            const uint32_t fr = in_leader(smem_u32(&bars.w_peer));
            const int nrecv = (T - (1 - pr) + 1) / 2;       // tiles 1 - pr, 3 - pr, ... < T
            int js = 0, jw = 0, jr = 0;
            uint64_t t_last = global_ns();
            while (js < nd || jw < nd || jr < nrecv) {
                bool progress = false;
                if (js < nd && mbar_test(smem_u32(&bars.s_read), js & 1)) {
                    if (lane == 0) mbar_arrive_cluster(fs);
                    ++js;
                    progress = true;
                }
                if (jw < nd && mbar_test(smem_u32(&bars.w_done), jw & 1)) {
                    if (lane == 0) mbar_arrive_cluster(fw);
                    ++jw;
                    progress = true;
                }
                if (jr < nrecv && mbar_test(smem_u32(&bars.w_recv), jr & 1)) {
                    if (lane == 0) mbar_arrive_cluster(fr);
                    ++jr;
                    progress = true;
                }
                __syncwarp();
                if (progress) {
                    t_last = global_ns();
                } else {
                    if (*abort_flag) break;
                    if (global_ns() - t_last > WAIT_LIMIT_NS) {
                        *abort_flag = 1;
                        break;
                    }
                }
            }
        }
    } else {
        // ------------------------------ softmax / epilogue warps --------------------------------
        const int q = warp & 3;                        // tensor-memory lane quarter of this warp
        const int half = (warp - (NPROD + 1)) >> 2;    // which half of the tile's columns
        constexpr int CB_PER = SN / 64;
        static_assert(CB_PER == 2, "the softmax loop reads two 32-column blocks per thread");
        const int cb0 = half * CB_PER;
        const int row = q * 32 + lane;
        const int64_t x = x0 + row;
        const int64_t xm = x + p.mask_delta;     // the streamed index masked for this row
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const bool self_mask = (p.mask_mode == GC_MASK_SELF);
        bool ok = true;
        // W buffer pr (32 KB) goes as one copy to the same place in the CTA that holds this x tile
        // in the other pair; the last softmax warp sends it once all eight have written
        const uint32_t my_w = w_smem + pr * 32768u;
        const uint32_t remote_w = mapa_u32(my_w, rank ^ 2u);
        const uint32_t remote_bar = mapa_u32(smem_u32(&bars.w_recv), rank ^ 2u);
        const bool sender = (q == 3 && half == 1);
        auto put_w_block = [&](int j, const uint32_t (&pk)[16]) {
            const uint32_t line = w_smem + pr * 32768u + half * CHUNK_BYTES + row * 128;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t addr = line + (((4 * j + i) ^ (row & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                             ::"r"(addr), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                               "r"(pk[4 * i + 3]) : "memory");
            }
        };
        float lse2_x = 0.f, l = 0.f, wmax = 0.f;
        int32_t pos_x = -1;
        // FA may have been launched ahead of the anchor kernel's completion: row_ref, the range
        // flag and everything this role writes come after it
        if (MODE == QMODE_FA) dep_wait();
        if (MODE != QMODE_DP && x < p.nx) {
            lse2_x = (MODE == QMODE_FA) ? p.row_ref[x] : p.row_lse[x] * 1.4426950408889634f;
            pos_x = p.pos_idx[x];
        }
        for (int j = 0; j < nd; ++j) {
            const int t = 2 * j + pr;
            const int64_t y0 = (lo + t) * SN;
            float lse2_y[CB_PER] = {};
            int32_t pos_y[CB_PER] = {};
            if (MODE == QMODE_DP) {
#pragma unroll
                for (int jj = 0; jj < CB_PER; ++jj) {
                    const int64_t y = y0 + (cb0 + jj) * 32 + lane;
                    float lse_y = INFINITY;
                    if (y < p.ny)
                        lse_y = p.nslots > 0 ? combined_lse(p.slot_m, p.slot_l, p.nslots, p.nq, y)
                                             : p.row_lse[y];
                    lse2_y[jj] = lse_y * 1.4426950408889634f;
                    pos_y[jj] = (y < p.ny) ? p.pos_idx[y] : -1;
                }
            }
            ok = mbar_wait(smem_u32(&bars.s_full), j & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sbuf = tmem + lane_addr + S_COL0;
            // Both 32-column blocks are read at once, so that the S tile is free again; the
            // arithmetic then takes one block at a time in a loop that is not unrolled: the body is
            // long, and the first pass through it runs at instruction-fetch speed.
            uint32_t va[32], vb[32];
            tmem_ld32(sbuf + cb0 * 32, va);
            tmem_ld32(sbuf + (cb0 + 1) * 32, vb);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.s_read));  // the S tile may be overwritten
            uint32_t keep_a[16], keep_b[16];
#pragma unroll 1
            for (int jj = 0; jj < CB_PER; ++jj) {
                const int cb = cb0 + jj;
                uint32_t v[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] = jj == 0 ? va[c] : vb[c];
                const float lse2_yj = jj == 0 ? lse2_y[0] : lse2_y[CB_PER - 1];
                const int32_t pos_yj = jj == 0 ? pos_y[0] : pos_y[CB_PER - 1];
                const int64_t yb = y0 + cb * 32;
                float w[32];
                if (MODE == QMODE_FA) {
                    const bool has_pos = pos_x >= yb && pos_x < yb + 32 && pos_x < p.ny &&
                                         !(self_mask && xm == pos_x);
                    if (has_pos) {
                        const int rel = (int)(pos_x - yb);
                        float sp = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) sp = __uint_as_float(v[c]);
                        p.pos_logit[x] = sp * p.inv_tau;
                    }
                    float s0 = 0.f, s1 = 0.f, m0 = 0.f;
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        w[c] = ex2(fmaf(__uint_as_float(v[c]), p.c1, -lse2_x));
                        w[c + 1] = ex2(fmaf(__uint_as_float(v[c + 1]), p.c1, -lse2_x));
                    }
                    if (yb + 32 > p.ny) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (yb + c >= p.ny) w[c] = 0.f;
                    }
                    if (self_mask && xm >= yb && xm < yb + 32) {
                        const int rel = (int)(xm - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) w[c] = 0.f;
                    }
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        s0 += w[c];
                        s1 += w[c + 1];
                        m0 = fmaxf(m0, fmaxf(w[c], w[c + 1]));
                    }
                    l += s0 + s1;
                    wmax = fmaxf(wmax, m0);
                    if (pos_x >= yb && pos_x < yb + 32) {                  // positive: fp32 later
                        const int rel = (int)(pos_x - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) w[c] = 0.f;
                    }
                } else if (MODE == QMODE_DQ) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        w[c] = ex2(fmaf(__uint_as_float(v[c]), p.c1, -lse2_x));
                    if (pos_x >= yb && pos_x < yb + 32) {
                        const int rel = (int)(pos_x - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) w[c] -= 1.f;
                    }
                    if (yb + 32 > p.ny) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (yb + c >= p.ny) w[c] = 0.f;
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float ls = __shfl_sync(0xffffffffu, lse2_yj, c);
                        w[c] = ex2(fmaf(__uint_as_float(v[c]), p.c1, -ls));   // OOB: ex2(-inf)
                    }
                    // one-hot: column c's query has its positive at row pos - x0 of this tile
                    const int64_t rel_row = (int64_t)pos_yj - x0;
                    const bool mine = (pos_yj >= 0) && rel_row >= q * 32 && rel_row < q * 32 + 32;
                    unsigned hits = __ballot_sync(0xffffffffu, mine);
                    while (hits) {
                        const int col = __ffs(hits) - 1;
                        hits &= hits - 1;
                        const int target = (int)__shfl_sync(0xffffffffu, (int)rel_row, col) - q * 32;
                        if (lane == target) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c == col) w[c] -= 1.f;
                        }
                    }
                }
                if (MODE != QMODE_FA && self_mask && xm >= yb && xm < yb + 32) {
                    const int rel = (int)(xm - yb);
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c == rel) w[c] = 0.f;
                }
                uint32_t packed[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(w[2 * r], w[2 * r + 1]);
                    packed[r] = *reinterpret_cast<uint32_t*>(&h);
                }
                if (jj == 0) {
#pragma unroll
                    for (int r = 0; r < 16; ++r) keep_a[r] = packed[r];
                } else {
#pragma unroll
                    for (int r = 0; r < 16; ++r) keep_b[r] = packed[r];
                }
            }
            // W buffer pr of both pairs must have been consumed (accumulation of tile t - 2)
            if (j >= 1) {
                ok = mbar_wait(smem_u32(&bars.w_empty[pr][0]), (j - 1) & 1, abort_flag) &&
                     mbar_wait(smem_u32(&bars.w_empty[pr][1]), (j - 1) & 1, abort_flag);
                if (!ok) break;
            }
            put_w_block(0, keep_a);
            put_w_block(1, keep_b);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.w_done));
            if (sender) {
                ok = mbar_wait(smem_u32(&bars.w_done), j & 1, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_cluster(remote_bar, 32768u);
                    dsmem_copy(remote_w, my_w, 32768u, remote_bar);
                }
                __syncwarp();
            }
        }
        if (MODE == QMODE_FA && ok && x < p.nx) {
            // one (scale, sum) slot per row, part of the streamed range, duty pair and column half
            const int64_t slot = (int64_t)((2 * g + pr) * 2 + half) * p.nq + x;
            p.part_m[slot] = lse2_x * 0.69314718055994531f;
            p.part_l[slot] = l;
            // weights beyond 2^100 (or not finite) cannot be accumulated safely
            if (!(wmax <= 1.2676506e30f)) *p.range_flag = 1;
        }
        // epilogue: accumulator columns of this CTA's half -> global memory
        if (ok) ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
        if (ok) {
            tc_fence_after();
            const bool final_out = (p.groups == 1) && MODE != QMODE_FA;
            const uint32_t slot = y_smem + (uint32_t)(warp - (NPROD + 1)) * 8192u;
            store_acc_blocks(tmem + lane_addr, c_count * 2, half, slot,
                             final_out ? p.out_scale : 1.f, lane, &mapO, c_begin * 64,
                             (int)x0 + q * 32, final_out ? 0 : g);
        }
    }

    // ------------------------------ teardown ------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        uint64_t t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, GC_DEV_WAIT_LIMIT);
        __syncthreads();
    }
    cluster_sync_all();   // no MMA, load, copy or arrival of another CTA touches this one any more
    if (warp == MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

template <int MODE>
cudaError_t launch_quad(const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& myh,
                        const CUtensorMap& mo, QuadParams p, int64_t clusters, cudaStream_t st,
                        bool overlap_prev = false) {
    const size_t fixed = 1024 + (size_t)Q_XRES * X_CHUNK_BYTES + 2 * 32768;
    int ns = (int)((SMEM_LIMIT - SMEM_STATIC_RESERVE - fixed) / CHUNK_BYTES);
    if (ns > MAX_STAGES) ns = MAX_STAGES;
    p.nstage = ns;
    const size_t dynamic_bytes = fixed + (size_t)ns * CHUNK_BYTES;
    // the attribute belongs to the (kernel, device) pair
    static bool configured_on[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    bool& configured = configured_on[dev];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(quad_kernel<MODE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(SMEM_LIMIT - SMEM_STATIC_RESERVE));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(clusters * 4));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = dynamic_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 4;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, quad_kernel<MODE>, mx, my, myh, mo, p);
}

}  // namespace


// Two column halves of an even number of chunks each, at most 384 columns per half, more than
// one x tile.
bool quad_applicable(int64_t nx, int d) {
    const int kc = d / 64;
    return d % 128 == 0 && parts_for(kc) == 2 && nx > XROWS;
}

int quad_groups(int64_t nx, int64_t ny) {
    const int64_t clusters = ((nx + XROWS - 1) / XROWS + 1) / 2;
    const int64_t steps = (ny + 127) / 128;
    int64_t g = (sm_count() / 4) / clusters;
    if (g < 1) g = 1;
    if (g > steps / 2) g = steps / 2;     // at least one tile per pair and part
    if (g < 1) g = 1;
    if (g > 8) g = 8;
    return (int)g;
}

cudaError_t quad_launch_sweep(const SweepArgs& a, cudaStream_t st) {
    const int kc = a.d / 64;
    CUtensorMap mx, my, myh, mo;
    if (!make_map(&mx, a.X, a.nx, a.d, a.ldx, XROWS) || !make_map(&my, a.Y, a.ny, a.d, a.ldy, 128) ||
        !make_map(&myh, a.Y, a.ny, a.d, a.ldy, 64))
        return cudaErrorInvalidValue;
    QuadParams p{};
    p.nx = a.nx; p.ny = a.ny;
    p.kc = kc; p.dpc = chunks_per_part(kc); p.groups = a.groups;
    p.mask_mode = a.mask_mode;
    p.mask_delta = a.mask_delta;
    p.inv_tau = a.inv_tau;
    p.c1 = 1.4426950408889634f * a.inv_tau;
    p.out_scale = a.out_scale;
    p.row_lse = a.row_lse; p.pos_idx = a.pos_idx;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    if (a.mode == SWEEP_DP && a.slot_l) {
        p.slot_m = a.slot_m; p.slot_l = a.slot_l; p.nslots = a.slots; p.nq = a.ny;
    }
    const bool ok_map = a.groups == 1 ? make_out_map(&mo, a.out, a.nx, a.d, a.ldo, 1)
                                      : make_out_map(&mo, a.partial, a.nx, a.d, a.d, a.groups);
    if (!ok_map) return cudaErrorInvalidValue;
    const int64_t clusters = (((a.nx + XROWS - 1) / XROWS + 1) / 2) * a.groups;
    if (a.mode == SWEEP_DQ) return launch_quad<QMODE_DQ>(mx, my, myh, mo, p, clusters, st);
    return launch_quad<QMODE_DP>(mx, my, myh, mo, p, clusters, st);
}

// Forward fused into the dQ sweep with the positive logit as each row's fixed scale (row_ref,
// log2 domain): writes (scale, sum) slots [4 groups][B] (scale = row_ref in natural-log units),
// pos_logit and the unscaled accumulators partial[groups][B][d] of sum_j 2^(s2_ij - ref_i) P_j
// over all allowed columns but the positive one; raises *range_flag when a weight exceeds 2^100.
cudaError_t quad_launch_fused_dq(const FwdArgs& a, float* partial, int groups, const float* row_ref,
                                 int* range_flag, cudaStream_t st, bool overlap_prev) {
    const Problem& pr = a.p;
    const int kc = pr.d / 64;
    CUtensorMap mx, my, myh, mo;
    if (!make_map(&mx, pr.Q, pr.B, pr.d, pr.ldq, XROWS) ||
        !make_map(&my, pr.P, pr.N, pr.d, pr.ldp, 128) ||
        !make_map(&myh, pr.P, pr.N, pr.d, pr.ldp, 64) ||
        !make_out_map(&mo, partial, pr.B, pr.d, pr.d, groups))
        return cudaErrorInvalidValue;
    QuadParams p{};
    p.nx = pr.B; p.ny = pr.N; p.nq = pr.B;
    p.kc = kc; p.dpc = chunks_per_part(kc); p.groups = groups;
    p.mask_mode = pr.mask_mode;
    p.mask_delta = pr.mask_shift;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.row_ref = row_ref;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.range_flag = range_flag;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    p.zero_me = reinterpret_cast<int*>(a.red);
    const int64_t clusters = (((pr.B + XROWS - 1) / XROWS + 1) / 2) * groups;
    return launch_quad<QMODE_FA>(mx, my, myh, mo, p, clusters, st, overlap_prev);
}

}  // namespace gc
