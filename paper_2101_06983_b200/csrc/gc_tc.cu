// Tensor-core sweeps with one CTA, or one CTA pair, per (x tile, accumulator part): bf16 inputs
// with d a multiple of 64 (up to 4096).  TMA-staged tiles in 128-byte-swizzled shared memory,
// tcgen05 MMAs with fp32 accumulators in tensor memory, the softmax arithmetic in registers.  One
// kernel template serves five sweeps:
//
//   FWD  (Eq. 1)    x = 128 queries,  y streams passages: S = X Y^T, online row max / sum.
//   DQ   (Eq. 5)    x = 128 queries,  y streams passages: W = exp(S - lse_x) - onehot, acc += W Y
//   DP   (Eq. 6-7)  x = 128 passages, y streams queries:  W = exp(S - lse_y) - onehot, acc += W Y
//   FQ   (Eq. 1+5)  forward fused into the dQ sweep: the row maximum runs online, W = exp(S -
//                   m_ref) with the positive column left out, acc += W Y; the accumulator is
//                   rescaled only when the maximum grows by more than 2^8.  A finalize pass forms
//                   (sum_g acc_g exp(m_g - lse) + (p_pos - 1) P_pos) / (B tau), positive term in fp32.
//   DA   (Eq. 1+5)  forward fused into the dQ sweep with a scale fixed before the sweep: W =
//                   2^(s2 - ref2_x), ref2_x = the row's positive logit (anchor kernel), positive
//                   column left out, row sums kept per part; used for rows narrow enough for two S
//                   buffers, where no running maximum has to be tracked.  Weights beyond 2^100
//                   raise a flag that hands the call to FWD + DQ + DP.
//   FS   (Eq. 1)    forward that also stores the bf16 weights 2^(s2 - ref2_x) of all pairs (the
//                   stored-weights comparison plan).
//
// Rows of two column halves with more than one x tile are served by the four-CTA sweeps of
// gc_quad.cu instead; there FQ and DP remain as the gated fallback.
//
// The stationary tile X (128 x d) stays resident in shared memory when d <= 512; for wider rows
// only its first chunks stay (6, or 2 beside shared-memory W buffers) and the others are
// re-streamed every step through the ring that also carries Y in (128 x 64) chunks.  Narrow rows
// double-buffer the S tile (128 x 128, fp32) in tensor memory and write W back over it as packed
// bf16 (A operand from tensor memory); wide rows have one S tile and, when paired, keep W in two
// shared-memory buffers so that S(t+1) is issued while softmax(t) runs.  The B operand of the
// accumulation MMA is the Y chunk read MN-major.  An accumulator of 128 x 768 fp32 does not fit
// the 512 tensor-memory columns, so wide rows are split into column parts (at most 384 columns),
// one CTA per part.  S is never written to global memory.
//
// Warp roles (352 threads): warps 0..1 = TMA producers (ring stages dealt out alternately), warp
// 2 = MMA issuer (and tensor-memory allocator), warps 3..10 = softmax / epilogue: two warps per
// tensor-memory lane quarter, each owning half of the tile's columns, one thread per tile row.
// Every wait is bounded: on a timeout the CTA raises GC_DEV_WAIT_LIMIT, drains and exits.
#include "tc_common.cuh"

namespace gc {

namespace {

// FQ: forward fused into dQ; FS: forward that also stores the bf16 weights
enum { MODE_FWD = 0, MODE_DQ = 1, MODE_DP = 2, MODE_FQ = 3, MODE_FS = 4, MODE_DA = 5 };

struct TcParams {
    int64_t nx, ny;
    int64_t nq;               // number of queries B (pitch of the forward partial arrays)
    int kc;                   // d / 64
    int xres;                 // X chunks [0, xres) stay resident, [xres, kc) are streamed
    int ipc;                  // chunks per ring item (1 or 2): a stage holds ipc * 16 KB
    int dparts, dpc;          // accumulator column parts and chunks per part
    int groups;
    int nstage;
    int mask_mode;
    float c1;                 // log2(e) / tau
    float inv_tau;
    float out_scale;
    const float* row_lse;
    const int32_t* pos_idx;
    float* out;
    int64_t ldo;
    float* partial;
    float* part_m;
    float* part_l;
    float* pos_logit;
    int* dev_status;
    const float* row_ref;     // FS, DA: per-query anchor of the weights, log2 domain
    int* range_flag;          // FS, DA: set to 1 when a weight leaves the range the anchor allows
    const float* slot_m;      // DP with nslots > 0: forward slots [nslots][ny] to merge instead of
    const float* slot_l;      //   reading row_lse
    int nslots;
    int64_t mask_delta;       // GC_MASK_SELF drops the pair (x, y) with y == x + mask_delta
    Gate gate;                // closed: the kernel returns at once
    int* zero_me;             // forward sweeps: the ticket word of the reduction that follows
};

struct Bars {
    uint64_t x_full;
    uint64_t y_full[MAX_STAGES];
    uint64_t y_empty[MAX_STAGES];
    uint64_t s_full[2];
    uint64_t w_full[2];
    uint64_t acc_full;
    uint64_t pair[4];          // FQ: the two softmax warps of a lane quarter agree on the row max
    uint64_t s_free;           // WS: every softmax warp has read the S tile (in the leader)
    uint64_t w_empty[2];       // WS: the MMAs that read W buffer b have completed
};

// ---------------------------------------------------------------------------------------------
// The sweep kernel
// ---------------------------------------------------------------------------------------------
// PAIR: the kernel runs as clusters of two CTAs that own two neighbouring x tiles of the same
// column part.  The leader (rank 0) issues every MMA with cta_group::2 (M = 256: 128 rows in each
// CTA's tensor memory); each CTA loads its own X chunks but only its half of every Y chunk (the
// 64 streamed rows of its rank for the S MMAs, the 64 columns of its rank for the accumulation
// MMAs), which halves the Y traffic into shared memory.  "Full" barriers live in the leader and
// count the bytes landing in both CTAs; "empty", s_full and acc_full are signalled in both CTAs by
// multicast commits; the softmax warps of both CTAs arrive on the leader's w_full.
// Narrow-row gradient sweeps (two S buffers, one CTA per tile) run two groups of softmax warps:
// group 0 takes the even tiles (S buffer 0), group 1 the odd ones (buffer 1).  A tile keeps the
// eight warps of its group busy for about three times as long as its MMAs take, so one group
// caps the sweep at one tile per softmax pass however many buffers there are.
template <int MODE, int NBUF, bool PAIR>
__host__ __device__ constexpr bool two_softmax_groups() {
    return NBUF == 2 && !PAIR && (MODE == MODE_DQ || MODE == MODE_DP || MODE == MODE_DA);
}
template <int MODE, int NBUF, bool PAIR>
__host__ __device__ constexpr int tc_threads() {
    return two_softmax_groups<MODE, NBUF, PAIR>() ? NTHREADS + 32 * NSOFT : NTHREADS;
}

template <int MODE, int SN, int NBUF, bool PAIR>
__global__ void __launch_bounds__((tc_threads<MODE, NBUF, PAIR>()), 1)
tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
          const __grid_constant__ CUtensorMap mapYh, const __grid_constant__ CUtensorMap mapO,
          const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float row_max_xch[2][XROWS];      // FQ: [column half][row] block maxima
    volatile int* abort_flag = &abort_s;
    if (gate_closed(p.gate)) return;            // same answer in every CTA
    if ((MODE == MODE_FWD || MODE == MODE_FS || MODE == MODE_FQ || MODE == MODE_DA) && blockIdx.x == 0 && threadIdx.x == 0 && p.zero_me) *p.zero_me = 0;

    static_assert(SN == 128, "a Y chunk is 128 rows: the same 16 KB as an X chunk");
    constexpr uint32_t S_COL0 = TMEM_COLS - NBUF * SN;  // S buffers sit at the top columns
    // WS ("W through shared memory"): paired wide-row sweeps write the bf16 weights to two
    // shared-memory buffers instead of over the single S tile.  The S tile is then free as soon as
    // the softmax warps have read it, S(t+1) is issued while softmax(t) computes, and acc(t)
    // follows from W buffer t & 1: the tensor pipe no longer waits for the softmax.
    constexpr bool NOACC = MODE == MODE_FWD || MODE == MODE_FS;   // no accumulation MMAs
    constexpr bool WS = PAIR && NBUF == 1 && !NOACC;
    // FS: the softmax warps stage their bf16 weights in two 32 KB buffers (where WS keeps W)
    constexpr bool WBUFS = WS || MODE == MODE_FS;
    constexpr int LAG = WS ? 1 : NBUF - 1;              // steps between S(t) and acc(t) issue
    constexpr int BSH = (NBUF == 2) ? 1 : 0;            // log2(NBUF)
    constexpr int WBUF = WS ? 2 : NBUF;                 // W buffers (w_full barriers in use)
    constexpr int WSH = (WBUF == 2) ? 1 : 0;
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;

    // work item: (x tile, column part, part of the streamed range)
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const bool leader = (rank == 0);
    constexpr uint32_t NCTA = PAIR ? 2u : 1u;
    int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int g = unit % p.groups;
    unit /= p.groups;
    const int dp = unit % p.dparts;
    const int64_t xt = PAIR ? 2 * (int64_t)(unit / p.dparts) + rank : unit / p.dparts;
    const int64_t x0 = xt * XROWS;
    const int c_begin = dp * p.dpc;
    const int c_count = NOACC ? 0 : min(p.dpc, p.kc - c_begin);

    int64_t lo, hi;
    part_range((p.ny + SN - 1) / SN, p.groups, g, &lo, &hi);
    const int T = (int)(hi - lo);

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t x_smem = base;
    const uint32_t w_smem = base + (uint32_t)p.xres * X_CHUNK_BYTES;   // WS: two 32 KB W buffers
    const uint32_t y_smem = w_smem + (WBUFS ? 2u * 32768u : 0u);       // the ring
    // a paired CTA holds half of every Y item, so its stages are one chunk (16 KB) and a streamed
    // X item is a single chunk; otherwise a stage holds ipc chunks of Y or of X
    const int xipc = PAIR ? 1 : p.ipc;
    const uint32_t stage_bytes = (uint32_t)xipc * CHUNK_BYTES;

    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bars.x_full), 1);
        for (int s = 0; s < MAX_STAGES; ++s) {
            mbar_init(smem_u32(&bars.y_full[s]), 1);
            mbar_init(smem_u32(&bars.y_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars.s_full[b]), 1);
            mbar_init(smem_u32(&bars.w_full[b]), NCTA * NSOFT);   // one arrival per softmax warp
        }
        mbar_init(smem_u32(&bars.acc_full), 1);
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&bars.pair[i]), 2);   // one per warp
        mbar_init(smem_u32(&bars.s_free), NCTA * NSOFT);
        for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&bars.w_empty[b]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        if (PAIR) {   // the same warp of both CTAs, same destination offset
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
    // shared::cluster address, in the leader, of the barrier at the same offset as `local`
    auto in_leader = [&](uint32_t local) -> uint32_t { return PAIR ? mapa_u32(local, 0) : local; };

    if (warp < NPROD) {
        // ------------------------------ TMA producers -----------------------------------------
        // Chunk number n of the stream goes to ring stage n % nstage; a stage always belongs to
        // the same producer warp (stage % NPROD), which therefore sees its phases in order.
        {   // all 32 lanes run the loop; one elected lane issues
            // one load, counted on the leader's barrier when the CTAs are paired
            auto tma = [&](uint32_t dst, const CUtensorMap* map, int col, int64_t r, uint32_t bar) {
                if (PAIR) tma_load_2d_pair(dst, map, col, (int)r, bar);
                else      tma_load_2d(dst, map, col, (int)r, bar);
            };
            const uint32_t x_full_bar = in_leader(smem_u32(&bars.x_full));
            if (warp == 0 && leader && elect_one())
                mbar_expect_tx(smem_u32(&bars.x_full), NCTA * (uint32_t)p.xres * X_CHUNK_BYTES);
            for (int c = warp; c < p.xres; c += NPROD)
                if (elect_one()) tma(x_smem + c * X_CHUNK_BYTES, &mapX, c * 64, x0, x_full_bar);
            int next = 0;
            uint32_t next_phase = 0;
            bool ok = true;
            // Claims the next ring stage if it belongs to this warp: waits until the MMAs that
            // read its previous contents have completed.  Returns the stage or -1.
            auto acquire = [&]() -> int {
                const int stage = next;
                const uint32_t phase = next_phase;
                if (++next == p.nstage) { next = 0; next_phase ^= 1u; }
                if (!ok || (stage & (NPROD - 1)) != warp) return -1;
                const bool got = mbar_wait(smem_u32(&bars.y_empty[stage]), phase ^ 1u, abort_flag);
                if (!got) {
                    ok = false;
                    return -1;
                }
                return stage;
            };
            // Ring items.  kind 0: Y for the S MMAs (ipc chunks; a paired CTA loads the 64 rows of
            // its rank); kind 1: streamed X chunks (ipc chunks of this CTA's 128 rows); kind 2: Y
            // for the accumulation MMAs (ipc chunks; a paired CTA loads the one chunk of its rank).
            auto load_item = [&](int kind, int chunk0, int64_t row) {
                const int stage = acquire();
                if (stage < 0) return;
                const uint32_t full = smem_u32(&bars.y_full[stage]);
                const uint32_t full_bar = in_leader(full);
                const uint32_t dst = y_smem + stage * stage_bytes;
                if (elect_one()) {
                    if (kind == 1) {
                        if (leader) mbar_expect_tx(full, NCTA * stage_bytes);
                        for (int i = 0; i < xipc; ++i)
                            tma(dst + i * CHUNK_BYTES, &mapX, (chunk0 + i) * 64, x0, full_bar);
                    } else if (!PAIR) {
                        mbar_expect_tx(full, stage_bytes);
                        for (int i = 0; i < p.ipc; ++i)
                            tma(dst + i * CHUNK_BYTES, &mapY, (chunk0 + i) * 64, row, full_bar);
                    } else if (kind == 0) {
                        if (leader) mbar_expect_tx(full, (uint32_t)p.ipc * CHUNK_BYTES);  // 2 halves
                        for (int i = 0; i < p.ipc; ++i)
                            tma(dst + i * (CHUNK_BYTES / 2), &mapYh, (chunk0 + i) * 64,
                                row + 64 * rank, full_bar);
                    } else {
                        if (leader) mbar_expect_tx(full, 2 * CHUNK_BYTES);      // one chunk per CTA
                        tma(dst, &mapY, (chunk0 + (int)rank) * 64, row, full_bar);
                    }
                }
            };
            for (int t = 0; t < T + LAG && ok; ++t) {
                if (t < T) {
                    for (int c = 0; c < p.kc; c += p.ipc) {
                        load_item(0, c, (lo + t) * SN);
                        for (int j = 0; j < p.ipc; j += xipc)
                            if (c + j >= p.xres) load_item(1, c + j, x0);
                    }
                }
                if (!NOACC && t >= LAG) {
                    for (int c = 0; c < c_count; c += p.ipc)
                        load_item(2, c_begin + c, (lo + t - LAG) * SN);
                }
            }
        }
    } else if (warp == MMA_WARP) {
        // ------------------------------ MMA issuer ----------------------------------------------
        if (leader) {   // all 32 lanes run the loop; one elected lane issues the MMAs and commits
            constexpr int MROWS = PAIR ? 2 * XROWS : XROWS;
            const uint32_t idesc_s = instr_desc(SN, false, MROWS);
            const uint32_t idesc_acc64 = instr_desc(64, true, MROWS);
            const uint32_t idesc_acc128 = instr_desc(128, true, MROWS);
            // arrives on the given barrier (of both CTAs when paired) when the MMAs so far are done
            auto commit = [&](uint32_t bar) {
                if (PAIR) tc_commit_pair(bar);
                else      tc_commit(bar);
            };
            // S-phase Y chunks of one stage are 16 KB apart, or 8 KB when each CTA holds 64 rows
            constexpr uint32_t YCH_LO = (PAIR ? CHUNK_BYTES / 2 : CHUNK_BYTES) >> 4;
            const uint32_t x_lo = desc_lo(x_smem, 0);
            const uint32_t ring_lo = desc_lo(y_smem, CHUNK_BYTES);   // LBO: next chunk of a stage
            constexpr uint32_t CH_LO = CHUNK_BYTES >> 4;
            const uint32_t stage_lo = stage_bytes >> 4;
            const uint32_t idesc_acc = (p.ipc == 2) ? idesc_acc128 : idesc_acc64;   // paired: ipc == 2
            int next = 0;
            uint32_t next_phase = 0;
            bool ok = mbar_wait(smem_u32(&bars.x_full), 0, abort_flag);
            tc_fence_after();
            // Waits for the next ring stage to be filled; returns its index or -1.
            auto next_stage = [&]() -> int {
                const int stage = next;
                const uint32_t phase = next_phase;
                if (++next == p.nstage) { next = 0; next_phase ^= 1u; }
                const bool got = mbar_wait(smem_u32(&bars.y_full[stage]), phase, abort_flag);
                if (!got) {
                    ok = false;
                    return -1;
                }
                return stage;   // filled by TMA (async proxy), read by the MMA: the mbarrier orders it
            };
            for (int t = 0; t < T + LAG && ok; ++t) {
                if (t < T) {
                    const int b = t & (NBUF - 1);
                    if (WS && t >= 1) {     // the softmax warps have read S(t-1) out of the tile
                        ok = mbar_wait(smem_u32(&bars.s_free), (t - 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    if (NOACC && t >= NBUF) {
                        ok = mbar_wait(smem_u32(&bars.w_full[b]), ((t - NBUF) >> BSH) & 1,
                                       abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    const uint32_t d_tmem = tmem + S_COL0 + b * SN;
                    for (int c = 0; c < p.kc && ok; c += p.ipc) {
                        const int ys = next_stage();
                        if (!ok) break;
                        const uint32_t yb = ring_lo + ys * stage_lo;
                        if (!PAIR) {
                            // one ring item of Y and (for streamed chunks) one of X: ipc chunks,
                            // issued from a single elected region (scalar work per item is what
                            // limits the issuing warp)
                            int xs = -1;
                            uint32_t xa = x_lo + c * CH_LO;
                            if (c >= p.xres) {
                                xs = next_stage();
                                if (!ok) break;
                                xa = ring_lo + xs * stage_lo;
                            }
                            if (elect_one()) {
                                if (c == 0) mma_ss<false, false>(d_tmem, xa, yb, idesc_s);
                                else        mma_ss<true, false>(d_tmem, xa, yb, idesc_s);
                                mma_ss<true, false>(d_tmem, xa + 2, yb + 2, idesc_s);
                                mma_ss<true, false>(d_tmem, xa + 4, yb + 4, idesc_s);
                                mma_ss<true, false>(d_tmem, xa + 6, yb + 6, idesc_s);
                                if (p.ipc == 2) {
                                    mma_ss<true, false>(d_tmem, xa + CH_LO, yb + CH_LO, idesc_s);
                                    mma_ss<true, false>(d_tmem, xa + CH_LO + 2, yb + CH_LO + 2, idesc_s);
                                    mma_ss<true, false>(d_tmem, xa + CH_LO + 4, yb + CH_LO + 4, idesc_s);
                                    mma_ss<true, false>(d_tmem, xa + CH_LO + 6, yb + CH_LO + 6, idesc_s);
                                }
                                if (xs >= 0) tc_commit(smem_u32(&bars.y_empty[xs]));
                                tc_commit(smem_u32(&bars.y_empty[ys]));
                            }
                        } else {
                            // paired: the Y item holds this CTA's 64 rows of two chunks (8 KB
                            // each), every streamed X chunk is an item of its own
                            for (int j = 0; j < 2 && ok; ++j) {
                                int xs = -1;
                                uint32_t xa = x_lo + (c + j) * CH_LO;
                                if (c + j >= p.xres) {
                                    xs = next_stage();
                                    if (!ok) break;
                                    xa = ring_lo + xs * stage_lo;
                                }
                                const uint32_t yj = yb + j * YCH_LO;
                                if (elect_one()) {
                                    if (c + j == 0) mma_ss<false, true>(d_tmem, xa, yj, idesc_s);
                                    else            mma_ss<true, true>(d_tmem, xa, yj, idesc_s);
                                    mma_ss<true, true>(d_tmem, xa + 2, yj + 2, idesc_s);
                                    mma_ss<true, true>(d_tmem, xa + 4, yj + 4, idesc_s);
                                    mma_ss<true, true>(d_tmem, xa + 6, yj + 6, idesc_s);
                                    if (xs >= 0) tc_commit_pair(smem_u32(&bars.y_empty[xs]));
                                    if (j == 1) tc_commit_pair(smem_u32(&bars.y_empty[ys]));
                                }
                            }
                        }
                    }
                    if (!ok) break;
                    if (elect_one()) commit(smem_u32(&bars.s_full[b]));
                }
                if (!NOACC && t >= LAG) {
                    const int u = t - LAG, b = u & (WBUF - 1);
                    ok = mbar_wait(smem_u32(&bars.w_full[b]), (u >> WSH) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t w_tmem = tmem + S_COL0 + (WS ? 0 : b * SN);
                    const uint32_t w_lo = desc_lo(w_smem + b * 32768u, 0);   // WS: K-major A operand
                    // one ring item per iteration: ipc chunks = 64 * ipc accumulator columns
                    for (int c = 0; c < c_count && ok; c += p.ipc) {
                        const int ys = next_stage();
                        if (!ok) break;
                        const uint32_t yb = ring_lo + ys * stage_lo;
                        const uint32_t d_tmem = tmem + c * 64;
                        if (elect_one()) {
                            // k-steps of the first column half read W at columns 8 k, those of
                            // the second half at SN/2 + 8 (k - KH)
                            constexpr int KH = SN / 32;
                            if (WS) {
                                // W[128 x 128] sits in shared memory as two K-major chunks of 64
                                if (u == 0) mma_ss<false, PAIR>(d_tmem, w_lo, yb, idesc_acc);
                                else        mma_ss<true, PAIR>(d_tmem, w_lo, yb, idesc_acc);
#pragma unroll
                                for (int k = 1; k < SN / 16; ++k)
                                    mma_ss<true, PAIR>(d_tmem, w_lo + (k / 4) * CH_LO + (k % 4) * 2,
                                                       yb + k * 128, idesc_acc);
                            } else {
                                if (u == 0) mma_ts<false, PAIR>(d_tmem, w_tmem, yb, idesc_acc);
                                else        mma_ts<true, PAIR>(d_tmem, w_tmem, yb, idesc_acc);
#pragma unroll
                                for (int k = 1; k < SN / 16; ++k)
                                    mma_ts<true, PAIR>(d_tmem,
                                                       w_tmem + (k / KH) * (SN / 2) + (k % KH) * 8,
                                                       yb + k * 128, idesc_acc);
                            }
                            commit(smem_u32(&bars.y_empty[ys]));
                        }
                    }
                    if (WS && ok && elect_one()) commit(smem_u32(&bars.w_empty[b]));
                }
            }
            if (ok && !NOACC && elect_one()) commit(smem_u32(&bars.acc_full));
        }
    } else {
        // ------------------------------ softmax / epilogue warps --------------------------------
        constexpr bool GROUPS2 = two_softmax_groups<MODE, NBUF, PAIR>();
        const int sw = warp - (NPROD + 1);             // 0..7, or 0..15 with two groups
        const int grp = GROUPS2 ? (sw >> 3) : 0;       // softmax group: tiles grp, grp + 2, ...
        const int q = warp & 3;                        // tensor-memory lane quarter of this warp
        const int half = (sw & 7) >> 2;                // which half of the tile's columns
        constexpr int CB_PER = SN / 64;                // 32-column blocks per half
        const int cb0 = half * CB_PER;
        const int row = q * 32 + lane;
        const int64_t x = x0 + row;
        const int64_t xm = x + p.mask_delta;     // the streamed index masked for this row
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const bool self_mask = (p.mask_mode == GC_MASK_SELF);
        bool ok = true;
        // w_full and s_free live in the CTA that issues the MMAs
        auto arrive_w = [&](uint32_t local) {
            if (PAIR && !leader) mbar_arrive_cluster(mapa_u32(local, 0));
            else                 mbar_arrive(local);
        };
        // WS: 32 packed bf16 weights (columns 32 j .. of this warp's column half) of this thread's
        // row go to W buffer wb as four 16-byte pieces of the row's 128-byte line in K chunk
        // `half`, at the swizzled piece index the K-major MMA descriptor expects.
        auto put_w_block = [&](int wb, int j, const uint32_t (&pk)[16]) {
            const uint32_t line = w_smem + wb * 32768u + half * CHUNK_BYTES + row * 128;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t addr = line + (((4 * j + i) ^ (row & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                             ::"r"(addr), "r"(pk[4 * i]), "r"(pk[4 * i + 1]), "r"(pk[4 * i + 2]),
                               "r"(pk[4 * i + 3]) : "memory");
            }
        };

        if (MODE == MODE_FWD) {
            float m = -INFINITY, l = 0.f;
            const int32_t pos_x = (x < p.nx) ? p.pos_idx[x] : -1;
            for (int t = 0; t < T; ++t) {
                const int b = t & (NBUF - 1);
                ok = mbar_wait(smem_u32(&bars.s_full[b]), (t >> BSH) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const int64_t y0 = (lo + t) * SN;
#pragma unroll 1
                for (int cb = cb0; cb < cb0 + CB_PER; ++cb) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + S_COL0 + b * SN + cb * 32, v);
                    tmem_ld_wait();
                    const int64_t yb = y0 + cb * 32;
                    if (yb >= p.ny) continue;
                    if (pos_x >= yb && pos_x < yb + 32 && !(self_mask && xm == pos_x)) {
                        const int rel = (int)(pos_x - yb);
                        float s = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) s = __uint_as_float(v[c]);
                        p.pos_logit[x] = s * p.inv_tau;
                    }
                    float s2[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) s2[c] = __uint_as_float(v[c]) * p.c1;
                    if (yb + 32 > p.ny) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (yb + c >= p.ny) s2[c] = -INFINITY;
                    }
                    if (self_mask && xm >= yb && xm < yb + 32) {
                        const int rel = (int)(xm - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) s2[c] = -INFINITY;
                    }
                    float bm = s2[0];
#pragma unroll
                    for (int c = 1; c < 32; ++c) bm = fmaxf(bm, s2[c]);
                    if (bm > -INFINITY) {
                        const float mn = fmaxf(m, bm);
                        float sum = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c) sum += ex2(s2[c] - mn);
                        l = l * ex2(m - mn) + sum;
                        m = mn;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_w(smem_u32(&bars.w_full[b]));
            }
            // one (max, sum) pair per row, part of the streamed range and column half
            if (ok && x < p.nx) {
                const int64_t slot = (int64_t)(2 * g + half) * p.nq + x;
                p.part_m[slot] = m * 0.69314718055994531f;   // back to natural log
                p.part_l[slot] = l;
            }
        } else if (MODE == MODE_FS) {
            // ---------------- forward sweep that also stores the weights ----------------
            // Every weight of query x is 2^(s2 - ref2[x]) with an anchor chosen before the sweep,
            // so all parts of the streamed range, and every later kernel, share one scale per
            // row.  l is this half's sum over its allowed columns, positive included; the stored
            // bf16 weight of the positive column is 0 (its term is added in fp32 later).
            const float ref2 = (x < p.nx) ? p.row_ref[x] : 0.f;
            const int32_t pos_x = (x < p.nx) ? p.pos_idx[x] : -1;
            float l = 0.f, wmax = 0.f;
            // this warp's 32 rows x 64 columns of a staging buffer: 4 KB, stored on their own
            const uint32_t my_stage = w_smem + half * CHUNK_BYTES + q * 4096;
            const bool rows_live = x0 + q * 32 < p.nx;
            for (int t = 0; t < T; ++t) {
                const int b = t & (NBUF - 1);
                const int64_t y0 = (lo + t) * SN;
                ok = mbar_wait(smem_u32(&bars.s_full[b]), (t >> BSH) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sbuf = tmem + lane_addr + S_COL0 + b * SN;
                uint32_t vv[CB_PER][32];
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) tmem_ld32(sbuf + (cb0 + j) * 32, vv[j]);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_w(smem_u32(&bars.w_full[b]));   // S buffer b may be reused
                // the store issued two steps ago has finished reading staging buffer t & 1
                if (t >= 2) {
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                }
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) {
                    const int64_t yb = y0 + (cb0 + j) * 32;
                    const bool has_pos = pos_x >= yb && pos_x < yb + 32 && pos_x < p.ny &&
                                         !(self_mask && xm == pos_x);
                    if (has_pos) {
                        const int rel = (int)(pos_x - yb);
                        float sp = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) sp = __uint_as_float(vv[j][c]);
                        p.pos_logit[x] = sp * p.inv_tau;
                    }
                    if (yb + 32 > p.ny) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (yb + c >= p.ny) vv[j][c] = __float_as_uint(-INFINITY);
                    }
                    if (self_mask && xm >= yb && xm < yb + 32) {
                        const int rel = (int)(xm - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) vv[j][c] = __float_as_uint(-INFINITY);
                    }
                    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
                    float m0 = 0.f, m1 = 0.f;
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        float w0 = ex2(fmaf(__uint_as_float(vv[j][c]), p.c1, -ref2));
                        float w1 = ex2(fmaf(__uint_as_float(vv[j][c + 1]), p.c1, -ref2));
                        float w2 = ex2(fmaf(__uint_as_float(vv[j][c + 2]), p.c1, -ref2));
                        float w3 = ex2(fmaf(__uint_as_float(vv[j][c + 3]), p.c1, -ref2));
                        s0 += w0; s1 += w1; s2 += w2; s3 += w3;
                        m0 = fmaxf(m0, fmaxf(w0, w1));
                        m1 = fmaxf(m1, fmaxf(w2, w3));
                        vv[j][c] = __float_as_uint(w0);
                        vv[j][c + 1] = __float_as_uint(w1);
                        vv[j][c + 2] = __float_as_uint(w2);
                        vv[j][c + 3] = __float_as_uint(w3);
                    }
                    l += (s0 + s1) + (s2 + s3);
                    wmax = fmaxf(wmax, fmaxf(m0, m1));
                    if (pos_x >= yb && pos_x < yb + 32) {                  // positive: fp32 later
                        const int rel = (int)(pos_x - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) vv[j][c] = 0u;
                    }
                    uint32_t packed[16];
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(vv[j][2 * r]),
                                                                 __uint_as_float(vv[j][2 * r + 1]));
                        packed[r] = *reinterpret_cast<uint32_t*>(&h);
                    }
                    put_w_block(t & 1, j, packed);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                // rows past nx and columns past ny are clipped by the tensor map
                if (lane == 0 && rows_live && y0 + half * 64 < p.ny)
                    tma_store_2d(&mapO, my_stage + (t & 1) * 32768u, (int)(y0 + half * 64),
                                 (int)x0 + q * 32);
            }
            if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            __syncwarp();
            if (ok && x < p.nx) {
                const int64_t slot = (int64_t)(2 * g + half) * p.nq + x;
                p.part_m[slot] = ref2 * 0.69314718055994531f;   // natural log units
                p.part_l[slot] = l;
                // weights beyond 2^100 (or not finite) cannot be accumulated safely
                if (!(wmax <= 1.2676506e30f)) *p.range_flag = 1;
            }
        } else if (MODE == MODE_FQ) {
            // ---------------- forward fused into the dQ sweep ----------------
            // m_ref is the power-of-two scale all weights of a row share (both column halves);
            // l is this half's sum of 2^(s2 - m_ref) over its allowed columns, positive included.
            float m_ref = 0.f, l = 0.f;
            const int32_t pos_x = (x < p.nx) ? p.pos_idx[x] : -1;
            for (int t = 0; t < T; ++t) {
                const int64_t y0 = (lo + t) * SN;
                ok = mbar_wait(smem_u32(&bars.s_full[0]), t & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sbuf = tmem + lane_addr + S_COL0;
                // ---- read the tile once: raw dot products of this half, dead columns at -inf ----
                uint32_t vv[CB_PER][32];
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) tmem_ld32(sbuf + (cb0 + j) * 32, vv[j]);
                tmem_ld_wait();
                if (WS) {   // the S tile may be overwritten now
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) arrive_w(smem_u32(&bars.s_free));
                }
                float bm = -INFINITY;
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) {
                    const int64_t yb = y0 + (cb0 + j) * 32;
                    const bool has_pos = pos_x >= yb && pos_x < yb + 32 && pos_x < p.ny &&
                                         !(self_mask && xm == pos_x);
                    if (has_pos) {
                        const int rel = (int)(pos_x - yb);
                        float sp = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) sp = __uint_as_float(vv[j][c]);
                        p.pos_logit[x] = sp * p.inv_tau;
                    }
                    if (yb + 32 > p.ny) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (yb + c >= p.ny) vv[j][c] = __float_as_uint(-INFINITY);
                    }
                    if (self_mask && xm >= yb && xm < yb + 32) {
                        const int rel = (int)(xm - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) vv[j][c] = __float_as_uint(-INFINITY);
                    }
#pragma unroll
                    for (int c = 0; c < 32; ++c) bm = fmaxf(bm, __uint_as_float(vv[j][c]));
                }
                bm *= p.c1;                                            // log2 domain (c1 > 0)
                // agree on the tile maximum with the warp that owns the other column half (the
                // partner reads this before it arrives on w_full for this step, and the next
                // write only happens after the S tile of the next step, which needs that arrival)
                row_max_xch[half][row] = bm;
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.pair[q]));
                ok = mbar_wait(smem_u32(&bars.pair[q]), t & 1, abort_flag);
                if (!ok) break;
                const float tile_max = fmaxf(bm, row_max_xch[half ^ 1][row]);
                if (t == 0) {
                    m_ref = (tile_max > -INFINITY) ? tile_max : 0.f;
                } else if (__any_sync(0xffffffffu, tile_max > m_ref + 8.f)) {
                    // rare: some row's maximum outgrew its reference by more than 2^8.  The
                    // tensor-memory accesses are warp-wide, so every lane moves its reference
                    // to max(m_ref, tile_max) (factor 1 where nothing changes).  Both warps of
                    // the quarter see the same rows and values, hence take the same branch, and
                    // rescale alternate 32-column blocks of the accumulator.
                    const float m_new = fmaxf(m_ref, tile_max);
                    const float f = ex2(m_ref - m_new);
                    l *= f;
                    if (WS) {   // acc(t-1) may still be running: wait for its completion
                        ok = mbar_wait(smem_u32(&bars.w_empty[(t - 1) & 1]), ((t - 1) >> 1) & 1,
                                       abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    for (int cb = half; cb < c_count * 2; cb += 2) {
                        uint32_t a[32];
                        tmem_ld32(tmem + lane_addr + cb * 32, a);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            a[c] = __float_as_uint(__uint_as_float(a[c]) * f);
                        tmem_st16(tmem + lane_addr + cb * 32,
                                  *reinterpret_cast<const uint32_t(*)[16]>(&a[0]));
                        tmem_st16(tmem + lane_addr + cb * 32 + 16,
                                  *reinterpret_cast<const uint32_t(*)[16]>(&a[16]));
                    }
                    m_ref = m_new;
                }
                // ---- weights 2^(s2 - m_ref) (0 for dead columns), their sum, bf16 W without the
                // positive ----
                if (WS && t >= 2) {   // W buffer t & 1 has been consumed by acc(t-2)
                    ok = mbar_wait(smem_u32(&bars.w_empty[t & 1]), ((t - 2) >> 1) & 1, abort_flag);
                    if (!ok) break;
                }
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) {
                    const int64_t yb = y0 + (cb0 + j) * 32;
                    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        float w0 = ex2(fmaf(__uint_as_float(vv[j][c]), p.c1, -m_ref));
                        float w1 = ex2(fmaf(__uint_as_float(vv[j][c + 1]), p.c1, -m_ref));
                        float w2 = ex2(fmaf(__uint_as_float(vv[j][c + 2]), p.c1, -m_ref));
                        float w3 = ex2(fmaf(__uint_as_float(vv[j][c + 3]), p.c1, -m_ref));
                        s0 += w0; s1 += w1; s2 += w2; s3 += w3;
                        vv[j][c] = __float_as_uint(w0);
                        vv[j][c + 1] = __float_as_uint(w1);
                        vv[j][c + 2] = __float_as_uint(w2);
                        vv[j][c + 3] = __float_as_uint(w3);
                    }
                    l += (s0 + s1) + (s2 + s3);
                    if (pos_x >= yb && pos_x < yb + 32) {                  // positive: fp32 later
                        const int rel = (int)(pos_x - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) vv[j][c] = 0u;
                    }
                    uint32_t packed[16];
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(vv[j][2 * r]),
                                                                 __uint_as_float(vv[j][2 * r + 1]));
                        packed[r] = *reinterpret_cast<uint32_t*>(&h);
                    }
                    if (WS) put_w_block(t & 1, j, packed);
                    else    tmem_st16(sbuf + half * (SN / 2) + j * 16, packed);
                }
                if (WS) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                else    tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_w(smem_u32(&bars.w_full[WS ? (t & 1) : 0]));
            }
            // (scale, sum) of this half; only the first column part writes (both parts agree)
            if (ok && x < p.nx && dp == 0) {
                const int64_t slot = (int64_t)(2 * g + half) * p.nq + x;
                p.part_m[slot] = m_ref * 0.69314718055994531f;
                p.part_l[slot] = l;
            }
            // unscaled accumulator part -> partial buffer [g][nx][d]
            if (ok) ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
            if (ok) {
                tc_fence_after();
                // every MMA and every load has completed: the dynamic shared memory is free
                const uint32_t slot = base + (uint32_t)(warp - (NPROD + 1)) * 8192u;
                store_acc_blocks(tmem + lane_addr, c_count * 2, half, slot, 1.f, lane, &mapO,
                                 c_begin * 64, (int)x0 + q * 32, g);
            }
        } else {
            // per-row constants (DQ: the row is a query)
            float lse2_x = 0.f, l_sum = 0.f;
            int32_t pos_x = -1;
            // DA may have been launched ahead of the anchor kernel's completion
            if (MODE == MODE_DA) dep_wait();
            if ((MODE == MODE_DQ || MODE == MODE_DA) && x < p.nx) {
                lse2_x = (MODE == MODE_DA) ? p.row_ref[x] : p.row_lse[x] * 1.4426950408889634f;
                pos_x = p.pos_idx[x];
            }
            for (int t = grp; t < T; t += (GROUPS2 ? 2 : 1)) {
                const int b = t & (NBUF - 1);
                const int64_t y0 = (lo + t) * SN;
                // DP: the columns are queries; lane j holds lse / pos of column 32 cb + j
                float lse2_y[CB_PER] = {};
                int32_t pos_y[CB_PER] = {};
                if (MODE == MODE_DP) {
#pragma unroll
                    for (int j = 0; j < CB_PER; ++j) {
                        const int64_t y = y0 + (cb0 + j) * 32 + lane;
                        float lse_y = INFINITY;
                        if (y < p.ny)
                            lse_y = p.nslots > 0
                                        ? combined_lse(p.slot_m, p.slot_l, p.nslots, p.ny, y)
                                        : p.row_lse[y];
                        lse2_y[j] = lse_y * 1.4426950408889634f;
                        pos_y[j] = (y < p.ny) ? p.pos_idx[y] : -1;
                    }
                }
                ok = mbar_wait(smem_u32(&bars.s_full[b]), (t >> BSH) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sbuf = tmem + lane_addr + S_COL0 + b * SN;
                // W of this half goes to the first columns of the half's own S region (already
                // read by this warp): columns half * SN/2 + 16 j for block j.
                // WS: both 32-column blocks are requested before the single wait, so that the S
                // tile can be released.  Otherwise one block at a time in a loop that is not
                // unrolled (W block j overwrites logits this thread has already read): half the
                // registers and half the instruction footprint.
                uint32_t vv[WS ? CB_PER : 1][32];
                if (WS) {
#pragma unroll
                    for (int j = 0; j < CB_PER; ++j) tmem_ld32(sbuf + (cb0 + j) * 32, vv[WS ? j : 0]);
                    tmem_ld_wait();
                }
                if (WS) {
                    // the S tile may be overwritten; W buffer t & 1 must have been consumed
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) arrive_w(smem_u32(&bars.s_free));
                    if (t >= 2) {
                        ok = mbar_wait(smem_u32(&bars.w_empty[t & 1]), ((t - 2) >> 1) & 1, abort_flag);
                        if (!ok) break;
                    }
                }
#pragma unroll(WS ? CB_PER : 1)
                for (int j = 0; j < CB_PER; ++j) {
                    const int cb = cb0 + j;
                    uint32_t (&v)[32] = vv[WS ? j : 0];
                    if (!WS) {
                        tmem_ld32(sbuf + cb * 32, v);
                        tmem_ld_wait();
                    }
                    const float lse2_yj = j == 0 ? lse2_y[0] : lse2_y[CB_PER - 1];
                    const int32_t pos_yj = j == 0 ? pos_y[0] : pos_y[CB_PER - 1];
                    const int64_t yb = y0 + cb * 32;
                    float w[32];
                    if (MODE == MODE_DQ) {
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
                    } else if (MODE == MODE_DA) {
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
                        // exponents two at a time (one issue slot per pair)
                        const uint64_t c1_2 = pack2(p.c1, p.c1), nref_2 = pack2(-lse2_x, -lse2_x);
#pragma unroll
                        for (int c = 0; c < 32; c += 2) {
                            float e0, e1;
                            unpack2(fma2(pack2(__uint_as_float(v[c]), __uint_as_float(v[c + 1])),
                                         c1_2, nref_2), e0, e1);
                            w[c] = ex2(e0);
                            w[c + 1] = ex2(e1);
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
                        // the weights are positive, so the row sum bounds the largest of them
                        uint64_t sa = pack2(0.f, 0.f), sb = pack2(0.f, 0.f);
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            sa = add2(sa, pack2(w[c], w[c + 1]));
                            sb = add2(sb, pack2(w[c + 2], w[c + 3]));
                        }
                        float s0, s1;
                        unpack2(add2(sa, sb), s0, s1);
                        l_sum += s0 + s1;
                        if (pos_x >= yb && pos_x < yb + 32) {      // positive: fp32, in the finalize
                            const int rel = (int)(pos_x - yb);
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c == rel) w[c] = 0.f;
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
                    if (self_mask && xm >= yb && xm < yb + 32) {
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
                    if (WS) put_w_block(t & 1, j, packed);
                    else    tmem_st16(sbuf + half * (SN / 2) + j * 16, packed);
                }
                if (WS) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                else    tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_w(smem_u32(&bars.w_full[WS ? (t & 1) : b]));
            }
            if (MODE == MODE_DA && ok && x < p.nx) {
                // one (scale, sum) slot per row, part of the streamed range, softmax group and
                // column half
                const int64_t slot = (int64_t)((2 * g + grp) * 2 + half) * p.nq + x;
                p.part_m[slot] = lse2_x * 0.69314718055994531f;
                p.part_l[slot] = l_sum;
                // weights beyond 2^100 (or not finite) cannot be accumulated safely
                if (!(l_sum <= 1.2676506e30f)) *p.range_flag = 1;
            }
            // epilogue: accumulator columns of this part -> global memory (32-column blocks are
            // dealt alternately to the two warps of a lane quarter); final values are scaled,
            // partial sums of a split sweep are not
            if (grp != 0) ok = false;      // the first group writes the accumulators
            if (ok) ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
            if (ok) {
                tc_fence_after();
                const bool final_out = (p.groups == 1) && MODE != MODE_DA;
                const uint32_t slot = base + (uint32_t)(warp - (NPROD + 1)) * 8192u;
                store_acc_blocks(tmem + lane_addr, c_count * 2, half, slot,
                                 final_out ? p.out_scale : 1.f, lane, &mapO, c_begin * 64,
                                 (int)x0 + q * 32, final_out ? 0 : g);
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

// The gradient sweeps use 128-wide S tiles: two buffers when the accumulator part leaves room
// (up to 256 columns), one otherwise.
int sweep_nbuf(int kc) { return chunks_per_part(kc) * 64 + 256 <= TMEM_COLS ? 2 : 1; }

struct SmemPlan { int xres; int ipc; int nstage; size_t dynamic_bytes; };

// Rows up to 512 wide keep the whole X tile resident; wider rows keep 6 chunks so that the ring
// still has 128 KB.  Ring items hold two chunks when every chunk count involved is even.
// `ws`: the paired wide-row sweeps also keep two 32 KB W buffers in shared memory.  Their step
// time follows the ring depth (measured at 4096 x 8192 x 768: 4 stages 0.388 ms, 6 stages 0.351,
// 8 stages 0.341, 10 stages with no resident chunk 0.344), so only 2 X chunks stay resident.
SmemPlan smem_plan(int kc, bool pair = false, bool ws = false) {
    SmemPlan sp;
    sp.xres = ws ? (kc < 2 ? kc : 2) : (kc <= 8 ? kc : 6);
    const int parts = parts_for(kc), dpc = chunks_per_part(kc);
    const bool even = kc % 2 == 0 && sp.xres % 2 == 0 && dpc % 2 == 0 &&
                      (kc - dpc * (parts - 1)) % 2 == 0;
    sp.ipc = even ? 2 : 1;
    size_t xbytes = (size_t)sp.xres * X_CHUNK_BYTES;
    size_t stage = pair ? (size_t)CHUNK_BYTES : (size_t)sp.ipc * CHUNK_BYTES;
    size_t wbytes = ws ? 2 * 32768 : 0;
    size_t avail = SMEM_LIMIT - SMEM_STATIC_RESERVE - 1024 - xbytes - wbytes;
    int ns = (int)(avail / stage);
    if (ns > MAX_STAGES) ns = MAX_STAGES;
    sp.nstage = ns;
    sp.dynamic_bytes = 1024 + xbytes + wbytes + (size_t)ns * stage;
    // keep one CTA per SM (each CTA allocates all 512 tensor-memory columns)
    if (sp.dynamic_bytes < 120 * 1024) sp.dynamic_bytes = 120 * 1024;
    return sp;
}

template <int MODE, int SN, int NBUF, bool PAIR>
cudaError_t launch_one(const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& myh,
                       const CUtensorMap& mo, const TcParams& p, int64_t ctas, cudaStream_t st,
                       bool overlap_prev = false) {
    constexpr bool WBUFS = (PAIR && NBUF == 1 && MODE != MODE_FWD) || MODE == MODE_FS;
    SmemPlan sp = smem_plan(p.kc, PAIR, WBUFS);
    // the attribute belongs to the (kernel, device) pair
    static bool configured_on[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    bool& configured = configured_on[dev];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(tc_kernel<MODE, SN, NBUF, PAIR>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(SMEM_LIMIT - SMEM_STATIC_RESERVE));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(tc_threads<MODE, NBUF, PAIR>());
    cfg.dynamicSmemBytes = sp.dynamic_bytes;
    cfg.stream = st;
    TcParams pp = p;
    pp.nstage = sp.nstage;
    pp.xres = sp.xres;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 2 : 1;
    if (!PAIR && !overlap_prev) {
        tc_kernel<MODE, SN, NBUF, false><<<(unsigned)ctas, tc_threads<MODE, NBUF, false>(),
                                           sp.dynamic_bytes, st>>>(
            mx, my, myh, mo, pp);
        return cudaGetLastError();
    }
    return cudaLaunchKernelEx(&cfg, tc_kernel<MODE, SN, NBUF, PAIR>, mx, my, myh, mo, pp);
}

// CTA pairs need two-chunk ring items (the accumulation MMAs split them by rank) and at least
// two x tiles.
// CTA pairs need two-chunk ring items and at least two x tiles.  The wide-row gradient sweeps
// (one S buffer) always pair: together with W in shared memory this takes the softmax off the
// tensor pipe's critical path.  The forward sweep pairs only when the streamed matrix does not
// stay in the L2 cache, where halving its traffic outweighs the cross-SM hand-offs.
bool use_pair(int mode, int kc, int64_t nx, int64_t ny) {
    if (mode == MODE_FS) return smem_plan(kc, false, true).ipc == 2 && nx > XROWS;
    if (smem_plan(kc).ipc != 2 || nx <= XROWS || sweep_nbuf(kc) != 1) return false;
    if (mode != MODE_FWD) return true;
    return ny * kc * 128 > ((int64_t)64 << 20);
}

// x tiles (rounded up to whole pairs when paired) * column parts * groups
int64_t cta_count(int mode, int kc, int64_t nx, int64_t ny, int parts, int groups) {
    int64_t tiles = (nx + XROWS - 1) / XROWS;
    if (use_pair(mode, kc, nx, ny)) tiles = (tiles + 1) / 2 * 2;
    return tiles * parts * groups;
}

template <int MODE, int SN, int NBUF>
cudaError_t launch(const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& myh,
                   const CUtensorMap& mo, const TcParams& p, cudaStream_t st,
                   bool overlap_prev = false) {
    const int64_t ctas = cta_count(MODE, p.kc, p.nx, p.ny, p.dparts, p.groups);
    if (use_pair(MODE, p.kc, p.nx, p.ny))
        return launch_one<MODE, SN, NBUF, true>(mx, my, myh, mo, p, ctas, st, overlap_prev);
    return launch_one<MODE, SN, NBUF, false>(mx, my, myh, mo, p, ctas, st, overlap_prev);
}

}  // namespace


bool tc_supported(int64_t B, int64_t N, int d, int dtype) {
    (void)B; (void)N;
    return dtype == GC_BF16 && d % 64 == 0 && d >= 64 && d <= MAX_D;
}

// Number of (max, sum) partial slots per query row written by the forward sweep: two column
// halves for each part of the passage range.
int tc_fwd_groups(int64_t B, int64_t N, int d) {
    (void)d;
    int64_t tiles = (B + XROWS - 1) / XROWS, steps = (N + 127) / 128;
    int64_t g = sm_count() / tiles;
    if (g < 1) g = 1;
    if (g > steps) g = steps;
    if (g > 16) g = 16;
    return (int)(2 * g);
}

int tc_sweep_groups(int64_t nx, int64_t ny, int d) {
    if (quad_applicable(nx, d)) return quad_groups(nx, ny);
    int kc = d / 64;
    int64_t units = ((nx + XROWS - 1) / XROWS) * parts_for(kc);
    int64_t steps = (ny + 127) / 128;
    int64_t g = sm_count() / units;
    if (g < 1) g = 1;
    if (g > steps) g = steps;
    if (g > 8) g = 8;
    return (int)g;
}

cudaError_t tc_launch_fwd(const FwdArgs& a, cudaStream_t st) {
    const Problem& pr = a.p;
    constexpr int SN = 128;
    CUtensorMap mx, my, myh;
    if (!make_map(&mx, pr.Q, pr.B, pr.d, pr.ldq, XROWS) ||
        !make_map(&my, pr.P, pr.N, pr.d, pr.ldp, SN) ||
        !make_map(&myh, pr.P, pr.N, pr.d, pr.ldp, SN / 2))
        return cudaErrorInvalidValue;
    TcParams p{};
    p.nx = pr.B; p.ny = pr.N; p.nq = pr.B;
    p.kc = pr.d / 64; p.dparts = 1; p.dpc = 0; p.groups = a.groups / 2;
    p.nstage = smem_plan(p.kc).nstage;
    p.xres = smem_plan(p.kc).xres;
    p.ipc = smem_plan(p.kc).ipc;
    p.mask_mode = pr.mask_mode;
    p.mask_delta = pr.mask_shift;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.zero_me = reinterpret_cast<int*>(a.red);
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    return launch<MODE_FWD, SN, 2>(mx, my, myh, mx, p, st);   // no accumulator output
}

// Forward sweep that also stores the weights 2^(s2_ij - row_ref[i]) as bf16 [B x N] (row pitch
// ldw elements; 0 at masked pairs and at the positive column).  Writes the same (scale, sum) slots
// and pos_logit as the plain forward sweep, with row_ref as the scale of every slot.
cudaError_t tc_launch_fwd_store(const FwdArgs& a, void* weights, int64_t ldw, const float* row_ref,
                                int* range_flag, cudaStream_t st) {
    const Problem& pr = a.p;
    constexpr int SN = 128;
    const int kc = pr.d / 64;
    CUtensorMap mx, my, myh, mw;
    if (!make_map(&mx, pr.Q, pr.B, pr.d, pr.ldq, XROWS) ||
        !make_map(&my, pr.P, pr.N, pr.d, pr.ldp, SN) ||
        !make_map(&myh, pr.P, pr.N, pr.d, pr.ldp, SN / 2) ||
        !make_map(&mw, weights, pr.B, (int)pr.N, ldw, 32))
        return cudaErrorInvalidValue;
    TcParams p{};
    p.nx = pr.B; p.ny = pr.N; p.nq = pr.B;
    p.kc = kc; p.dparts = 1; p.dpc = 0; p.groups = a.groups / 2;
    const SmemPlan sp = smem_plan(kc, false, true);
    p.nstage = sp.nstage;
    p.xres = sp.xres;
    p.ipc = sp.ipc;
    p.mask_mode = pr.mask_mode;
    p.mask_delta = pr.mask_shift;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.zero_me = reinterpret_cast<int*>(a.red);
    p.dev_status = a.dev_status;
    p.row_ref = row_ref;
    p.range_flag = range_flag;
    return launch<MODE_FS, SN, 2>(mx, my, myh, mw, p, st);
}

bool tc_fused_applicable(int d) { return sweep_nbuf(d / 64) == 1; }

// Forward fused into the dQ sweep: writes (scale, sum) slots [2 groups][B], pos_logit and the
// unscaled accumulators partial[groups][B][d].
cudaError_t tc_launch_fused_dq(const FwdArgs& a, float* partial, int groups, cudaStream_t st) {
    const Problem& pr = a.p;
    constexpr int SN = 128;
    const int kc = pr.d / 64;
    CUtensorMap mx, my, myh;
    if (!make_map(&mx, pr.Q, pr.B, pr.d, pr.ldq, XROWS) ||
        !make_map(&my, pr.P, pr.N, pr.d, pr.ldp, SN) ||
        !make_map(&myh, pr.P, pr.N, pr.d, pr.ldp, SN / 2))
        return cudaErrorInvalidValue;
    TcParams p{};
    p.nx = pr.B; p.ny = pr.N; p.nq = pr.B;
    p.kc = kc; p.dparts = parts_for(kc); p.dpc = chunks_per_part(kc); p.groups = groups;
    p.nstage = smem_plan(kc).nstage;
    p.xres = smem_plan(kc).xres;
    p.ipc = smem_plan(kc).ipc;
    p.mask_mode = pr.mask_mode;
    p.mask_delta = pr.mask_shift;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.zero_me = reinterpret_cast<int*>(a.red);
    p.partial = partial;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    CUtensorMap mo;
    if (!make_out_map(&mo, partial, pr.B, pr.d, pr.d, groups)) return cudaErrorInvalidValue;
    return launch<MODE_FQ, SN, 1>(mx, my, myh, mo, p, st);
}

bool tc_anchor_applicable(int d) { return sweep_nbuf(d / 64) == 2; }

// Forward fused into the dQ sweep of narrow rows with row_ref (log2 domain) as each row's fixed
// scale: writes (scale, sum) slots [4 groups][B] (scale = row_ref in natural-log units),
// pos_logit and the unscaled accumulators partial[groups][B][d] of sum_j 2^(s2_ij - ref_i) P_j
// over all allowed columns but the positive one; raises *range_flag when a weight exceeds 2^100.
cudaError_t tc_launch_anchored_dq(const FwdArgs& a, float* partial, int groups,
                                  const float* row_ref, int* range_flag, cudaStream_t st,
                                  bool overlap_prev) {
    const Problem& pr = a.p;
    if (narrow_applicable(pr.d, GC_BF16))
        return narrow_launch_anchored_dq(a, partial, groups, row_ref, range_flag, st, overlap_prev);
    constexpr int SN = 128;
    const int kc = pr.d / 64;
    CUtensorMap mx, my, myh, mo;
    if (!make_map(&mx, pr.Q, pr.B, pr.d, pr.ldq, XROWS) ||
        !make_map(&my, pr.P, pr.N, pr.d, pr.ldp, SN) ||
        !make_map(&myh, pr.P, pr.N, pr.d, pr.ldp, SN / 2) ||
        !make_out_map(&mo, partial, pr.B, pr.d, pr.d, groups))
        return cudaErrorInvalidValue;
    TcParams p{};
    p.nx = pr.B; p.ny = pr.N; p.nq = pr.B;
    p.kc = kc; p.dparts = parts_for(kc); p.dpc = chunks_per_part(kc); p.groups = groups;
    p.nstage = smem_plan(kc).nstage;
    p.xres = smem_plan(kc).xres;
    p.ipc = smem_plan(kc).ipc;
    p.mask_mode = pr.mask_mode;
    p.mask_delta = pr.mask_shift;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.partial = partial;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.row_ref = row_ref;
    p.range_flag = range_flag;
    p.zero_me = reinterpret_cast<int*>(a.red);
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    return launch<MODE_DA, SN, 2>(mx, my, myh, mo, p, st, overlap_prev);
}

cudaError_t tc_launch_sweep(const SweepArgs& a, cudaStream_t st) {
    if (quad_applicable(a.nx, a.d)) return quad_launch_sweep(a, st);
    // (a dP sweep that merges forward slots itself stays on the kernels below)
    if (narrow_applicable(a.d, GC_BF16) && !(a.mode == SWEEP_DP && a.slot_l))
        return narrow_launch_sweep(a, st);
    const int kc = a.d / 64;
    constexpr int SN = 128;
    CUtensorMap mx, my, myh;
    if (!make_map(&mx, a.X, a.nx, a.d, a.ldx, XROWS) ||
        !make_map(&my, a.Y, a.ny, a.d, a.ldy, SN) || !make_map(&myh, a.Y, a.ny, a.d, a.ldy, SN / 2))
        return cudaErrorInvalidValue;
    TcParams p{};
    p.nx = a.nx; p.ny = a.ny; p.nq = 0;
    p.kc = kc; p.dparts = parts_for(kc); p.dpc = chunks_per_part(kc); p.groups = a.groups;
    p.nstage = smem_plan(kc).nstage;
    p.xres = smem_plan(kc).xres;
    p.ipc = smem_plan(kc).ipc;
    p.mask_mode = a.mask_mode;
    p.mask_delta = a.mask_delta;
    p.inv_tau = a.inv_tau;
    p.c1 = 1.4426950408889634f * a.inv_tau;
    p.out_scale = a.out_scale;
    p.row_lse = a.row_lse; p.pos_idx = a.pos_idx;
    p.out = a.out; p.ldo = a.ldo; p.partial = a.partial;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    if (a.mode == SWEEP_DP && a.slot_l) { p.slot_m = a.slot_m; p.slot_l = a.slot_l; p.nslots = a.slots; }
    CUtensorMap mo;
    const bool ok_map = a.groups == 1 ? make_out_map(&mo, a.out, a.nx, a.d, a.ldo, 1)
                                      : make_out_map(&mo, a.partial, a.nx, a.d, a.d, a.groups);
    if (!ok_map) return cudaErrorInvalidValue;
    const bool two = sweep_nbuf(kc) == 2;
    if (a.mode == SWEEP_DQ)
        return two ? launch<MODE_DQ, SN, 2>(mx, my, myh, mo, p, st)
                   : launch<MODE_DQ, SN, 1>(mx, my, myh, mo, p, st);
    return two ? launch<MODE_DP, SN, 2>(mx, my, myh, mo, p, st)
               : launch<MODE_DP, SN, 1>(mx, my, myh, mo, p, st);
}

}  // namespace gc
