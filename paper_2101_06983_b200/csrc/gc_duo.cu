// Gradient sweeps for rows of two column halves (d = 512, 640, 768): one persistent kernel whose
// CTA pairs take one of two roles, so that every tensor-core instruction is 256 wide and every
// logit tile is computed once per sweep.
//
//   S pairs    compute logit tiles of 256 x rows x 256 y rows (M = 256 over the pair, N = 256,
//              both operands streamed in 64-wide K chunks like a plain GEMM), two tiles in
//              tensor memory at a time; their softmax warps turn a tile into bf16 weights W
//              (Eq. 4-7) in registers and write them to a small ring in global memory that stays
//              in the L2 cache.  No accumulator.
//   acc pairs  hold a 256 x (d / 2) fp32 accumulator in tensor memory and run acc += W(t) Y(t)
//              (Eq. 5 / Eq. 6-7) with W tiles read back from the ring and Y tiles read MN-major.
//
// A team is two S pairs (they alternate over the team's tiles) and two acc pairs (left and right
// column half; both read every W tile): eight SMs, balanced tensor work (a tile costs an S pair
// twice what it costs an acc pair, and each acc pair takes every tile).  The tile grid (x pairs
// x y tiles, x-major) is cut into one contiguous range per team.  Where a range starts in the
// middle of an x pair's row of tiles, the acc pairs write that piece to a per-team "extra" plane
// and a later pass adds it to the piece that began at the row's first tile.
//
// Hand-off: a ring slot holds one W tile as eight 16 KB chunk images (2 CTAs x 4 chunks of 128
// rows x 64 columns, rows of 128 bytes).  The S pair's softmax warps write their rows straight
// from registers (32 bytes per store) and, a little later, fence and add 1 to the slot's ready
// counter (release); the acc pairs poll it (acquire, bounded), load the chunks with bulk tensor
// loads and add 1 to the slot's consumed counter once they have landed; the S pair reuses a slot
// after both acc pairs have consumed it.  Shared memory holds nothing but the operand rings: a
// load takes about 3 K cycles to come back when every SM streams, so the bytes in flight, not the
// request rate, are what sustains the operand bandwidth.  Tiles are produced and consumed in one global order, so no wait can
// be cyclic; all CTAs of the launch must be resident at once (the host sizes the grid for that).
// Every wait is bounded.
#include "tc_common.cuh"

namespace gc {

namespace {

enum { DMODE_DQ = 1, DMODE_DP = 2, DMODE_FA = 3 };

constexpr int DUO_TILE = 256;                  // x rows of a pair = y rows of a tile
constexpr int DUO_RING = 4;                    // W slots per S pair
constexpr int S_STAGES = 6;                    // S role: stages of one X chunk + one Y chunk
constexpr uint32_t S_STAGE_BYTES = 2 * CHUNK_BYTES;
constexpr int A_STAGES = 4;                    // acc role: W chunks (16 KB)
constexpr int B_STAGES = 4;                    // acc role: 64 y rows x this CTA's columns
constexpr uint32_t B_ATOM_BYTES = 8192;        // 64 rows x 64 columns
constexpr uint32_t B_STAGE_BYTES = 3 * B_ATOM_BYTES;
constexpr uint32_t TAB_BYTES = NSOFT * 1024;   // DP: per warp, lse and pos_idx of its 128 queries
constexpr size_t DUO_SMEM_S = (size_t)S_STAGES * S_STAGE_BYTES + TAB_BYTES;
constexpr uint32_t STG_BYTES = NSOFT * 8192;   // acc role: two 4 KB staging buffers per epilogue warp
constexpr size_t DUO_SMEM_A = (size_t)A_STAGES * CHUNK_BYTES + (size_t)B_STAGES * B_STAGE_BYTES +
                              STG_BYTES;
constexpr size_t DUO_SMEM = 1024 + (DUO_SMEM_S > DUO_SMEM_A ? DUO_SMEM_S : DUO_SMEM_A);
static_assert(DUO_SMEM <= SMEM_LIMIT - SMEM_STATIC_RESERVE, "shared memory budget");
// Warps: 0..2 issue the bulk loads (S role: 0 and 1; warp 2 publishes finished W tiles), 3 issues
// the MMAs, 4..11 are the softmax / epilogue warps (twelve warps: registers are handed out to
// four warps at a time, a thirteenth would cost as much as sixteen).
constexpr int DPROD = 3;
constexpr int DMMA_WARP = DPROD;
constexpr int DTHREADS = 32 * (DPROD + 1 + NSOFT);
constexpr int DUO_FLAG_WORDS = 64;             // words before the counters (word 0: abort)

struct DuoParams {
    int64_t nx, ny;
    int64_t nq;               // number of queries B (pitch of the slot arrays)
    int64_t YT, total;        // y tiles per x pair, tiles in all
    int nteams;
    int kc;                   // d / 64
    int dpc;                  // chunks per column half
    int mask_mode;
    float c1;                 // log2(e) / tau
    float inv_tau;
    float out_scale;
    const float* row_lse;
    const int32_t* pos_idx;
    const float* row_ref;     // FA: anchor of each query's weights, log2 domain
    float* part_m;            // FA: (scale, sum) slots, written
    float* part_l;
    float* pos_logit;         // FA
    int* range_flag;          // FA
    int* flags;               // word 0: abort; then ready[S pair][slot][rank], consumed[S pair][slot]
    uint8_t* ring;            // W ring
    float* out_main;          // [nx][ld_main]: pieces that begin at the first tile of their x pair
    int64_t ld_main;
    float* extra;             // [nteams][256][d]: the other pieces, one plane per team
    int* dev_status;
    Gate gate;
    int* zero_me;
};

struct DuoBars {
    uint64_t full[S_STAGES];       // S role: ring stage filled (in the leader, both CTAs' bytes);
    uint64_t empty[S_STAGES];      //   acc role: W chunk ring
    uint64_t b_full[B_STAGES];     // acc role: Y ring
    uint64_t b_empty[B_STAGES];
    uint64_t t_full[2];            // S role: S tile b complete; acc role: [0] accumulator complete
    uint64_t t_free[2];            // this CTA's eight warps have read it
    uint64_t t_free_peer[2];       // leader: the same of the second CTA, forwarded by its idle MMA warp
    uint64_t w_stored[DUO_RING];   // S role: the eight softmax warps have written their rows of a slot
};

// ---- schedule: tile s = xp * YT + yt; team t owns the contiguous range [lo, hi) -----------------
__host__ __device__ inline void team_range(int64_t total, int nteams, int t, int64_t* lo,
                                           int64_t* hi) {
    const int64_t base = total / nteams, rem = total % nteams;
    *lo = t * base + (t < rem ? t : rem);
    *hi = *lo + base + (t < rem ? 1 : 0);
}
__host__ __device__ inline int team_of(int64_t total, int nteams, int64_t s) {
    const int64_t base = total / nteams, rem = total % nteams;
    if (s < rem * (base + 1)) return (int)(s / (base + 1));
    return (int)(rem + (s - rem * (base + 1)) / base);
}

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu(int* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_relaxed_gpu(int* p, int v) {
    asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() {
    asm volatile("fence.proxy.async;" ::: "memory");
}
// Waits (whole warp, bounded) until *addr >= target.  False when aborting or out of time.
__device__ __forceinline__ bool poll_ge(const int* addr, int target, volatile int* abort_flag,
                                        int* gabort, int lane) {
    const uint64_t t0 = global_ns();
    uint32_t spins = 0;
    while (true) {
        int v = 0;
        if (lane == 0) v = ld_acquire_gpu(addr);
        v = __shfl_sync(0xffffffffu, v, 0);
        if (v >= target) return true;
        if ((++spins & 15u) == 0u) {
            int stop = 0;
            if (lane == 0) {
                stop = *abort_flag | *reinterpret_cast<volatile int*>(gabort);
                if (!stop && global_ns() - t0 > WAIT_LIMIT_NS) stop = 1;
                if (stop) {
                    *abort_flag = 1;
                    *reinterpret_cast<volatile int*>(gabort) = 1;
                }
            }
            if (__shfl_sync(0xffffffffu, stop, 0)) return false;
        }
        __nanosleep(40);
    }
}
// D[tmem] (+)= A[smem] * B[smem] over the CTA pair, accumulate flag at run time
__device__ __forceinline__ void mma_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo,
                                         uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %4};\n\t"
        "mov.b64 db, {%2, %4};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(DESC_HI), "r"(acc)
        : "memory");
}

template <int MODE>
__global__ void __launch_bounds__(DTHREADS, 1)
duo_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapYs,
           const __grid_constant__ CUtensorMap mapYa, const __grid_constant__ CUtensorMap mapWld,
           const __grid_constant__ CUtensorMap mapMain, const __grid_constant__ CUtensorMap mapExtra,
           const DuoParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) DuoBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;
    if (gate_closed(p.gate)) return;            // same answer in every CTA
    if (MODE == DMODE_FA && blockIdx.x == 0 && threadIdx.x == 0 && p.zero_me) *p.zero_me = 0;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);   // warp-uniform
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();        // 0, 1
    const bool leader = (rank == 0);
    const int cid = (int)(blockIdx.x >> 1);
    const int team = cid >> 2;
    const int role = cid & 3;
    const bool s_role = role < 2;
    const int sidx = role & 1;                      // S role: which of the team's two S pairs
    const int hidx = role & 1;                      // acc role: which column half
    int* const gabort = p.flags;

    int64_t s_lo, s_hi;
    team_range(p.total, p.nteams, team, &s_lo, &s_hi);
    const int nk = (int)(s_hi - s_lo);              // tiles of the team
    const int nS = 2 * p.nteams;                    // S pairs of the launch
    int* const ready = p.flags + DUO_FLAG_WORDS;                    // [nS][DUO_RING][2]
    int* const consumed = ready + nS * DUO_RING * 2;                // [nS][DUO_RING]
    // first ring row (of 64 bf16) of chunk `chunk` of CTA `r` in slot `slot` of S pair `sp`
    auto ring_row = [&](int sp, int slot, int r, int chunk) -> int {
        return ((((sp * DUO_RING + slot) * 2 + r) * 4) + chunk) * 128;
    };

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < S_STAGES; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        for (int s = 0; s < B_STAGES; ++s) {
            mbar_init(smem_u32(&bars.b_full[s]), 1);
            mbar_init(smem_u32(&bars.b_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars.t_full[b]), 1);
            mbar_init(smem_u32(&bars.t_free[b]), NSOFT);
            mbar_init(smem_u32(&bars.t_free_peer[b]), 1);
        }
        for (int b = 0; b < DUO_RING; ++b) mbar_init(smem_u32(&bars.w_stored[b]), NSOFT);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == DMMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();               // both CTAs' barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    auto in_leader = [&](uint32_t local) -> uint32_t { return mapa_u32(local, 0); };

    if (s_role) {
        // =========================================================================================
        // S role
        // =========================================================================================
        const uint32_t ring_smem = base;
        const uint32_t tab_smem = base + S_STAGES * S_STAGE_BYTES;
        const int sp = 2 * team + sidx;
        if (warp == 2) {
            // ------------------------------ publisher ------------------------------------------
            // The softmax warps' stores of a tile become visible to the acc pairs here: one fence
            // after all eight warps have arrived covers their stores (release is cumulative), and
            // it stalls this warp instead of theirs.
            const int nj = (nk - sidx + 1) / 2;
            for (int j = 0; j < nj; ++j) {
                const int slot = j % DUO_RING;
                if (!mbar_wait(smem_u32(&bars.w_stored[slot]), (uint32_t)((j / DUO_RING) & 1), abort_flag))
                    break;
                __threadfence();
                if (lane == 0) red_release_gpu(ready + (sp * DUO_RING + slot) * 2 + (int)rank, NSOFT);
                __syncwarp();
            }
        } else if (warp < 2) {
            // ------------------------------ TMA producers -------------------------------------
            int stage = 0, item = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int k = sidx; k < nk && ok; k += 2) {
                const int64_t s = s_lo + k;
                const int64_t xp = s / p.YT, yt = s - xp * p.YT;
                const int xrow = (int)(xp * DUO_TILE + rank * 128);
                const int yrow = (int)(yt * DUO_TILE + rank * 128);
                for (int c = 0; c < p.kc; ++c, ++item) {
                    const int st = stage;
                    const uint32_t ph = phase;
                    if (++stage == S_STAGES) { stage = 0; phase ^= 1u; }
                    if ((item & 1) != warp) continue;
                    if (!mbar_wait(smem_u32(&bars.empty[st]), ph ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars.full[st]);
                    const uint32_t full_bar = in_leader(full);
                    const uint32_t dst = ring_smem + st * S_STAGE_BYTES;
                    if (elect_one()) {
                        if (leader) mbar_expect_tx(full, 2 * S_STAGE_BYTES);
                        tma_load_2d_pair(dst, &mapX, c * 64, xrow, full_bar);
                        tma_load_2d_pair(dst + CHUNK_BYTES, &mapYs, c * 64, yrow, full_bar);
                    }
                }
            }
        } else if (warp == DMMA_WARP) {
            if (leader) {
                // ------------------------------ MMA issuer --------------------------------------
                const uint32_t idesc_s = instr_desc(DUO_TILE, false, 2 * XROWS);
                constexpr uint32_t CH_LO = CHUNK_BYTES >> 4;
                const uint32_t ring_lo = desc_lo(ring_smem, 0);
                int stage = 0;
                uint32_t phase = 0;
                bool ok = true;
                int j = 0;
                for (int k = sidx; k < nk && ok; k += 2, ++j) {
                    const int b = j & 1;
                    if (j >= 2) {       // the softmax warps of both CTAs have read tile j - 2
                        const uint32_t par = (uint32_t)(((j >> 1) - 1) & 1);
                        ok = mbar_wait(smem_u32(&bars.t_free[b]), par, abort_flag) &&
                             mbar_wait(smem_u32(&bars.t_free_peer[b]), par, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    const uint32_t d_tmem = tmem + (uint32_t)b * DUO_TILE;
                    for (int c = 0; c < p.kc; ++c) {
                        const int st = stage;
                        const uint32_t ph = phase;
                        if (++stage == S_STAGES) { stage = 0; phase ^= 1u; }
                        if (!mbar_wait(smem_u32(&bars.full[st]), ph, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const uint32_t xa = ring_lo + st * (S_STAGE_BYTES >> 4);
                        const uint32_t ya = xa + CH_LO;
                        if (elect_one()) {
                            mma_pair(d_tmem, xa, ya, idesc_s, c > 0 ? 1u : 0u);
                            mma_pair(d_tmem, xa + 2, ya + 2, idesc_s, 1u);
                            mma_pair(d_tmem, xa + 4, ya + 4, idesc_s, 1u);
                            mma_pair(d_tmem, xa + 6, ya + 6, idesc_s, 1u);
                            tc_commit_pair(smem_u32(&bars.empty[st]));
                        }
                    }
                    if (ok && elect_one()) tc_commit_pair(smem_u32(&bars.t_full[b]));
                }
            } else {
                // Forwarder: "this CTA's warps have read S tile j" becomes one arrival on the leader
                const int nj = (nk - sidx + 1) / 2;
                for (int j = 0; j < nj; ++j) {
                    const int b = j & 1;
                    if (!mbar_wait(smem_u32(&bars.t_free[b]), (uint32_t)((j >> 1) & 1), abort_flag))
                        break;
                    if (lane == 0) mbar_arrive_cluster(in_leader(smem_u32(&bars.t_free_peer[b])));
                    __syncwarp();
                }
            }
        } else {
            // ------------------------------ softmax warps ---------------------------------------
            const int sw = warp - (DPROD + 1);             // 0..7
            const int q = warp & 3;                        // tensor-memory lane quarter
            const int half = sw >> 2;                      // columns [128 half, 128 half + 128)
            const int row = q * 32 + lane;
            const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
            const bool self_mask = (p.mask_mode == GC_MASK_SELF);
            // DP: logsumexp (log2 domain) and positive of the 128 streamed queries of this warp's
            // column half, private to the warp so that no block-wide barrier is needed
            float* const lse_tab = reinterpret_cast<float*>(smem_raw + (tab_smem - smem_u32(smem_raw))) +
                                   sw * 256;
            int32_t* const pos_tab = reinterpret_cast<int32_t*>(lse_tab + 128);
            bool ok = true;
            float lse2_x = 0.f, l = 0.f;
            int32_t pos_x = -1;
            int64_t cur_xp = -1, x = 0;
            // FA may have been launched ahead of the anchor kernel's completion: row_ref, the
            // range flag, the slot arrays and everything this role writes come after it
            if (MODE == DMODE_FA) dep_wait();
            auto flush_slots = [&]() {
                if (MODE != DMODE_FA || cur_xp < 0 || x >= p.nx) return;
                const int rel = team - team_of(p.total, p.nteams, cur_xp * p.YT);
                const int64_t slot = (int64_t)((rel * 2 + sidx) * 2 + half) * p.nq + x;
                p.part_m[slot] = lse2_x * 0.69314718055994531f;
                p.part_l[slot] = l;
                // weights are >= 0, so a row sum within 2^100 bounds every weight of the row; one
                // beyond it (or not finite) cannot be accumulated safely
                if (!(l <= 1.2676506e30f)) *p.range_flag = 1;
            };
            int j = 0;
            for (int k = sidx; k < nk; k += 2, ++j) {
                const int b = j & 1;
                const int64_t s = s_lo + k;
                const int64_t xp = s / p.YT, yt = s - xp * p.YT;
                const int64_t x0 = xp * DUO_TILE + rank * 128;      // first x row of this CTA
                const int64_t y0 = yt * DUO_TILE;
                if (xp != cur_xp) {
                    flush_slots();
                    cur_xp = xp;
                    x = x0 + row;
                    l = 0.f;
                    lse2_x = 0.f;
                    pos_x = -1;
                    if (MODE != DMODE_DP && x < p.nx) {
                        lse2_x = (MODE == DMODE_FA) ? p.row_ref[x]
                                                    : p.row_lse[x] * 1.4426950408889634f;
                        pos_x = p.pos_idx[x];
                    }
                }
                if (MODE == DMODE_DP) {
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int t = i * 32 + lane;
                        const int64_t y = y0 + half * 128 + t;
                        lse_tab[t] = (y < p.ny) ? p.row_lse[y] * 1.4426950408889634f : INFINITY;
                        pos_tab[t] = (y < p.ny) ? p.pos_idx[y] : -1;
                    }
                    __syncwarp();
                }
                ok = mbar_wait(smem_u32(&bars.t_full[b]), (uint32_t)((j >> 1) & 1), abort_flag);
                if (!ok) break;
                tc_fence_after();
                const int slot = j % DUO_RING, use = j / DUO_RING;
                if (use > 0) {      // both acc pairs have taken the tile that was in this slot
                    ok = poll_ge(consumed + sp * DUO_RING + slot, 2 * use, abort_flag, gabort, lane);
                    if (!ok) break;
                    fence_proxy_async_all();
                }
                const uint32_t sbuf = tmem + lane_addr + (uint32_t)b * DUO_TILE;
                // weights of one 32-column block: v (logits, fp32 bits) -> 32 bf16 = 64 bytes of
                // this thread's row of the chunk image, written as two 32-byte stores
                auto weights = [&](uint32_t (&v)[32], int cb, int lb, uint8_t* dst) {
                    const int64_t yb = y0 + cb * 32;
                    float w[32];
                    if (MODE == DMODE_FA) {
                        const bool has_pos = pos_x >= yb && pos_x < yb + 32 && pos_x < p.ny &&
                                             !(self_mask && x == pos_x);
                        if (has_pos) {
                            const int rel = (int)(pos_x - yb);
                            float spv = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c == rel) spv = __uint_as_float(v[c]);
                            p.pos_logit[x] = spv * p.inv_tau;
                        }
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            w[c] = ex2(fmaf(__uint_as_float(v[c]), p.c1, -lse2_x));
                        if (yb + 32 > p.ny) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (yb + c >= p.ny) w[c] = 0.f;
                        }
                        if (self_mask && x >= yb && x < yb + 32) {
                            const int rel = (int)(x - yb);
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c == rel) w[c] = 0.f;
                        }
                        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            s0 += w[c];
                            s1 += w[c + 1];
                            s2 += w[c + 2];
                            s3 += w[c + 3];
                        }
                        l += (s0 + s1) + (s2 + s3);
                        if (pos_x >= yb && pos_x < yb + 32) {      // positive: fp32, later
                            const int rel = (int)(pos_x - yb);
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (c == rel) w[c] = 0.f;
                        }
                    } else if (MODE == DMODE_DQ) {
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
                        const float4* lt = reinterpret_cast<const float4*>(lse_tab + lb);
#pragma unroll
                        for (int c = 0; c < 32; c += 4) {
                            const float4 l4 = lt[c >> 2];          // OOB query: ex2(-inf) = 0
                            w[c] = ex2(fmaf(__uint_as_float(v[c]), p.c1, -l4.x));
                            w[c + 1] = ex2(fmaf(__uint_as_float(v[c + 1]), p.c1, -l4.y));
                            w[c + 2] = ex2(fmaf(__uint_as_float(v[c + 2]), p.c1, -l4.z));
                            w[c + 3] = ex2(fmaf(__uint_as_float(v[c + 3]), p.c1, -l4.w));
                        }
                        // one-hot: column c's query has its positive at row pos - x0 of this CTA
                        const int32_t pos_yj = pos_tab[lb + lane];
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
                    if (MODE != DMODE_FA && self_mask && x >= yb && x < yb + 32) {
                        const int rel = (int)(x - yb);
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c == rel) w[c] = 0.f;
                    }
                    uint32_t pk[16];
#pragma unroll
                    for (int r = 0; r < 16; ++r) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(w[2 * r], w[2 * r + 1]);
                        pk[r] = *reinterpret_cast<uint32_t*>(&h);
                    }
#pragma unroll
                    for (int i = 0; i < 2; ++i)
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                     ::"l"(dst + 32 * i), "r"(pk[8 * i]), "r"(pk[8 * i + 1]),
                                       "r"(pk[8 * i + 2]), "r"(pk[8 * i + 3]), "r"(pk[8 * i + 4]),
                                       "r"(pk[8 * i + 5]), "r"(pk[8 * i + 6]), "r"(pk[8 * i + 7])
                                     : "memory");
                };
                // The loads of the next chunk's two blocks are issued as soon as the registers of
                // the current ones are free, so that only the first load of a tile is waited for.
                uint32_t va[32], vb[32];
                tmem_ld32(sbuf + (half * 4) * 32, va);
                tmem_ld32(sbuf + (half * 4 + 1) * 32, vb);
#pragma unroll 1
                for (int ch = 0; ch < 2; ++ch) {
                    const int chunk = half * 2 + ch;       // 64-column chunk of the tile
                    // this thread's 128-byte row of the chunk image in the ring
                    uint8_t* const dst = p.ring +
                        ((size_t)ring_row(sp, slot, (int)rank, chunk) + (size_t)row) * 128;
                    tmem_ld_wait();
                    if (ch == 1) {                         // the S tile may be overwritten
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bars.t_free[b]));
                    }
                    weights(va, chunk * 2, ch * 64, dst);
                    if (ch == 0) tmem_ld32(sbuf + (half * 4 + 2) * 32, va);
                    weights(vb, chunk * 2 + 1, ch * 64 + 32, dst + 64);
                    if (ch == 0) tmem_ld32(sbuf + (half * 4 + 3) * 32, vb);
                }
                // this warp's rows of the tile are on their way: tell the publisher
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.w_stored[slot]));
            }
            if (ok) flush_slots();
        }
    } else {
        // =========================================================================================
        // accumulation role
        // =========================================================================================
        const uint32_t a_smem = base;
        const uint32_t b_smem = base + A_STAGES * CHUNK_BYTES;
        const uint32_t stg_smem = b_smem + B_STAGES * B_STAGE_BYTES;
        const int c_begin = hidx * p.dpc;
        const int c_count = min(p.dpc, p.kc - c_begin);
        const int ngr = (p.dpc + 1) / 2;                   // 128-column groups of a half (2 or 3)
        const int64_t xp_first = s_lo / p.YT;
        const int npieces = (int)((s_hi - 1) / p.YT - xp_first) + 1;
        if (warp == 0) {
            // ------------------------------ W chunks from the ring ------------------------------
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int k = 0; k < nk && ok; ++k) {
                const int sp = 2 * team + (k & 1), j = k >> 1;
                const int slot = j % DUO_RING, use = j / DUO_RING;
                ok = poll_ge(ready + (sp * DUO_RING + slot) * 2 + (int)rank, NSOFT * (use + 1),
                             abort_flag, gabort, lane);
                if (!ok) break;
                fence_proxy_async_all();
                for (int c = 0; c < 4; ++c) {
                    const int st = stage;
                    const uint32_t ph = phase;
                    if (++stage == A_STAGES) { stage = 0; phase ^= 1u; }
                    if (!mbar_wait(smem_u32(&bars.empty[st]), ph ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars.full[st]);
                    if (lane == 0) {        // the lane whose acquire saw the slot ready
                        if (leader) mbar_expect_tx(full, 2 * CHUNK_BYTES);
                        tma_load_2d_pair(a_smem + st * CHUNK_BYTES, &mapWld, 0,
                                         ring_row(sp, slot, (int)rank, c), in_leader(full));
                    }
                    __syncwarp();
                }
            }
        } else if (warp < DPROD) {
            // ------------------------------ Y tiles, 64 rows at a time (two warps) --------------
            // Columns of this CTA: the N = 256 instruction takes columns [0, 128) of its 256 from
            // rank 0 and [128, 256) from rank 1; the N = 128 one that follows takes 64 from each.
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int k = 0; k < nk && ok; ++k) {
                const int64_t s = s_lo + k;
                const int64_t yt = s % p.YT;
                for (int c = 0; c < 4; ++c) {
                    const int st = stage;
                    const uint32_t ph = phase;
                    if (++stage == B_STAGES) { stage = 0; phase ^= 1u; }
                    if ((c & 1) != warp - 1) continue;
                    if (!mbar_wait(smem_u32(&bars.b_empty[st]), ph ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = smem_u32(&bars.b_full[st]);
                    const uint32_t full_bar = in_leader(full);
                    const uint32_t dst = b_smem + st * B_STAGE_BYTES;
                    const int yrow = (int)(yt * DUO_TILE + c * 64);
                    if (elect_one()) {
                        if (leader) mbar_expect_tx(full, 2u * (uint32_t)(ngr == 3 ? 3 : 2) * B_ATOM_BYTES);
                        tma_load_2d_pair(dst, &mapYa, (c_begin + 2 * (int)rank) * 64, yrow, full_bar);
                        tma_load_2d_pair(dst + B_ATOM_BYTES, &mapYa,
                                         (c_begin + 2 * (int)rank + 1) * 64, yrow, full_bar);
                        if (ngr == 3)
                            tma_load_2d_pair(dst + 2 * B_ATOM_BYTES, &mapYa,
                                             (c_begin + 4 + (int)rank) * 64, yrow, full_bar);
                    }
                }
            }
        } else if (warp == DMMA_WARP) {
            if (leader) {
                // ------------------------------ MMA issuer --------------------------------------
                const uint32_t idesc256 = instr_desc(256, true, 2 * XROWS);
                const uint32_t idesc128 = instr_desc(128, true, 2 * XROWS);
                int sa = 0, sb = 0;
                uint32_t pa = 0, pb = 0;
                bool ok = true;
                int piece = 0;
                for (int k = 0; k < nk && ok; ++k) {
                    const int64_t s = s_lo + k;
                    const int64_t yt = s % p.YT;
                    const bool first = (k == 0 || yt == 0);
                    if (first && k > 0) {
                        ++piece;       // the epilogue warps of both CTAs have read the accumulator
                        const uint32_t par = (uint32_t)((piece - 1) & 1);
                        ok = mbar_wait(smem_u32(&bars.t_free[0]), par, abort_flag) &&
                             mbar_wait(smem_u32(&bars.t_free_peer[0]), par, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    for (int c = 0; c < 4; ++c) {
                        ok = mbar_wait(smem_u32(&bars.full[sa]), pa, abort_flag) &&
                             mbar_wait(smem_u32(&bars.b_full[sb]), pb, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t a_lo = desc_lo(a_smem + sa * CHUNK_BYTES, 0);
                        const uint32_t b_lo = desc_lo(b_smem + sb * B_STAGE_BYTES, B_ATOM_BYTES);
                        const uint32_t b2_lo = b_lo + ((2 * B_ATOM_BYTES) >> 4);
                        if (elect_one()) {
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {
                                const uint32_t acc = (first && c == 0 && kk == 0) ? 0u : 1u;
                                mma_pair(tmem, a_lo + 2 * kk, b_lo + 128 * kk, idesc256, acc);
                                if (ngr == 3)
                                    mma_pair(tmem + 256, a_lo + 2 * kk, b2_lo + 128 * kk, idesc128, acc);
                            }
                            tc_commit_pair(smem_u32(&bars.empty[sa]));
                            tc_commit_pair(smem_u32(&bars.b_empty[sb]));
                            if (c == 3) {       // all four chunks of the tile have left the ring
                                const int sp = 2 * team + (k & 1), j = k >> 1;
                                // (the loads have completed: nothing of this thread's needs
                                // publishing, and a release here would stall the issuing thread)
                                red_relaxed_gpu(consumed + sp * DUO_RING + (j % DUO_RING), 1);
                            }
                        }
                        if (++sa == A_STAGES) { sa = 0; pa ^= 1u; }
                        if (++sb == B_STAGES) { sb = 0; pb ^= 1u; }
                    }
                    const bool last = (k == nk - 1) || ((s + 1) % p.YT == 0);
                    if (ok && last && elect_one()) tc_commit_pair(smem_u32(&bars.t_full[0]));
                }
            } else {
                // Forwarder: "this CTA's warps have read the accumulator of piece i"
                for (int i = 0; i + 1 < npieces; ++i) {
                    if (!mbar_wait(smem_u32(&bars.t_free[0]), (uint32_t)(i & 1), abort_flag)) break;
                    if (lane == 0) mbar_arrive_cluster(in_leader(smem_u32(&bars.t_free_peer[0])));
                    __syncwarp();
                }
            }
        } else {
            // ------------------------------ epilogue warps --------------------------------------
            const int sw = warp - (DPROD + 1);
            const int q = warp & 3;
            const int half = sw >> 2;                      // alternate 32-column blocks
            const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
            const uint32_t buf0 = stg_smem + (uint32_t)sw * 8192u;
            int nst = 0;                                   // bulk stores issued by this warp
            for (int i = 0; i < npieces; ++i) {
                if (!mbar_wait(smem_u32(&bars.t_full[0]), (uint32_t)(i & 1), abort_flag)) break;
                tc_fence_after();
                const int64_t xp = xp_first + i;
                // the piece that begins at the first tile of its x pair is the "main" one
                const bool main_piece = (i > 0) || (s_lo % p.YT == 0);
                const CUtensorMap* map = main_piece ? &mapMain : &mapExtra;
                const int row0 = (main_piece ? (int)(xp * DUO_TILE) : 0) + (int)rank * 128 + q * 32;
                const int plane = main_piece ? 0 : team;
                const float sc = (main_piece && MODE != DMODE_FA) ? p.out_scale : 1.f;
                for (int cb = half; cb < c_count * 2; cb += 2, ++nst) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_addr + cb * 32, v);
                    // the store issued two blocks ago has finished reading this buffer
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                    tmem_ld_wait();
                    const uint32_t buf = buf0 + (uint32_t)(nst & 1) * 4096u;
                    stage_block(buf, v, sc, lane);
                    __syncwarp();
                    if (lane == 0) tma_store_3d(map, buf, c_begin * 64 + cb * 32, row0, plane);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.t_free[0]));
            }
            if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            __syncwarp();
        }
    }

    // ------------------------------ teardown ------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        uint64_t t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (threadIdx.x == 0) {
            *reinterpret_cast<volatile int*>(gabort) = 1;
            if (p.dev_status) atomicOr(p.dev_status, GC_DEV_WAIT_LIMIT);
        }
        __syncthreads();
    }
    cluster_sync_all();   // no MMA, load or arrival of the other CTA touches this one any more
    if (warp == DMMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// Adds the extra planes to the rows whose x pair was split between teams: out[row] += scale *
// extra[t][row - first row of the pair].  blockIdx.y = team; a team whose extra plane belongs to
// the same x pair as the team before it leaves its plane to the first such team, which adds the
// planes of the whole run in team order (one thread owns an element, so the sum does not depend on
// timing).
__global__ void __launch_bounds__(256)
duo_fixup_kernel(const float4* __restrict__ extra, int64_t nx, int d4, int64_t YT, int64_t total,
                 int nteams, float scale, float* __restrict__ out, int64_t ldo, const Gate gate) {
    if (gate_closed(gate)) return;
    const int t0 = (int)blockIdx.y + 1;
    int64_t lo, hi;
    team_range(total, nteams, t0, &lo, &hi);
    if (lo % YT == 0) return;                              // this team has no extra plane
    const int64_t xp = lo / YT;
    if (t0 > 1) {
        int64_t plo, phi;
        team_range(total, nteams, t0 - 1, &plo, &phi);
        if (plo % YT != 0 && plo / YT == xp) return;       // the run began earlier
    }
    const int64_t per_plane = (int64_t)DUO_TILE * d4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < per_plane;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int r = (int)(e / d4);
        const int c = 4 * (int)(e - (int64_t)r * d4);
        const int64_t row = xp * DUO_TILE + r;
        if (row >= nx) continue;
        float4* dst = reinterpret_cast<float4*>(out + row * ldo + c);
        float4 o = *dst;
        for (int t = t0; t < nteams; ++t) {
            if (t > t0) {
                team_range(total, nteams, t, &lo, &hi);
                if (lo % YT == 0 || lo / YT != xp) break;
            }
            const float4 v = extra[(int64_t)t * per_plane + e];
            o.x = fmaf(v.x, scale, o.x); o.y = fmaf(v.y, scale, o.y);
            o.z = fmaf(v.z, scale, o.z); o.w = fmaf(v.w, scale, o.w);
        }
        *dst = o;
    }
}

// Finishes the fused forward + dQ sweep (Eq. 5): dQ_i = (2^(ref2_i - lse2_i) (main_i + the extra
// planes of the teams that began inside row i's x pair, in team order) + (p_pos - 1) P_pos) /
// (B tau), positive term in fp32 from the exact row.  A row whose pos_idx is unusable gets none.
__global__ void __launch_bounds__(256)
duo_dq_finalize_kernel(const float4* __restrict__ main_plane, const float4* __restrict__ extra,
                       const float* __restrict__ row_ref2, const float* __restrict__ row_lse,
                       const float* __restrict__ pos_ws, const int32_t* __restrict__ pos_idx,
                       const __nv_bfloat16* __restrict__ P, int64_t ldp, int64_t B, int64_t N, int d4,
                       int mask_mode, int64_t YT, int64_t total, int nteams, float scale,
                       float* __restrict__ out, int64_t ldo, const Gate gate) {
    if (gate_closed(gate)) return;
    const int64_t all = B * d4;
    const int64_t per_plane = (int64_t)DUO_TILE * d4;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < all;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = e / d4;
        const int c4 = (int)(e - i * d4);
        const int64_t xp = i / DUO_TILE;
        const int r = (int)(i - xp * DUO_TILE);
        float4 acc = main_plane[e];
        const int t0 = team_of(total, nteams, xp * YT);
        const int t1 = team_of(total, nteams, (xp + 1) * YT - 1);
        for (int t = t0 + 1; t <= t1; ++t) {
            const float4 v = extra[(int64_t)t * per_plane + (int64_t)r * d4 + c4];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        const float lse = row_lse[i];
        const float w = exp2f(row_ref2[i] - lse * 1.4426950408889634f);
        acc.x *= w; acc.y *= w; acc.z *= w; acc.w *= w;
        const int32_t rr = pos_idx[i];
        const bool usable = rr >= 0 && (int64_t)rr < N && !(mask_mode == GC_MASK_SELF && (int64_t)rr == i);
        if (usable) {
            const float pm1 = expf(pos_ws[i] - lse) - 1.f;
            const __nv_bfloat16* pr = P + (int64_t)rr * ldp + 4 * c4;
            acc.x = fmaf(pm1, __bfloat162float(pr[0]), acc.x);
            acc.y = fmaf(pm1, __bfloat162float(pr[1]), acc.y);
            acc.z = fmaf(pm1, __bfloat162float(pr[2]), acc.z);
            acc.w = fmaf(pm1, __bfloat162float(pr[3]), acc.w);
        }
        *reinterpret_cast<float4*>(out + i * ldo + 4 * c4) =
            make_float4(acc.x * scale, acc.y * scale, acc.z * scale, acc.w * scale);
    }
}

// The ring as a matrix of 128-byte rows (64 bf16): chunk images one after another.
bool make_ring_map(CUtensorMap* map, void* ring, int64_t rows, int box_rows) {
    return make_map(map, ring, rows, 64, 64, box_rows);
}

// Co-resident clusters of two CTAs of this kernel on the current device (cached per device).
template <int MODE>
int duo_resident_clusters() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return 0;
    }
    if (cached[dev] == 0) {
        if (cudaFuncSetAttribute(duo_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)DUO_SMEM) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 74);
        cfg.blockDim = dim3(DTHREADS);
        cfg.dynamicSmemBytes = DUO_SMEM;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, duo_kernel<MODE>, &cfg) != cudaSuccess) {
            cudaGetLastError();
            n = 0;
        }
        cached[dev] = n > 0 ? n : -1;
    }
    return cached[dev] > 0 ? cached[dev] : 0;
}

template <int MODE>
cudaError_t launch_duo(const CUtensorMap& mx, const CUtensorMap& mys, const CUtensorMap& mya,
                       const CUtensorMap& mwld, const CUtensorMap& mmain, const CUtensorMap& mextra,
                       const DuoParams& p, cudaStream_t st, bool overlap_prev) {
    if (duo_resident_clusters<MODE>() < 4 * p.nteams) return cudaErrorLaunchOutOfResources;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.nteams * 8));
    cfg.blockDim = dim3(DTHREADS);
    cfg.dynamicSmemBytes = DUO_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, duo_kernel<MODE>, mx, mys, mya, mwld, mmain, mextra, p);
}

int64_t tiles_of(int64_t n) { return (n + DUO_TILE - 1) / DUO_TILE; }

}  // namespace

// Rows of two column halves of an even number of chunks each (d = 512, 640, 768), more than one
// x tile, and a device that keeps at least one team resident.
bool duo_applicable(int64_t nx, int d) {
    const int kc = d / 64;
    return d % 128 == 0 && parts_for(kc) == 2 && nx > XROWS && duo_max_teams() >= 1;
}

int duo_max_teams() {
    int n = duo_resident_clusters<DMODE_DQ>();
    const int b = duo_resident_clusters<DMODE_DP>(), c = duo_resident_clusters<DMODE_FA>();
    if (b < n) n = b;
    if (c < n) n = c;
    return n / 4;
}

int duo_teams(int64_t nx, int64_t ny) {
    const int64_t total = tiles_of(nx) * tiles_of(ny);
    int64_t t = duo_max_teams();
    if (t > total) t = total;
    return (int)(t < 1 ? 1 : t);
}

// Largest number of teams that share one x pair's row of tiles (= slots of row sums per query
// / 4 in the fused sweep).
int duo_max_pieces(int64_t nx, int64_t ny) {
    const int64_t XP = tiles_of(nx), YT = tiles_of(ny), total = XP * YT;
    const int nteams = duo_teams(nx, ny);
    int most = 1;
    // the count changes only where a team range begins: look at the pairs those tiles are in
    for (int t = 0; t < nteams; ++t) {
        int64_t lo, hi;
        team_range(total, nteams, t, &lo, &hi);
        const int64_t xp = lo / YT;
        const int n = team_of(total, nteams, (xp + 1) * YT - 1) - team_of(total, nteams, xp * YT) + 1;
        if (n > most) most = n;
    }
    return most;
}

size_t duo_ring_bytes(int nteams) { return (size_t)nteams * 2 * DUO_RING * 8 * CHUNK_BYTES; }
size_t duo_flag_bytes(int nteams) {
    return sizeof(int) * (size_t)(DUO_FLAG_WORDS + 2 * nteams * DUO_RING * 3);
}
size_t duo_extra_bytes(int nteams, int d) { return (size_t)nteams * DUO_TILE * (size_t)d * sizeof(float); }

namespace {

struct DuoMaps { CUtensorMap mx, mys, mya, mwld, mmain, mextra; };

bool duo_setup(DuoParams* p, DuoMaps* m, const void* X, int64_t ldx, int64_t nx, const void* Y,
               int64_t ldy, int64_t ny, int d, const DuoScratch& ws, float* main_out, int64_t ld_main) {
    p->nx = nx; p->ny = ny;
    p->YT = tiles_of(ny);
    p->total = tiles_of(nx) * p->YT;
    p->nteams = duo_teams(nx, ny);
    p->kc = d / 64;
    p->dpc = chunks_per_part(p->kc);
    p->flags = ws.flags;
    p->ring = static_cast<uint8_t*>(ws.ring);
    p->out_main = main_out;
    p->ld_main = ld_main;
    p->extra = ws.extra;
    const int64_t ring_rows = (int64_t)p->nteams * 2 * DUO_RING * 8 * 128;
    return make_map(&m->mx, X, nx, d, ldx, XROWS) && make_map(&m->mys, Y, ny, d, ldy, 128) &&
           make_map(&m->mya, Y, ny, d, ldy, 64) && make_ring_map(&m->mwld, ws.ring, ring_rows, 128) &&
           make_out_map(&m->mmain, main_out, nx, d, ld_main, 1) &&
           make_out_map(&m->mextra, ws.extra, DUO_TILE, d, d, p->nteams);
}

}  // namespace

// dQ (Eq. 5) or dP (Eq. 6-7) sweep with a given row_lse: writes out_scale * acc to a.out, the
// pieces of split x pairs through the extra planes and a fix-up pass.  ws.flags must be zero.
cudaError_t duo_launch_sweep(const SweepArgs& a, const DuoScratch& ws, cudaStream_t st) {
    DuoParams p{};
    DuoMaps m;
    if (!duo_setup(&p, &m, a.X, a.ldx, a.nx, a.Y, a.ldy, a.ny, a.d, ws, a.out, a.ldo))
        return cudaErrorInvalidValue;
    p.mask_mode = a.mask_mode;
    p.inv_tau = a.inv_tau;
    p.c1 = 1.4426950408889634f * a.inv_tau;
    p.out_scale = a.out_scale;
    p.row_lse = a.row_lse; p.pos_idx = a.pos_idx;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    cudaError_t e = a.mode == SWEEP_DQ
        ? launch_duo<DMODE_DQ>(m.mx, m.mys, m.mya, m.mwld, m.mmain, m.mextra, p, st, false)
        : launch_duo<DMODE_DP>(m.mx, m.mys, m.mya, m.mwld, m.mmain, m.mextra, p, st, false);
    if (e != cudaSuccess || p.nteams < 2) return e;
    const int d4 = a.d / 4;
    const int64_t blocks = ((int64_t)DUO_TILE * d4 + 255) / 256;
    duo_fixup_kernel<<<dim3((unsigned)blocks, (unsigned)(p.nteams - 1)), 256, 0, st>>>(reinterpret_cast<const float4*>(ws.extra), a.nx,
                                                      d4, p.YT, p.total, p.nteams, a.out_scale, a.out,
                                                      a.ldo, a.gate);
    return cudaGetLastError();
}

// Forward fused into the dQ sweep with the positive logit as each row's fixed scale (row_ref,
// log2 domain): writes (scale, sum) slots [4 * duo_max_pieces][B] (scale = row_ref in natural-log
// units; slots of teams that took no tile of a row keep the -inf the anchor kernel wrote),
// pos_logit, and the unscaled accumulators of sum_j 2^(s2_ij - ref_i) P_j over all allowed
// columns but the positive one: main_plane [B][d] plus the extra planes of split x pairs.  Raises
// *range_flag when a weight exceeds 2^100.  ws.flags must be zero.
cudaError_t duo_launch_fused_dq(const FwdArgs& a, float* main_plane, const DuoScratch& ws,
                                const float* row_ref, int* range_flag, cudaStream_t st,
                                bool overlap_prev) {
    const Problem& pr = a.p;
    DuoParams p{};
    DuoMaps m;
    if (!duo_setup(&p, &m, pr.Q, pr.ldq, pr.B, pr.P, pr.ldp, pr.N, pr.d, ws, main_plane, pr.d))
        return cudaErrorInvalidValue;
    p.nq = pr.B;
    p.mask_mode = pr.mask_mode;
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.row_ref = row_ref;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.range_flag = range_flag;
    p.dev_status = a.dev_status;
    p.gate = a.gate;
    p.zero_me = reinterpret_cast<int*>(a.red);
    return launch_duo<DMODE_FA>(m.mx, m.mys, m.mya, m.mwld, m.mmain, m.mextra, p, st, overlap_prev);
}

cudaError_t duo_launch_dq_finalize(const float* main_plane, const DuoScratch& ws, const float* row_ref2,
                                   const float* row_lse, const float* pos_ws, const int32_t* pos_idx,
                                   const void* P, int64_t ldp, int64_t B, int64_t N, int d,
                                   int mask_mode, float scale, float* out, int64_t ldo, Gate gate,
                                   cudaStream_t st) {
    const int64_t YT = tiles_of(N), total = tiles_of(B) * YT;
    const int nteams = duo_teams(B, N);
    int64_t all = B * (d / 4);
    int64_t blocks = (all + 255) / 256;
    const int cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    duo_dq_finalize_kernel<<<(int)blocks, 256, 0, st>>>(
        reinterpret_cast<const float4*>(main_plane), reinterpret_cast<const float4*>(ws.extra),
        row_ref2, row_lse, pos_ws, pos_idx, static_cast<const __nv_bfloat16*>(P), ldp, B, N, d / 4,
        mask_mode, YT, total, nteams, scale, out, ldo, gate);
    return cudaGetLastError();
}

}  // namespace gc
