// Tensor-core plan for bf16 inputs with d a multiple of 64 (up to 4096): TMA-staged tiles in
// 128-byte-swizzled shared memory, tcgen05 MMAs with fp32 accumulators in tensor memory, the
// softmax arithmetic in registers.  One kernel template serves three sweeps:
//
//   FWD  (Eq. 1)    x = 128 queries,  y streams passages: S = X Y^T, online row max / sum.
//   DQ   (Eq. 5)    x = 128 queries,  y streams passages: W = exp(S - lse_x) - onehot, acc += W Y
//   DP   (Eq. 6-7)  x = 128 passages, y streams queries:  W = exp(S - lse_y) - onehot, acc += W Y
//   FQ   (Eq. 1+5)  forward fused into the dQ sweep (used by gc_build_cache for wide rows): the
//                   row maximum runs online, W = exp(S - m_ref) with the positive column left
//                   out, acc += W Y; the accumulator is rescaled only when the maximum grows by
//                   more than 2^8.  A finalize pass forms (sum_g acc_g exp(m_g - lse)
//                   + (p_pos - 1) P_pos) / (B tau) with the positive term in fp32.
//
// The stationary tile X (128 x d) stays resident in shared memory when d <= 512; for wider rows
// only its first 6 column chunks stay and the others are re-streamed every step, which leaves
// room for a ring of eight 16 KB stages: the load -> MMA -> release chain of a stage is about
// 1500-2000 cycles long, so the bytes in flight, not the L2 bandwidth, bound the MMA rate.
// Y arrives in (SN x 64) chunks through the same mbarrier ring.  S tiles (128 x SN, fp32) are double buffered in tensor
// memory so the MMAs of step t+1 run while the softmax warps work on step t.  W is written
// back over its S buffer as packed bf16 and used as the A operand (from tensor memory) of the
// second MMA, whose B operand is the same Y chunk read MN-major.  An accumulator of 128 x 768
// fp32 does not fit the 512 tensor-memory columns, so wide rows are split into column parts
// (at most 384 columns each), one CTA per part.  S is never written to global memory.
//
// Warp roles (416 threads): warps 0..3 = TMA producers (the ring stages are dealt out to four
// issuing warps), warp 4 = MMA issuer (and tensor-memory allocator), warps 5..12 = softmax /
// epilogue: two warps per tensor-memory lane quarter, each owning half of the tile's columns,
// one thread per tile row.
// Every wait is bounded: on a timeout the CTA raises GC_DEV_WAIT_LIMIT, drains and exits.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include "gc_internal.h"

namespace gc {

namespace {

constexpr int XROWS = 128;                 // rows of the stationary tile = MMA M
constexpr int CHUNK_BYTES_PER_ROW = 128;   // 64 bf16 = one swizzle row
constexpr uint32_t X_CHUNK_BYTES = XROWS * CHUNK_BYTES_PER_ROW;
constexpr int NPROD = 2;                   // TMA producer warps
constexpr int MMA_WARP = NPROD;
constexpr int NSOFT = 8;                   // softmax / epilogue warps
constexpr int NTHREADS = 32 * (NPROD + 1 + NSOFT);
constexpr int MAX_STAGES = 12;
constexpr uint32_t CHUNK_BYTES = 16384;    // 128 rows x 64 columns: one X chunk or one Y chunk
constexpr int TMEM_COLS = 512;
constexpr int MAX_D = 4096;                // wider rows just take more column parts
constexpr int MAX_PART_CHUNKS = 6;         // 384 accumulator columns
constexpr size_t SMEM_LIMIT = 232448;      // 227 KB per block
constexpr size_t SMEM_STATIC_RESERVE = 2048;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;

enum { MODE_FWD = 0, MODE_DQ = 1, MODE_DP = 2, MODE_FQ = 3 };   // FQ: forward fused into dQ

// Optional diagnostics (-DGC_TC_TRACE): cycles each role spends waiting, summed over CTAs.
#ifdef GC_TC_TRACE
enum { TR_MMA_TOTAL, TR_MMA_WAIT_Y, TR_MMA_WAIT_W, TR_SM_TOTAL, TR_SM_WAIT_S, TR_SM_EPI,
       TR_PROD_TOTAL, TR_PROD_WAIT, TR_CTAS, TR_MMA_ISSUE, TR_MMA_COMMIT, TR_ACC_ISSUE, TR_ACC_COMMIT, TR_SFULL_COMMIT,
       TR_CTA_LIFE, TR_SETUP, TR_T0_MIN, TR_T0_MAX, TR_T1_MIN, TR_T1_MAX, TR_COUNT };
__device__ unsigned long long g_trace[4][TR_COUNT];
#define TR_DECL(v) long long v = 0
#define TR_BEGIN(v) long long v##_t0 = clock64()
#define TR_END(v) v += clock64() - v##_t0
#define TR_ADD(mode, slot, v) atomicAdd(&g_trace[mode][slot], (unsigned long long)(v))
#else
#define TR_DECL(v)
#define TR_BEGIN(v)
#define TR_END(v)
#define TR_ADD(mode, slot, v)
#endif

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
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the CTA is aborting or the time limit passed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try(bar, parity)) return true;
    uint64_t t0 = global_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if ((++spins & 127u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > WAIT_LIMIT_NS) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
// True on exactly one lane of a converged warp.  The surrounding loops run on all 32 lanes with
// warp-uniform values, so that addresses and descriptors can stay in uniform registers, which
// is where bulk-tensor and tcgen05 instructions read them from.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// ---- CTA-pair (cluster of 2) helpers -------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\t"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];"
                 ::"r"(cluster_addr) : "memory");
}
// Bulk tensor load of a CTA pair: the data lands in the executing CTA, the transaction bytes are
// counted on an mbarrier that may live in the other CTA of the pair (no multicast).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0,
                                                 int c1, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar_cluster)
        : "memory");
}
// Arrives on the mbarrier at this offset in both CTAs of the pair once all MMAs issued so far
// by this thread have completed.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
        "[%0], %1;"
        ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
// Shared-memory matrix descriptors for 128-byte-swizzled tiles with 128-byte rows.  The high
// word is constant: stride between 8-row groups = 1024 bytes (>> 4), descriptor version 1,
// layout type 2 (SWIZZLE_128B).  The low word holds the start address (>> 4) and, in bits 16-29,
// the leading byte offset (>> 4): the distance between 64-element atoms along M/N of an
// MN-major operand (ignored for K-major operands).  A K-major operand advances 32 bytes
// (low word + 2) per K = 16; an MN-major operand advances 16 rows = 2048 bytes (low word + 128).
constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr >> 4) & 0x3FFFu) | ((lbo_bytes >> 4) << 16);
}
// D[tmem] (+)= A[smem] * B[smem].  The issuing thread is alone on its scheduler, so every scalar
// instruction spent per MMA shows up as idle tensor time: keep the operands precomputed.
template <bool ACC, bool PAIR>
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo,
                                       uint32_t idesc) {
    if (PAIR) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, %5, 0;\n\t"
            "mov.b64 da, {%1, %4};\n\t"
            "mov.b64 db, {%2, %4};\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(DESC_HI), "n"(ACC ? 1 : 0)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
            "setp.ne.b32 p, %5, 0;\n\t"
            "mov.b64 da, {%1, %4};\n\t"
            "mov.b64 db, {%2, %4};\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(DESC_HI), "n"(ACC ? 1 : 0)
            : "memory");
    }
}
// D[tmem] (+)= A[tmem] * B[smem]
template <bool ACC, bool PAIR>
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo,
                                       uint32_t idesc) {
    if (PAIR) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
            "setp.ne.b32 p, %5, 0;\n\t"
            "mov.b64 db, {%2, %4};\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(DESC_HI), "n"(ACC ? 1 : 0)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
            "setp.ne.b32 p, %5, 0;\n\t"
            "mov.b64 db, {%2, %4};\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}"
            ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(DESC_HI), "n"(ACC ? 1 : 0)
            : "memory");
    }
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]),
          "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]),
          "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]),
          "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]),
          "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// ---- epilogue: accumulator blocks leave through shared memory and bulk tensor stores ---------------
// One warp's block of 32 rows x 32 fp32 columns is written to a 4 KB buffer in the 128-byte
// swizzle the tensor map expects (16-byte chunk j of row r at chunk j ^ (r & 7)), which also
// makes the float4 stores conflict-free, and then leaves with one bulk tensor store; rows past
// the end of the matrix are clipped by the tensor map.
__device__ __forceinline__ void stage_block(uint32_t buf, const uint32_t (&v)[32], float sc,
                                            int lane) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t addr = buf + lane * 128 + ((j ^ (lane & 7)) << 4);
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};"
                     ::"r"(addr), "f"(__uint_as_float(v[4 * j]) * sc),
                       "f"(__uint_as_float(v[4 * j + 1]) * sc),
                       "f"(__uint_as_float(v[4 * j + 2]) * sc),
                       "f"(__uint_as_float(v[4 * j + 3]) * sc)
                     : "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the bulk store
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1,
                                             int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Writes accumulator blocks cb = half, half + 2, ... (32 columns each) of this warp's 32 rows.
// `slot` is the warp's 8 KB staging area (two buffers).
__device__ __forceinline__ void store_acc_blocks(uint32_t tmem_rows, int nblocks, int half,
                                                 uint32_t slot, float sc, int lane,
                                                 const CUtensorMap* mapO, int col0, int row0,
                                                 int plane) {
    int n = 0;
    for (int cb = half; cb < nblocks; cb += 2, ++n) {
        uint32_t v[32];
        tmem_ld32(tmem_rows + cb * 32, v);
        if (n >= 2) {   // the store issued two blocks ago has finished reading this buffer
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            __syncwarp();
        }
        tmem_ld_wait();
        const uint32_t buf = slot + (n & 1) * 4096;
        stage_block(buf, v, sc, lane);
        __syncwarp();
        if (lane == 0) tma_store_3d(mapO, buf, col0 + cb * 32, row0, plane);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, M = 128.
__device__ __forceinline__ uint32_t instr_desc(int n, bool b_mn_major, int m = XROWS) {
    uint32_t d = 0;
    d |= 1u << 4;                          // D format f32
    d |= 1u << 7;                          // A format bf16
    d |= 1u << 10;                         // B format bf16
    d |= (b_mn_major ? 1u : 0u) << 16;     // B major
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(m >> 4) << 24;          // 128, or 256 for an MMA across a CTA pair
    return d;
}

__device__ __forceinline__ void part_range(int64_t steps, int groups, int g, int64_t* lo,
                                           int64_t* hi) {
    int64_t base = steps / groups, rem = steps % groups;
    *lo = g * base + (g < rem ? g : rem);
    *hi = *lo + base + (g < rem ? 1 : 0);
}

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
template <int MODE, int SN, int NBUF, bool PAIR>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
          const __grid_constant__ CUtensorMap mapYh, const __grid_constant__ CUtensorMap mapO,
          const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float row_max_xch[2][XROWS];      // FQ: [column half][row] block maxima
    volatile int* abort_flag = &abort_s;

    static_assert(SN == 128, "a Y chunk is 128 rows: the same 16 KB as an X chunk");
    constexpr uint32_t S_COL0 = TMEM_COLS - NBUF * SN;  // S buffers sit at the top columns
    // WS ("W through shared memory"): paired wide-row sweeps write the bf16 weights to two
    // shared-memory buffers instead of over the single S tile.  The S tile is then free as soon as
    // the softmax warps have read it, S(t+1) is issued while softmax(t) computes, and acc(t)
    // follows from W buffer t & 1: the tensor pipe no longer waits for the softmax.
    constexpr bool WS = PAIR && NBUF == 1 && MODE != MODE_FWD;
    constexpr int LAG = WS ? 1 : NBUF - 1;              // steps between S(t) and acc(t) issue
    constexpr int BSH = (NBUF == 2) ? 1 : 0;            // log2(NBUF)
    constexpr int WBUF = WS ? 2 : NBUF;                 // W buffers (w_full barriers in use)
    constexpr int WSH = (WBUF == 2) ? 1 : 0;
#ifdef GC_TC_TRACE
    const unsigned long long cta_t0 = global_ns();
    const long long cta_c0 = clock64();
#endif
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
    const int c_count = (MODE == MODE_FWD) ? 0 : min(p.dpc, p.kc - c_begin);

    int64_t lo, hi;
    part_range((p.ny + SN - 1) / SN, p.groups, g, &lo, &hi);
    const int T = (int)(hi - lo);

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t x_smem = base;
    const uint32_t w_smem = base + (uint32_t)p.xres * X_CHUNK_BYTES;   // WS: two 32 KB W buffers
    const uint32_t y_smem = w_smem + (WS ? 2u * 32768u : 0u);          // the ring
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
#ifdef GC_TC_TRACE
    if (threadIdx.x == 0) TR_ADD(MODE, TR_SETUP, clock64() - cta_c0);
#endif
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
            TR_DECL(tr_wait);
            TR_BEGIN(tr_total);
            // Claims the next ring stage if it belongs to this warp: waits until the MMAs that
            // read its previous contents have completed.  Returns the stage or -1.
            auto acquire = [&]() -> int {
                const int stage = next;
                const uint32_t phase = next_phase;
                if (++next == p.nstage) { next = 0; next_phase ^= 1u; }
                if (!ok || (stage & (NPROD - 1)) != warp) return -1;
                TR_BEGIN(tr_wait);
                const bool got = mbar_wait(smem_u32(&bars.y_empty[stage]), phase ^ 1u, abort_flag);
                TR_END(tr_wait);
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
                if (MODE != MODE_FWD && t >= LAG) {
                    for (int c = 0; c < c_count; c += p.ipc)
                        load_item(2, c_begin + c, (lo + t - LAG) * SN);
                }
            }
#ifdef GC_TC_TRACE
            if (warp == 0 && lane == 0) {
                TR_ADD(MODE, TR_PROD_TOTAL, clock64() - tr_total_t0);
                TR_ADD(MODE, TR_PROD_WAIT, tr_wait);
                TR_ADD(MODE, TR_CTAS, 1);
            }
#endif
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
            TR_DECL(tr_wy);
            TR_DECL(tr_ww);
            TR_DECL(tr_is);
            TR_DECL(tr_cm);
            TR_DECL(tr_ai);
            TR_DECL(tr_ac);
            TR_DECL(tr_sf);
            TR_BEGIN(tr_total);
            bool ok = mbar_wait(smem_u32(&bars.x_full), 0, abort_flag);
            tc_fence_after();
            // Waits for the next ring stage to be filled; returns its index or -1.
            auto next_stage = [&]() -> int {
                const int stage = next;
                const uint32_t phase = next_phase;
                if (++next == p.nstage) { next = 0; next_phase ^= 1u; }
                TR_BEGIN(tr_wy);
                const bool got = mbar_wait(smem_u32(&bars.y_full[stage]), phase, abort_flag);
                TR_END(tr_wy);
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
                    if (MODE == MODE_FWD && t >= NBUF) {
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
                            TR_BEGIN(tr_is);
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
                            TR_END(tr_is);
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
                                TR_BEGIN(tr_is);
                                if (elect_one()) {
                                    if (c + j == 0) mma_ss<false, true>(d_tmem, xa, yj, idesc_s);
                                    else            mma_ss<true, true>(d_tmem, xa, yj, idesc_s);
                                    mma_ss<true, true>(d_tmem, xa + 2, yj + 2, idesc_s);
                                    mma_ss<true, true>(d_tmem, xa + 4, yj + 4, idesc_s);
                                    mma_ss<true, true>(d_tmem, xa + 6, yj + 6, idesc_s);
                                    if (xs >= 0) tc_commit_pair(smem_u32(&bars.y_empty[xs]));
                                    if (j == 1) tc_commit_pair(smem_u32(&bars.y_empty[ys]));
                                }
                                TR_END(tr_is);
                            }
                        }
                    }
                    if (!ok) break;
                    TR_BEGIN(tr_sf);
                    if (elect_one()) commit(smem_u32(&bars.s_full[b]));
                    TR_END(tr_sf);
                }
                if (MODE != MODE_FWD && t >= LAG) {
                    const int u = t - LAG, b = u & (WBUF - 1);
                    TR_BEGIN(tr_ww);
                    ok = mbar_wait(smem_u32(&bars.w_full[b]), (u >> WSH) & 1, abort_flag);
                    TR_END(tr_ww);
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
                        TR_BEGIN(tr_ai);
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
                        TR_END(tr_ai);
                    }
                    if (WS && ok && elect_one()) commit(smem_u32(&bars.w_empty[b]));
                }
            }
            if (ok && MODE != MODE_FWD && elect_one()) commit(smem_u32(&bars.acc_full));
#ifdef GC_TC_TRACE
            if (lane == 0) {
            TR_ADD(MODE, TR_MMA_TOTAL, clock64() - tr_total_t0);
            TR_ADD(MODE, TR_MMA_WAIT_Y, tr_wy);
            TR_ADD(MODE, TR_MMA_WAIT_W, tr_ww);
            TR_ADD(MODE, TR_MMA_ISSUE, tr_is);
            TR_ADD(MODE, TR_MMA_COMMIT, tr_cm);
            TR_ADD(MODE, TR_ACC_ISSUE, tr_ai);
            TR_ADD(MODE, TR_ACC_COMMIT, tr_ac);
            TR_ADD(MODE, TR_SFULL_COMMIT, tr_sf);
            }
#endif
        }
    } else {
        // ------------------------------ softmax / epilogue warps --------------------------------
        const int q = warp & 3;                        // tensor-memory lane quarter of this warp
        const int half = (warp - (NPROD + 1)) >> 2;    // which half of the tile's columns
        constexpr int CB_PER = SN / 64;                // 32-column blocks per half
        const int cb0 = half * CB_PER;
        const int row = q * 32 + lane;
        const int64_t x = x0 + row;
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
        TR_DECL(tr_ws);
        TR_DECL(tr_epi);
        TR_BEGIN(tr_total);

        if (MODE == MODE_FWD) {
            float m = -INFINITY, l = 0.f;
            const int32_t pos_x = (x < p.nx) ? p.pos_idx[x] : -1;
            for (int t = 0; t < T; ++t) {
                const int b = t & (NBUF - 1);
                TR_BEGIN(tr_ws);
                ok = mbar_wait(smem_u32(&bars.s_full[b]), (t >> BSH) & 1, abort_flag);
                TR_END(tr_ws);
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
                    if (pos_x >= yb && pos_x < yb + 32 && !(self_mask && x == pos_x)) {
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
                    if (self_mask && x >= yb && x < yb + 32) {
                        const int rel = (int)(x - yb);
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
        } else if (MODE == MODE_FQ) {
            // ---------------- forward fused into the dQ sweep ----------------
            // m_ref is the power-of-two scale all weights of a row share (both column halves);
            // l is this half's sum of 2^(s2 - m_ref) over its allowed columns, positive included.
            float m_ref = 0.f, l = 0.f;
            const int32_t pos_x = (x < p.nx) ? p.pos_idx[x] : -1;
            for (int t = 0; t < T; ++t) {
                const int64_t y0 = (lo + t) * SN;
                TR_BEGIN(tr_ws);
                ok = mbar_wait(smem_u32(&bars.s_full[0]), t & 1, abort_flag);
                TR_END(tr_ws);
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
                                         !(self_mask && x == pos_x);
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
                    if (self_mask && x >= yb && x < yb + 32) {
                        const int rel = (int)(x - yb);
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
            TR_BEGIN(tr_epi);
            if (ok) ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
            if (ok) {
                tc_fence_after();
                // every MMA and every load has completed: the dynamic shared memory is free
                const uint32_t slot = base + (uint32_t)(warp - (NPROD + 1)) * 8192u;
                store_acc_blocks(tmem + lane_addr, c_count * 2, half, slot, 1.f, lane, &mapO,
                                 c_begin * 64, (int)x0 + q * 32, g);
            }
            TR_END(tr_epi);
        } else {
            // per-row constants (DQ: the row is a query)
            float lse2_x = 0.f;
            int32_t pos_x = -1;
            if (MODE == MODE_DQ && x < p.nx) {
                lse2_x = p.row_lse[x] * 1.4426950408889634f;
                pos_x = p.pos_idx[x];
            }
            for (int t = 0; t < T; ++t) {
                const int b = t & (NBUF - 1);
                const int64_t y0 = (lo + t) * SN;
                // DP: the columns are queries; lane j holds lse / pos of column 32 cb + j
                float lse2_y[CB_PER];
                int32_t pos_y[CB_PER];
                if (MODE == MODE_DP) {
#pragma unroll
                    for (int j = 0; j < CB_PER; ++j) {
                        const int64_t y = y0 + (cb0 + j) * 32 + lane;
                        lse2_y[j] = (y < p.ny) ? p.row_lse[y] * 1.4426950408889634f : INFINITY;
                        pos_y[j] = (y < p.ny) ? p.pos_idx[y] : -1;
                    }
                }
                TR_BEGIN(tr_ws);
                ok = mbar_wait(smem_u32(&bars.s_full[b]), (t >> BSH) & 1, abort_flag);
                TR_END(tr_ws);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sbuf = tmem + lane_addr + S_COL0 + b * SN;
                // W of this half goes to the first columns of the half's own S region (already
                // read by this warp): columns half * SN/2 + 16 j for block j.
                // both 32-column blocks are requested before the single wait
                uint32_t vv[CB_PER][32];
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) tmem_ld32(sbuf + (cb0 + j) * 32, vv[j]);
                tmem_ld_wait();
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
#pragma unroll
                for (int j = 0; j < CB_PER; ++j) {
                    const int cb = cb0 + j;
                    uint32_t (&v)[32] = vv[j];
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
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            const float ls = __shfl_sync(0xffffffffu, lse2_y[j], c);
                            w[c] = ex2(fmaf(__uint_as_float(v[c]), p.c1, -ls));   // OOB: ex2(-inf)
                        }
                        // one-hot: column c's query has its positive at row pos - x0 of this tile
                        const int64_t rel_row = (int64_t)pos_y[j] - x0;
                        const bool mine = (pos_y[j] >= 0) && rel_row >= q * 32 && rel_row < q * 32 + 32;
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
                    if (self_mask && x >= yb && x < yb + 32) {
                        const int rel = (int)(x - yb);
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
            // epilogue: accumulator columns of this part -> global memory (32-column blocks are
            // dealt alternately to the two warps of a lane quarter); final values are scaled,
            // partial sums of a split sweep are not
            TR_BEGIN(tr_epi);
            if (ok) ok = mbar_wait(smem_u32(&bars.acc_full), 0, abort_flag);
            if (ok) {
                tc_fence_after();
                const bool final_out = (p.groups == 1);
                const uint32_t slot = base + (uint32_t)(warp - (NPROD + 1)) * 8192u;
                store_acc_blocks(tmem + lane_addr, c_count * 2, half, slot,
                                 final_out ? p.out_scale : 1.f, lane, &mapO, c_begin * 64,
                                 (int)x0 + q * 32, final_out ? 0 : g);
            }
            TR_END(tr_epi);
        }
#ifdef GC_TC_TRACE
        if (q == 0 && half == 0 && lane == 0) {
            TR_ADD(MODE, TR_SM_TOTAL, clock64() - tr_total_t0);
            TR_ADD(MODE, TR_SM_WAIT_S, tr_ws);
            TR_ADD(MODE, TR_SM_EPI, tr_epi);
        }
#endif
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
#ifdef GC_TC_TRACE
    if (threadIdx.x == 0) {
        const unsigned long long t1 = global_ns();
        TR_ADD(MODE, TR_CTA_LIFE, clock64() - cta_c0);
        atomicMin(&g_trace[MODE][TR_T0_MIN], cta_t0);
        atomicMax(&g_trace[MODE][TR_T0_MAX], cta_t0);
        atomicMin(&g_trace[MODE][TR_T1_MIN], t1);
        atomicMax(&g_trace[MODE][TR_T1_MAX], t1);
    }
#endif
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

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) !=
                cudaSuccess || qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// Row-major bf16 matrix [rows x d], boxes of (box_rows x 64 columns), 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int d, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// fp32 destination of the accumulators as [planes][rows][d]: the output matrix itself (one plane,
// row pitch ld) or the per-part partial sums (planes = parts of the streamed range, pitch d).
// Boxes of 32 rows x 32 columns, 128-byte swizzle.
bool make_out_map(CUtensorMap* map, float* base, int64_t rows, int d, int64_t ld, int planes) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)planes};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)rows * (cuuint64_t)ld * 4};
    cuuint32_t box[3] = {32, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int parts_for(int kc) { return (kc + MAX_PART_CHUNKS - 1) / MAX_PART_CHUNKS; }
int chunks_per_part(int kc) { int n = parts_for(kc); return (kc + n - 1) / n; }

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
    sp.xres = ws ? 2 : (kc <= 8 ? kc : 6);
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
                       const CUtensorMap& mo, const TcParams& p, int64_t ctas, cudaStream_t st) {
    constexpr bool WS = PAIR && NBUF == 1 && MODE != MODE_FWD;
    SmemPlan sp = smem_plan(p.kc, PAIR, WS);
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(tc_kernel<MODE, SN, NBUF, PAIR>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(SMEM_LIMIT - SMEM_STATIC_RESERVE));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = sp.dynamic_bytes;
    cfg.stream = st;
    TcParams pp = p;
    pp.nstage = sp.nstage;
    pp.xres = sp.xres;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (!PAIR) {
        tc_kernel<MODE, SN, NBUF, false><<<(unsigned)ctas, NTHREADS, sp.dynamic_bytes, st>>>(
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
                   const CUtensorMap& mo, const TcParams& p, cudaStream_t st) {
    const int64_t ctas = cta_count(MODE, p.kc, p.nx, p.ny, p.dparts, p.groups);
    if (use_pair(MODE, p.kc, p.nx, p.ny))
        return launch_one<MODE, SN, NBUF, true>(mx, my, myh, mo, p, ctas, st);
    return launch_one<MODE, SN, NBUF, false>(mx, my, myh, mo, p, ctas, st);
}

}  // namespace

#ifdef GC_TC_TRACE
extern "C" int gc_debug_trace(unsigned long long* out, int clear) {
    if (out && cudaMemcpyFromSymbol(out, g_trace, sizeof(g_trace)) != cudaSuccess) return 1;
    if (clear) {
        static unsigned long long zero[4][TR_COUNT] = {};
        for (int m = 0; m < 4; ++m) zero[m][TR_T0_MIN] = zero[m][TR_T1_MIN] = ~0ull;
        if (cudaMemcpyToSymbol(g_trace, zero, sizeof(zero)) != cudaSuccess) return 1;
    }
    return 0;
}
#endif

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
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.dev_status = a.dev_status;
    return launch<MODE_FWD, SN, 2>(mx, my, myh, mx, p, st);   // no accumulator output
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
    p.inv_tau = 1.f / pr.tau;
    p.c1 = 1.4426950408889634f / pr.tau;
    p.pos_idx = pr.pos_idx;
    p.part_m = a.part_m; p.part_l = a.part_l; p.pos_logit = a.pos_logit;
    p.partial = partial;
    p.dev_status = a.dev_status;
    CUtensorMap mo;
    if (!make_out_map(&mo, partial, pr.B, pr.d, pr.d, groups)) return cudaErrorInvalidValue;
    return launch<MODE_FQ, SN, 1>(mx, my, myh, mo, p, st);
}

cudaError_t tc_launch_sweep(const SweepArgs& a, cudaStream_t st) {
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
    p.inv_tau = a.inv_tau;
    p.c1 = 1.4426950408889634f * a.inv_tau;
    p.out_scale = a.out_scale;
    p.row_lse = a.row_lse; p.pos_idx = a.pos_idx;
    p.out = a.out; p.ldo = a.ldo; p.partial = a.partial;
    p.dev_status = a.dev_status;
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
