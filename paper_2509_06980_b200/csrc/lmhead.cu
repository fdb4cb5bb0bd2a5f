// Fused LM-head variant: the logits z = hidden W^T are formed tile by tile on the tensor cores
// (tcgen05.mma, operands staged in shared memory by TMA, accumulators in tensor memory) and consumed
// by the softmax / loss epilogue straight from tensor memory, so they never reach HBM.
//
// One warp-specialised kernel template serves three contractions (all bf16 x bf16 -> fp32):
//   LSE   z tile = H W^T, epilogue keeps a running (max, sum exp) per token      -> log-sum-exp;
//         for rows that take part in the backward it also stores e = exp(z - rho_t) as bf16, rho_t a
//         per-row reference known before the sweep (or exp(z - tile max) on the fallback path)
//   GH    grad_hidden = f_t (e W)      (A = e K-major, B = W vocabulary-major rows: N-major operand;
//                                       f_t = c_t exp(rho_t - lse_t) applied in the epilogue)
//   GW    grad_W     += e^T (f_t H)    (both operands token-major rows: M-/N-major operands)
// CTA = 192 threads: warp 0 issues TMA loads into a multi-stage ring, warp 1 issues the MMAs (one
// thread), warps 2..5 drain the accumulator with tcgen05.ld (one token row per thread).  The sweeps
// use a double-buffered 128 x 256 fp32 accumulator (all 512 TMEM columns), so the drain of a tile
// overlaps the multiplies of the next; the gradient contractions use both halves as two
// accumulators that share every B slab.  Every mbarrier wait is bounded; a wait that runs out raises
// a CTA-wide abort flag, all roles leave their loops, tensor memory is released and RLF_DEV_TIMEOUT
// is set.  The persistent workers of a launch meet on a global counter before each of their units
// (pacing), which keeps the operand slabs they share in L2.
//
// Forward + backward: the tokens are partitioned into unmasked rows and the others (only the first
// carry gradient).  Unmasked rows go by chunks: LSE with the exponentials stored in a [chunk, V] bf16
// scratch, per-row factors once the rows' log-sum-exp is known, then GH and GW read the scratch:
// three contractions per unmasked row, one per masked row, no recomputation and no pass over the
// scratch in between.  The logits themselves are never stored; the bf16 scratch is (stated in the
// entry point's contract).
#include <cuda.h>

#include <atomic>
#include <mutex>

#include "common.cuh"

namespace rlf {
namespace lm {

constexpr int BM = 128, BN = 256, BK = 64;
// Single-CTA form: each CTA multiplies a 128 x 256 tile (A 16 KB + B 32 KB per stage, 4 stages).
// Pair form (cta_group::2): two CTAs of a cluster multiply a 256 x 256 tile; each stages its own 128
// rows of A and HALF of B (16 KB + 16 KB per stage, 6 stages), the leader CTA issues the MMAs, and
// each CTA's tensor memory receives its own 128 rows of the accumulator.  Per flop the pair form
// moves two thirds of the shared-memory bytes of the single form.
constexpr int kABytes = BM * BK * 2;
constexpr int kDrainPitch = 36;              // floats per row of a drain staging tile (32 + 4 of padding)
// Two-accumulator pair form (ACC2, the two gradient contractions): a pair works on TWO 256-row tiles
// against the same 256 columns, each CTA staging two A tiles beside its half of B (48 KB per stage, 4
// stages), so every B slab that crosses L2 -> shared memory is used for 512 rows: three quarters of
// the shared-memory fill bytes per flop of the plain pair form, and half the passes over the B
// matrix.  The two accumulators take all 512 TMEM columns, so the drain of a unit does not overlap the
// next unit's multiplies; with K running over the whole vocabulary or a whole chunk of tokens the
// drain is a per cent or two of a unit.
template <bool PAIR, bool ACC2 = false> struct Cfg {
    static_assert(PAIR || !ACC2, "two accumulators per CTA exist in pair form only");
    static constexpr int kAcc = ACC2 ? 2 : 1;
    static constexpr int kStages = ACC2 ? 4 : (PAIR ? 6 : 4);
    static constexpr int kBRows = PAIR ? BN / 2 : BN;
    static constexpr int kBBytes = kBRows * BK * 2;
    static constexpr int kStageBytes = kAcc * kABytes + kBBytes;
    // + alignment slack, the barriers, and (two-accumulator form) a 32 x 32 fp32 staging tile per drain warp
    static constexpr int kDrainBytes = ACC2 ? 4 * 32 * kDrainPitch * 4 : 0;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256 + kDrainBytes;
};
constexpr int kMaxStages = 6;
constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kSlabBytes = 64 * BK * 2;      // one 64-wide slab of an MN-major operand: 64 k-rows of 128 B

enum Mode { kLse = 0, kGradHidden = 2, kGradW = 3 };

// The [rows, V] scratch that carries a chunk's exponentials, then its dZ, is stored in blocks of
// 128 token rows x 64 vocabulary columns (16 KB, rows of 128 bytes), blocks of one token tile side by
// side: element (row, col) sits at ((row / 128 * nc + col / 64) * 128 + row % 128) * 64 + col % 64,
// nc = 4 x the number of 256-column tiles.  Every operand box the two gradient contractions fetch
// (128 or 64 rows of 128 bytes) is then one contiguous piece of memory, and so is what a warp of the
// sweep's epilogue stores; with plain rows of 2 V bytes each of those touched 64 - 128 DRAM pages for
// 128 bytes apiece.
constexpr int kDzBlockRows = 128, kDzBlockCols = 64;
__host__ __device__ __forceinline__ long long dz_offset(long long row, int col, int nc) {
    return (((row >> 7) * nc + (col >> 6)) * kDzBlockRows + (row & 127)) * kDzBlockCols + (col & 63);
}

struct GemmParams {
    int mode;
    int M, N;                 // extent of the output tile grid in rows / columns (valid elements)
    int m_tiles, n_tiles, k_slabs;
    int nsplit, n_tiles_per_split;
    int m_block;              // kLse: row units per scheduling block
    float2* part;             // kLse: [M][nsplit] (max, sum exp)
    float* part_u;            // kLse (optional): [M][nsplit] sum of 2^x x, x the base-2 exponent against that max
    __nv_bfloat16* dz;        // kLse (optional) out, blocked scratch (see dz_offset): exp(z - tile max) as bf16
    float* tmax;              // kLse with dz: [M][n_tiles] the tile maxima those exponentials refer to
    int dz_nc;                // 64-column blocks per token tile of the blocked scratch; also set for the
                              // gradient contractions, whose A operand is that scratch
    __nv_bfloat16* out_bf16;  // kGradHidden out [M][out_stride]
    float* out_f32;           // kGradW out [M][out_stride]
    long long out_stride;
    int accumulate;
    int32_t* dev_status;
    // Token extent known only on the device (launches over the gathered unmasked / masked rows):
    // when live_count is set, the token extent of this launch is
    // clamp(*live_count - live_off, 0, M or K as built on the host).
    const int* live_count;
    int live_off;
    const int32_t* row_index; // kGradHidden: output row of compact row r is row_index[live_off + r]
    const float* ref;         // kLse with dz (optional): per-row reference of the stored exponentials (see below)
    const float* row_scale;   // kGradHidden (optional): fp32 factor of compact row r applied to its output row
    const int* run_flag;      // optional: the launch does nothing unless *run_flag == run_want
    int run_want;
    // Pacing (optional): a counter, zero at launch, on which the load-issuing threads of all workers meet
    // before each of their units but the first.  Workers that share operand slabs through L2 then
    // request them within a short time of each other; left alone they drift apart over a launch until
    // each fetches its slabs from HBM on its own.  Waits are bounded and only delay loads: a worker
    // that gives up runs on unpaced.
    int* pace;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
constexpr int kWaitPolls = 1 << 22;
constexpr int kPacePolls = 1 << 14;          // a pacing wait gives up after about 10 ms and is not taken again
// wait (bounded) until the pacing counter has reached `want`; `seen` is a value read earlier
__device__ __forceinline__ void pace_settle(const int* counter, int seen, long long want, bool& keep_waiting) {
    int polls = 0;
    while ((long long)seen < want) {
        if (++polls > kPacePolls) { keep_waiting = false; return; }
        __nanosleep(64);
        asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
    }
}
// bounded wait; on failure (or if another role already gave up) returns false
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (int i = 0; i < kWaitPolls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 1023) == 1023 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// cta_group::2 forms: the MMA spans both CTAs of the pair; its commit arrives on the same barrier
// offset in both CTAs; TMA loads of either CTA credit a barrier in the leader CTA.
__device__ __forceinline__ void tc_mma2(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// The multicast here is that of a BARRIER SIGNAL: the commit arrives on the mbarrier at the same offset in
// both CTAs of the pair (mask 0b11).  No load in this file is multicast -- every cp.async.bulk.tensor
// below is a plain per-CTA copy -- and every tensor map covers this GPU's own memory.
__device__ __forceinline__ void tc_commit2(uint32_t bar) {
    const unsigned short both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 :: "r"(bar), "h"(both) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 :: "r"(dst), "l"(map), "r"(leader_bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" :: "r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t pair_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void pair_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// the same load without its wait, and the wait: the registers pass through the wait as in/out operands
// so that no use of them can be scheduled ahead of it
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait(uint32_t (&v)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                   "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                   "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :: "memory");
}

// Shared-memory operand descriptor, 128-byte swizzle, descriptor version 1.
//   K-major tile  (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart): LBO 1, SBO 1024 B.
//   MN-major tile (64-wide slabs, each 64 k-rows of 128 B): LBO = slab pitch 8192 B, SBO 1024 B.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, bool mn_major) {
    const uint64_t lbo = mn_major ? (uint64_t)(kSlabBytes >> 4) : 1ull;
    return (uint64_t)((addr & 0x3FFFF) >> 4) | (lbo << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: D fp32, A and B bf16, M = 128, N = 256, majorness per operand.
__host__ __device__ constexpr uint32_t instr_desc(bool a_mn, bool b_mn, int m) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct SmemCtl {
    unsigned long long full[kMaxStages];
    unsigned long long empty[kMaxStages];
    unsigned long long tmem_full[2];
    unsigned long long tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

static_assert(sizeof(SmemCtl) <= 256, "the barriers share a 256-byte slot behind the stage ring");

// ---- the kernel -----------------------------------------------------------------------------
template <bool PAIR, bool ACC2>
__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const GemmParams p) {
    using C = Cfg<PAIR, ACC2>;
    constexpr int NACC = C::kAcc;
    extern __shared__ unsigned char smem_raw[];
    // a launch that is conditional on a device-side flag (uniform over the grid): leave before
    // anything is set up
    if (p.run_flag && *p.run_flag != p.run_want) return;
    // operand stages must sit on 1024-byte boundaries (swizzle atom)
    const uint32_t raw = smem_addr(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem_raw + (tiles - raw) + C::kStages * C::kStageBytes);
    float* drain_stage = reinterpret_cast<float*>(smem_raw + (tiles - raw) + C::kStages * C::kStageBytes + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool a_mn = p.mode == kGradW;
    const bool b_mn = p.mode == kGradHidden || p.mode == kGradW;
    const bool sweep = p.mode == kLse;                      // a unit sweeps several vocabulary tiles
    // in pair form the scheduling unit covers two token tiles: this CTA takes tile 2 * mp + rank
    const int rank = PAIR ? (int)pair_rank() : 0;
    int M = p.M, m_tiles = p.m_tiles, k_slabs = p.k_slabs;
    if (p.live_count) {
        const int host_extent = p.mode == kGradW ? p.k_slabs * BK : p.M;
        const int live = max(0, min(*p.live_count - p.live_off, host_extent));
        if (p.mode == kGradW) k_slabs = (live + BK - 1) / BK;
        else { M = live; m_tiles = (live + BM - 1) / BM; }
    }
    // no tokens under a grad_W tile: nothing to add; without accumulate the tile is still written (zeros)
    const bool no_k = k_slabs == 0;
    // token (or vocabulary) tiles per scheduling unit: 1, 2 in pair form, 4 with two accumulators; this
    // CTA's tile for accumulator a of unit m is kTilesPerUnit * m + 2 * a + rank
    constexpr int kTilesPerUnit = (PAIR ? 2 : 1) * NACC;
    const int m_units = (m_tiles + kTilesPerUnit - 1) / kTilesPerUnit;
    const int units = (no_k && p.accumulate) ? 0 : sweep ? m_units * p.nsplit : m_units * p.n_tiles;
    const int worker = PAIR ? blockIdx.x >> 1 : blockIdx.x;
    const int workers = PAIR ? gridDim.x >> 1 : gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(smem_addr(&ctl->full[s]), 1);
            mbar_init(smem_addr(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_addr(&ctl->tmem_full[b]), 1);
            mbar_init(smem_addr(&ctl->tmem_empty[b]), PAIR ? 8 : 4);
        }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         :: "r"(smem_addr(&ctl->tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         :: "r"(smem_addr(&ctl->tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) pair_sync();        // both CTAs' barriers exist before either signals the other
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // unit -> (m unit, first n tile, one-past-last n tile)
    const int split_base = sweep ? p.n_tiles / p.nsplit : 0, split_rem = sweep ? p.n_tiles % p.nsplit : 0;
    auto unit_range = [&](int u, int& m, int& n0, int& n1) {
        if (sweep) {
            // blocks of m_block row units; inside a block, units run over its row units first, then
            // over the splits: the CTAs running at one time share both the rows of the head they
            // sweep and a set of token tiles small enough to stay in L2
            const int per_block = p.m_block * p.nsplit;
            const int blk = u / per_block, within = u - blk * per_block;
            const int rows_here = min(p.m_block, m_units - blk * p.m_block);
            const int sp = within / rows_here;
            m = blk * p.m_block + (within - sp * rows_here);
            // column tiles dealt evenly: the first split_rem splits hold one tile more than the others
            n0 = sp * split_base + min(sp, split_rem);
            n1 = n0 + split_base + (sp < split_rem ? 1 : 0);
        } else {
            // column tiles fastest: the CTAs running at the same time share their A slabs (the dZ
            // rows or columns) in L2 instead of each streaming the whole scratch from HBM
            n0 = u % p.n_tiles;
            m = u / p.n_tiles;
            n1 = n0 + 1;
        }
    };

    if (warp == 0) {
        // ---------------- TMA producer (one per CTA) ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            long long pace_due = 0;       // arrivals expected on the counter before this worker goes on
            bool pace_wait = p.pace != nullptr, pace_pending = false;
            int pace_seen = 0;
            int iter = 0;
            for (int u = worker; u < units && ok && !no_k; u += workers, ++iter) {
                int m, n0, n1;
                unit_range(u, m, n0, n1);
                const int with_me = min(workers, units - iter * workers);     // workers that have a unit number `iter`
                long long pos = 0;
                for (int n = n0; n < n1 && ok; ++n) {
                    const int b_row0 = n * BN + rank * C::kBRows;      // this CTA's rows of the B tile
                    for (int kb = 0; kb < k_slabs; ++kb, ++pos) {
                        // the meeting point before a unit: announce the arrival and read the counter; the value
                        // is looked at two k-slabs later, so its round trip to L2 overlaps the issue of those
                        // slabs' loads instead of draining the ring
                        if (p.pace && iter > 0 && pos == 0) {
                            pace_due += with_me;
                            if (rank == 0) asm volatile("red.relaxed.gpu.global.add.s32 [%0], 1;" :: "l"(p.pace) : "memory");
                            if (pace_wait) {
                                asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(pace_seen) : "l"(p.pace) : "memory");
                                pace_pending = true;
                            }
                        }
                        if (pace_pending && pos >= 2) {
                            pace_settle(p.pace, pace_seen, pace_due, pace_wait);
                            pace_pending = false;
                        }
                        if (!mbar_wait(smem_addr(&ctl->empty[stage]), phase ^ 1u, &ctl->abort_flag)) { ok = false; break; }
                        const uint32_t own_bar = smem_addr(&ctl->full[stage]);
                        const uint32_t bar = PAIR ? map_to_cta(own_bar, 0) : own_bar;   // the leader's barrier
                        const uint32_t sa0 = tiles + stage * C::kStageBytes;
                        const uint32_t sb = sa0 + NACC * kABytes;
                        if (!PAIR) mbar_expect_tx(own_bar, C::kStageBytes);
                        else if (rank == 0) mbar_expect_tx(own_bar, 2 * C::kStageBytes);
                        auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
                            if (PAIR) tma_load_2d_pair(dst, map, bar, x, y);
                            else tma_load_2d(dst, map, bar, x, y);
                        };
#pragma unroll
                        for (int a = 0; a < NACC; ++a) {
                            const int my_m = kTilesPerUnit * m + 2 * a + rank;
                            const uint32_t sa = sa0 + a * kABytes;
                            if (p.mode == kGradHidden) {
                                // dZ block (token tile my_m, vocabulary block kb): 128 rows of 128 bytes
                                load(sa, &map_a, 0, (my_m * p.dz_nc + kb) * kDzBlockRows);
                            } else if (p.mode == kGradW) {
                                // dZ^T: vocabulary blocks 2 my_m + j, the 64 token rows of k-slab kb
                                for (int j = 0; j < BM / 64; ++j)
                                    load(sa + j * kSlabBytes, &map_a, 0,
                                         ((kb >> 1) * p.dz_nc + (my_m * 2 + j)) * kDzBlockRows + (kb & 1) * 64);
                            } else {
                                load(sa, &map_a, kb * BK, my_m * BM);
                            }
                        }
                        if (!b_mn) {
                            load(sb, &map_b, kb * BK, b_row0);
                        } else {
                            for (int j = 0; j < C::kBRows / 64; ++j) load(sb + j * kSlabBytes, &map_b, b_row0 + j * 64, kb * BK);
                        }
                        if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (in pair form: the leader CTA only) ----------------
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc(a_mn, b_mn, PAIR ? 2 * BM : BM);
            const uint32_t a_kstep = a_mn ? (16 * 128) >> 4 : 32 >> 4;   // 16 k per instruction, in 16-byte units
            const uint32_t b_kstep = b_mn ? (16 * 128) >> 4 : 32 >> 4;
            int stage = 0;
            uint32_t phase = 0;
            int buf = 0;
            uint32_t tphase[2] = {0, 0};
            bool ok = true;
            for (int u = worker; u < units && ok && !no_k; u += workers) {
                int m, n0, n1;
                unit_range(u, m, n0, n1);
                for (int n = n0; n < n1 && ok; ++n) {
                    if (!mbar_wait(smem_addr(&ctl->tmem_empty[buf]), tphase[buf] ^ 1u, &ctl->abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)buf * BN;
                    for (int kb = 0; kb < k_slabs; ++kb) {
                        if (!mbar_wait(smem_addr(&ctl->full[stage]), phase, &ctl->abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sa = tiles + stage * C::kStageBytes;
                        const uint64_t adesc = smem_desc(sa, a_mn);
                        const uint64_t bdesc = smem_desc(sa + NACC * kABytes, b_mn);
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k) {
                            if (ACC2) {
                                // accumulator a (TMEM columns a * 256 ..) takes A tile a; both share the B slab
#pragma unroll
                                for (int a = 0; a < NACC; ++a)
                                    tc_mma2(tmem_base + (uint32_t)(a * BN),
                                            adesc + (uint64_t)(a * (kABytes >> 4)) + (uint64_t)(k * a_kstep),
                                            bdesc + (uint64_t)(k * b_kstep), idesc, (kb | k) ? 1u : 0u);
                            } else if (PAIR) tc_mma2(d_tmem, adesc + (uint64_t)(k * a_kstep), bdesc + (uint64_t)(k * b_kstep), idesc,
                                                     (kb | k) ? 1u : 0u);
                            else tc_mma(d_tmem, adesc + (uint64_t)(k * a_kstep), bdesc + (uint64_t)(k * b_kstep), idesc,
                                        (kb | k) ? 1u : 0u);
                        }
                        // frees the stage (in both CTAs) when these MMAs retire
                        if (PAIR) tc_commit2(smem_addr(&ctl->empty[stage]));
                        else tc_commit(smem_addr(&ctl->empty[stage]));
                        if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    // accumulator complete (in both CTAs)
                    if (PAIR) tc_commit2(smem_addr(&ctl->tmem_full[buf]));
                    else tc_commit(smem_addr(&ctl->tmem_full[buf]));
                    tphase[buf] ^= 1u;
                    if (!ACC2) buf ^= 1;              // with two accumulators per unit there is one "buffer": both
                }
            }
        }
    } else {
        // ---------------- epilogue: warps 2..5, one accumulator row per thread ----------------
        const int quarter = warp & 3;                    // TMEM lane quarter this warp may read
        const int row_in_tile = quarter * 32 + lane;
        int buf = 0;
        uint32_t tphase[2] = {0, 0};
        bool ok = true;
        for (int u = worker; u < units && ok; u += workers) {
            int m, n0, n1;
            unit_range(u, m, n0, n1);
            const int row = (kTilesPerUnit * m + rank) * BM + row_in_tile;     // accumulator 0's row
            const bool row_ok = row < M;
            float run_m = -INFINITY, run_s = 0.0f;       // kLse
            float run_u = 0.0f;                          // kLse with entropy: sum of 2^x x against run_m
            for (int n = n0; n < n1 && ok; ++n) {
                if (!no_k) {
                    // one lane polls for the warp (128 polling threads would only burn issue slots and
                    // power while the tile is being multiplied); the shuffle hands its result to the others
                    int got = 0;
                    if (lane == 0) got = mbar_wait(smem_addr(&ctl->tmem_full[buf]), tphase[buf], &ctl->abort_flag) ? 1 : 0;
                    got = __shfl_sync(0xffffffffu, got, 0);
                    if (!got) { ok = false; break; }
                    tc_fence_after();
                }
                const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * BN;
                const int col0 = n * BN;
                if (p.mode == kLse && p.dz && p.ref) {
                    // Forward sweep that keeps the tile for the backward, exponentials taken against a
                    // reference rho known BEFORE the sweep (one per row): e = exp(z - rho) is summed for
                    // the log-sum-exp and stored as bf16 in one pass over the accumulator.  bf16 has
                    // fp32's exponent range, so any rho within some tens of the row's log-sum-exp
                    // keeps every entry that matters a normal number at full relative precision, and
                    // dZ = (c_t exp(rho - lse)) e needs only a per-row factor afterwards.  A row whose
                    // reference turns out too far off shows in its sum (inf, or far from one) and
                    // sends its chunk through the per-tile-maximum path instead.
                    const float off = row_ok ? -p.ref[row] * kLog2e : 0.0f;
                    float ts0 = 0.0f, ts1 = 0.0f;
#pragma unroll 1
                    for (int c = 0; c < BN / 32; ++c) {
                        const int cb = col0 + c * 32;
                        const int nvalid = max(0, min(32, p.N - cb));
                        uint32_t o[16];
                        if (nvalid > 0) {                  // warp-uniform: the tensor-memory load is a warp-wide instruction
                            uint32_t v[32];
                            tc_ld32(t_row + (uint32_t)(c * 32), v);
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                float e0 = ex2_approx(fmaf(__uint_as_float(v[2 * i]), kLog2e, off));
                                float e1 = ex2_approx(fmaf(__uint_as_float(v[2 * i + 1]), kLog2e, off));
                                if (2 * i >= nvalid) e0 = 0.0f;
                                if (2 * i + 1 >= nvalid) e1 = 0.0f;
                                ts0 += e0;
                                ts1 += e1;
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[i]) : "f"(e1), "f"(e0));
                            }
                        }
                        if (nvalid <= 0 || !row_ok) {
                            // columns past the vocabulary and rows past the live extent (up to the end of
                            // this pair of token tiles) read as zeros in the gradient contractions
#pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = 0u;
                        }
                        uint4* d4 = reinterpret_cast<uint4*>(p.dz + dz_offset(row, cb, p.dz_nc));
                        d4[0] = make_uint4(o[0], o[1], o[2], o[3]);
                        d4[1] = make_uint4(o[4], o[5], o[6], o[7]);
                        d4[2] = make_uint4(o[8], o[9], o[10], o[11]);
                        d4[3] = make_uint4(o[12], o[13], o[14], o[15]);
                    }
                    run_s += ts0 + ts1;
                    if (row_ok) run_m = p.ref[row];
                } else if (p.mode == kLse && p.dz) {
                    // Forward sweep that keeps the tile for the backward.  Pass 1 over the accumulator:
                    // the row's maximum inside this tile; pass 2: e = exp(z - that maximum), summed for
                    // the log-sum-exp and stored as bf16 (e <= 1: no overflow whatever the logits are;
                    // the relative rounding error is that of a bf16 gradient entry).
                    float tm = -INFINITY;
#pragma unroll 1
                    for (int c = 0; c < BN / 32; ++c) {
                        const int cb = col0 + c * 32;
                        if (cb >= p.N) break;
                        uint32_t v[32];
                        tc_ld32(t_row + (uint32_t)(c * 32), v);
                        const int nvalid = min(32, p.N - cb);
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i < nvalid) tm = fmaxf(tm, __uint_as_float(v[i]));
                    }
                    const float tms = (tm == -INFINITY) ? 0.0f : tm;
                    if (tm > run_m) {
                        run_s *= ex2_approx((run_m - tm) * kLog2e);
                        run_m = tm;
                    }
                    const float off = -tms * kLog2e;
                    float ts0 = 0.0f, ts1 = 0.0f;
#pragma unroll 1
                    for (int c = 0; c < BN / 32; ++c) {
                        // every column block of the tile is written: the scratch covers whole tiles and
                        // the columns past the vocabulary must read as zeros (warp-uniform conditions)
                        const int cb = col0 + c * 32;
                        const int nvalid = max(0, min(32, p.N - cb));
                        uint32_t o[16];
                        if (nvalid > 0) {
                            uint32_t v[32];
                            tc_ld32(t_row + (uint32_t)(c * 32), v);
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                float e0 = ex2_approx(fmaf(__uint_as_float(v[2 * i]), kLog2e, off));
                                float e1 = ex2_approx(fmaf(__uint_as_float(v[2 * i + 1]), kLog2e, off));
                                if (2 * i >= nvalid) e0 = 0.0f;
                                if (2 * i + 1 >= nvalid) e1 = 0.0f;
                                ts0 += e0;
                                ts1 += e1;
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[i]) : "f"(e1), "f"(e0));
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = 0u;
                        }
                        if (row_ok) {
                            uint4* d4 = reinterpret_cast<uint4*>(p.dz + dz_offset(row, cb, p.dz_nc));
                            d4[0] = make_uint4(o[0], o[1], o[2], o[3]);
                            d4[1] = make_uint4(o[4], o[5], o[6], o[7]);
                            d4[2] = make_uint4(o[8], o[9], o[10], o[11]);
                            d4[3] = make_uint4(o[12], o[13], o[14], o[15]);
                        }
                    }
                    if (tm != -INFINITY) run_s += (ts0 + ts1) * ex2_approx((tm - run_m) * kLog2e);
                    if (row_ok) p.tmax[(long long)row * p.n_tiles + n] = tms;
                } else {
                // 32-column chunks of the accumulator(s), software-pipelined: the tensor-memory load of
                // chunk ac + 1 is in flight while chunk ac is consumed (with two accumulators the drain is
                // not hidden behind the next unit's multiplies, so its latency chain matters)
                auto consume = [&](int ac, uint32_t (&v)[32]) {
                    // accumulator a of this unit: the token (vocabulary) tile 2 a further on, TMEM columns a * 256 ..
                    const int a = ac / (BN / 32), c = ac - a * (BN / 32);
                    const int row_a = row + a * 2 * BM;
                    const bool row_ok_a = row_a < M;
                    const int cb = col0 + c * 32;
                    if (cb >= p.N) return;               // whole chunk beyond the valid columns (warp-uniform)
                    if (no_k) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = 0u;
                    }
                    const int nvalid = min(32, p.N - cb);
                    if (p.mode == kLse) {
                        float cm = -INFINITY;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i < nvalid) cm = fmaxf(cm, __uint_as_float(v[i]));
                        if (cm > run_m) {
                            // a larger maximum shifts every exponent so far by dx <= 0:
                            // s -> 2^dx s,  u -> 2^dx (u + dx s)
                            const float dx = (run_m - cm) * kLog2e;       // -inf on the first chunk
                            const float f = ex2_approx(dx);               // exp2(-inf) = 0 on the first chunk
                            if (p.part_u) run_u = (run_m == -INFINITY) ? 0.0f : f * fmaf(dx, run_s, run_u);
                            run_s *= f;
                            run_m = cm;
                        }
                        const float off = -run_m * kLog2e;
                        float s0 = 0.0f, s1 = 0.0f;
                        if (p.part_u) {
                            float u0 = 0.0f, u1 = 0.0f;
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                if (i < nvalid) {
                                    const float x = fmaf(__uint_as_float(v[i]), kLog2e, off), e = ex2_approx(x);
                                    s0 += e;
                                    u0 = fmaf(e, x, u0);
                                }
                                if (i + 1 < nvalid) {
                                    const float x = fmaf(__uint_as_float(v[i + 1]), kLog2e, off), e = ex2_approx(x);
                                    s1 += e;
                                    u1 = fmaf(e, x, u1);
                                }
                            }
                            run_u += u0 + u1;
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                if (i < nvalid) s0 += ex2_approx(fmaf(__uint_as_float(v[i]), kLog2e, off));
                                if (i + 1 < nvalid) s1 += ex2_approx(fmaf(__uint_as_float(v[i + 1]), kLog2e, off));
                            }
                        }
                        run_s += s0 + s1;
                    } else if (p.mode == kGradHidden) {
                        if (row_ok_a) {
                            const long long orow = p.row_index ? (long long)p.row_index[p.live_off + row_a] : (long long)row_a;
                            __nv_bfloat16* dst = p.out_bf16 + orow * p.out_stride + cb;
                            const float sc = p.row_scale ? p.row_scale[row_a] : 1.0f;
                            if (nvalid == 32) {
                                uint32_t o[16];
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[i])
                                        : "f"(__uint_as_float(v[2 * i + 1]) * sc), "f"(__uint_as_float(v[2 * i]) * sc));
                                uint4* d4 = reinterpret_cast<uint4*>(dst);
                                d4[0] = make_uint4(o[0], o[1], o[2], o[3]);
                                d4[1] = make_uint4(o[4], o[5], o[6], o[7]);
                                d4[2] = make_uint4(o[8], o[9], o[10], o[11]);
                                d4[3] = make_uint4(o[12], o[13], o[14], o[15]);
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (i < nvalid) dst[i] = __float2bfloat16_rn(__uint_as_float(v[i]) * sc);
                            }
                        }
                    } else if (ACC2 && nvalid == 32) {   // kGradW, two-accumulator form: the drain is not hidden
                        // One accumulator row per thread means a warp's store touches 32 rows for 16 bytes
                        // each.  The 32 x 32 chunk goes through a padded staging tile in shared memory
                        // instead (rows of 144 bytes: conflict-free both ways), and comes back with eight
                        // lanes along each row, so that a warp's store covers 4 rows x 128 contiguous bytes.
                        float* stg = drain_stage + (warp - 2) * (32 * kDrainPitch);
                        float4* w4 = reinterpret_cast<float4*>(stg + lane * kDrainPitch);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            w4[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                                __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                        __syncwarp();
                        const int piece = lane & 7, rq = lane >> 3;
                        const int row_w0 = row_a - lane;                 // first row of this warp's 32
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const int r = rq + 4 * j;
                            const float4 val = *reinterpret_cast<const float4*>(stg + r * kDrainPitch + piece * 4);
                            if (row_w0 + r < M) {
                                float4* d4 = reinterpret_cast<float4*>(p.out_f32 + (long long)(row_w0 + r) * p.out_stride + cb) + piece;
                                // accumulation is a fire-and-forget vector reduction at the memory side (no
                                // read round trip in the drain); each element gets exactly one addend per
                                // launch, so the result does not depend on timing
                                if (p.accumulate)
                                    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                                                 :: "l"(d4), "f"(val.x), "f"(val.y), "f"(val.z), "f"(val.w) : "memory");
                                else
                                    *d4 = val;
                            }
                        }
                        __syncwarp();                                    // the tile is free for the next chunk
                    } else {   // kGradW
                        if (row_ok_a) {
                            float* dst = p.out_f32 + (long long)row_a * p.out_stride + cb;
                            if (nvalid == 32) {
                                float4* d4 = reinterpret_cast<float4*>(dst);
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    if (p.accumulate)
                                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                                                     :: "l"(d4 + i), "r"(v[4 * i]), "r"(v[4 * i + 1]), "r"(v[4 * i + 2]),
                                                        "r"(v[4 * i + 3]) : "memory");
                                    else
                                        d4[i] = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                                            __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (i < nvalid) dst[i] = __uint_as_float(v[i]) + (p.accumulate ? dst[i] : 0.0f);
                            }
                        }
                    }
                };
                constexpr int kChunks = NACC * (BN / 32);
                const uint32_t t_buf = t_row;
                uint32_t va[32], vb[32];
                if (!no_k) tc_ld32_issue(t_buf, va);
#pragma unroll 1
                for (int ac = 0; ac < kChunks; ac += 2) {
                    if (!no_k) {
                        tc_ld_wait(va);
                        tc_ld32_issue(t_buf + (uint32_t)((ac + 1) * 32), vb);      // kChunks is even
                    }
                    consume(ac, va);
                    if (!no_k) {
                        tc_ld_wait(vb);
                        if (ac + 2 < kChunks) tc_ld32_issue(t_buf + (uint32_t)((ac + 2) * 32), va);
                    }
                    consume(ac + 1, vb);
                }
                }
                // hand the accumulator buffer back to the MMA warp
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && !no_k) {
                    if (PAIR) mbar_arrive_cluster(map_to_cta(smem_addr(&ctl->tmem_empty[buf]), 0));
                    else mbar_arrive(smem_addr(&ctl->tmem_empty[buf]));
                }
                tphase[buf] ^= 1u;
                if (!ACC2) buf ^= 1;
            }
            if (p.mode == kLse && row_ok && ok) {
                // inverse of unit_range's n0(sp)
                const int big = split_rem * (split_base + 1);
                const int sp = n0 < big ? n0 / (split_base + 1) : split_rem + (n0 - big) / max(split_base, 1);
                p.part[(long long)row * p.nsplit + sp] = make_float2(run_m, run_s);
                if (p.part_u) p.part_u[(long long)row * p.nsplit + sp] = run_u;
            }
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (ctl->abort_flag) {
        // copies or MMAs may still be in flight: give them time before the memory is released
        if (threadIdx.x == 0 && p.dev_status) atomicOr(p.dev_status, RLF_DEV_TIMEOUT);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    if (PAIR) pair_sync();        // the peer may still be signalling this CTA's barriers until here
    if (warp == 0) {
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

// ---- small kernels around it ----------------------------------------------------------------
// <h, w> over D bf16 elements by one warp, fp32 accumulation (every lane gets the sum)
__device__ __forceinline__ float warp_dot_bf16(const uint4* __restrict__ h, const uint4* __restrict__ w, int D, int lane) {
    float acc = 0.0f;
    for (int i = lane; i < D / 8; i += 32) {
        const uint4 a = h[i], b = w[i];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc = fmaf(__uint_as_float(aw[k] << 16), __uint_as_float(bw[k] << 16), acc);
            acc = fmaf(__uint_as_float(aw[k] & 0xffff0000u), __uint_as_float(bw[k] & 0xffff0000u), acc);
        }
    }
    return warp_sum(acc);
}

// z_target[t] = <hidden[t, :], W[ids[t], :]> in fp32: one warp per token
__global__ void __launch_bounds__(256)
target_logit_kernel(const __nv_bfloat16* __restrict__ hidden, const __nv_bfloat16* __restrict__ W,
                    const float4* __restrict__ rec, int64_t T, int32_t D, float* __restrict__ zy) {
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const int lane = threadIdx.x & 31;
    const int y = __float_as_int(rec[t].w) & 0x7fffffff;
    const uint4* h = reinterpret_cast<const uint4*>(hidden + t * (int64_t)D);
    const uint4* w = reinterpret_cast<const uint4*>(W + (int64_t)y * D);
    const float acc = warp_dot_bf16(h, w, D, lane);
    if (lane == 0) zy[t] = acc;
}

// One token's row statistics from its per-split (max, sum exp) partials, and its gradient coefficient
// c_t = -(w_t) (dpg/dlogp + beta (1 - exp(ref - logp))), w_t = the token's loss weight.
struct TokenStats {
    float lse, logp, coef;
    bool finite;
};
__device__ __forceinline__ TokenStats token_stats(const float2* __restrict__ parts, int nsplit, float zy, const float4 rec,
                                                  const float* __restrict__ wtok, int64_t t,
                                                  const long long* __restrict__ denom, float eps_clip, float eps_hi,
                                                  float beta) {
    float M = -INFINITY;
    for (int j = 0; j < nsplit; ++j) M = fmaxf(M, parts[j].x);
    float S = 0.0f;
    for (int j = 0; j < nsplit; ++j) {
        const float2 ms = parts[j];
        if (ms.x != -INFINITY) S += ms.y * expf(ms.x - M);
    }
    TokenStats o;
    o.lse = M + logf(S);
    o.logp = (zy - M) - logf(S);
    o.finite = (M > -INFINITY) && (M < INFINITY) && (S > 0.0f) && (S < INFINITY) && (fabsf(o.logp) < INFINITY);
    o.coef = 0.0f;
    if ((__float_as_int(rec.w) < 0) && o.finite) {
        const long long N = *denom;
        const float inv_n = wtok ? wtok[t] : 1.0f / (float)(N > 1 ? N : 1);
        const float A = rec.z;
        const float rho = expf(o.logp - rec.x);
        const bool clipped = ((A > 0.0f) && (rho > 1.0f + eps_hi)) || ((A < 0.0f) && (rho < 1.0f - eps_clip));
        const float dpg = clipped ? 0.0f : -A * rho;
        o.coef = -inv_n * fmaf(beta, -expm1f(rec.y - o.logp), dpg);
    }
    return o;
}

// merge the per-split (max, sum exp) pairs of every token into lse, logp and the gradient coefficient
__global__ void __launch_bounds__(256)
combine_kernel(const float2* __restrict__ part, int nsplit, const float* __restrict__ zy,
               const float4* __restrict__ rec, int64_t T, const long long* __restrict__ denom, float eps_clip,
               float eps_hi, const float* __restrict__ wtok, float beta, float* __restrict__ logp_out,
               float* __restrict__ lse_out, float* __restrict__ coef_out, int32_t* __restrict__ dev_status) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const TokenStats ts = token_stats(part + t * nsplit, nsplit, zy[t], rec[t], wtok, t, denom, eps_clip, eps_hi, beta);
    logp_out[t] = ts.finite ? ts.logp : __int_as_float(0x7fc00000);
    lse_out[t] = ts.finite ? ts.lse : 0.0f;
    coef_out[t] = ts.coef;
    if (!ts.finite && dev_status) atomicOr(dev_status, RLF_DEV_NONFINITE);
}

// forward-only pass from target ids alone: z_target per token (NaN and a status bit for an id outside
// the vocabulary), one warp per token
__global__ void __launch_bounds__(256)
target_logit_ids_kernel(const __nv_bfloat16* __restrict__ hidden, const __nv_bfloat16* __restrict__ W,
                        const int32_t* __restrict__ ids, int64_t T, int32_t D, int32_t V, float* __restrict__ zy,
                        int32_t* __restrict__ dev_status) {
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const int lane = threadIdx.x & 31;
    const int y = ids[t];
    if (y < 0 || y >= V) {
        if (lane == 0) {
            zy[t] = __int_as_float(0x7fc00000);
            if (dev_status) atomicOr(dev_status, RLF_DEV_BAD_TARGET);
        }
        return;
    }
    const uint4* h = reinterpret_cast<const uint4*>(hidden + t * (int64_t)D);
    const uint4* w = reinterpret_cast<const uint4*>(W + (int64_t)y * D);
    const float acc = warp_dot_bf16(h, w, D, lane);
    if (lane == 0) zy[t] = acc;
}

// merge the per-split (max, s, u) triples of every token: logp = z_y - lse, H = ln S - ln2 U / S with
// S = sum_k s_k 2^dx_k, U = sum_k 2^dx_k (u_k + s_k dx_k), dx_k the split's base against the row maximum
__global__ void __launch_bounds__(256)
combine_logp_entropy_kernel(const float2* __restrict__ part, const float* __restrict__ part_u, int nsplit,
                            const float* __restrict__ zy, int64_t T, float* __restrict__ logp_out,
                            float* __restrict__ entropy_out, int32_t* __restrict__ dev_status) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    float M = -INFINITY;
    for (int j = 0; j < nsplit; ++j) M = fmaxf(M, part[t * nsplit + j].x);
    float S = 0.0f, U = 0.0f;
    for (int j = 0; j < nsplit; ++j) {
        const float2 ms = part[t * nsplit + j];
        if (ms.x == -INFINITY) continue;
        const float dx = (ms.x - M) * kLog2e;
        const float f = exp2f(dx);
        S += ms.y * f;
        if (part_u && f > 0.0f) U += f * fmaf(ms.y, dx, part_u[t * nsplit + j]);
    }
    const float lnS = logf(S);
    const float logp = (zy[t] - M) - lnS;
    const bool finite = (M > -INFINITY) && (M < INFINITY) && (S > 0.0f) && (S < INFINITY);
    const float nan = __int_as_float(0x7fc00000);
    logp_out[t] = (finite && fabsf(logp) < INFINITY) ? logp : nan;      // NaN z_y (bad target id) stays NaN
    if (entropy_out) entropy_out[t] = finite ? lnS - kLn2 * U / S : nan;
    if (!finite && dev_status) atomicOr(dev_status, RLF_DEV_NONFINITE);
}

// Masked rows contribute nothing to either gradient, so the backward (and the part of the forward
// that keeps logits for it) runs over the unmasked rows only.  Stable partition of the tokens by
// the live bit of their record (token order is kept inside each part, so results do not depend on
// timing): one CTA scans the T flags.  counts[0] = live rows, counts[1] = the others.
__global__ void __launch_bounds__(1024)
partition_rows_kernel(const float4* __restrict__ rec, int T, int32_t* __restrict__ idx_live,
                      int32_t* __restrict__ idx_dead, int* __restrict__ counts) {
    __shared__ int warp_tot[32];
    __shared__ int base_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) base_s = 0;
    __syncthreads();
    for (int t0 = 0; t0 < T; t0 += 1024) {
        const int t = t0 + tid;
        const bool live = t < T && __float_as_int(rec[t].w) < 0;
        const unsigned bal = __ballot_sync(0xffffffffu, live);
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < 32; ++w) {
            const int c = warp_tot[w];
            if (w < warp) before += c;
            total += c;
        }
        const int base = base_s;
        const int live_before = base + before + __popc(bal & ((1u << lane) - 1u));
        if (live) idx_live[live_before] = t;
        else if (t < T) idx_dead[t - live_before] = t;
        __syncthreads();
        if (tid == 0) base_s = base + total;
    }
    __syncthreads();
    if (tid == 0) { counts[0] = base_s; counts[1] = T - base_s; }
}

// out row r <- hidden row idx[r] for r < *count; rows up to the next multiple of 256 are zero-filled
// (the contractions read whole tiles)
// ref_out (optional): the reference of row r's stored exponentials, its target logit plus kRefShift
constexpr float kRefShift = 32.0f;
__global__ void __launch_bounds__(128)
gather_rows_kernel(const __nv_bfloat16* __restrict__ hidden, int D, const int32_t* __restrict__ idx,
                   const int* __restrict__ count, __nv_bfloat16* __restrict__ out, const float* __restrict__ zy,
                   float* __restrict__ ref_out) {
    const int n = *count;
    const int r = blockIdx.x;
    if (r >= ((n + 255) & ~255)) return;
    if (ref_out && threadIdx.x == 0) ref_out[r] = r < n ? zy[idx[r]] + kRefShift : 0.0f;
    uint4* dst = reinterpret_cast<uint4*>(out + (long long)r * D);
    const int nv = D / 8;
    if (r < n) {
        const uint4* src = reinterpret_cast<const uint4*>(hidden + (long long)idx[r] * D);
        for (int i = threadIdx.x; i < nv; i += blockDim.x) dst[i] = src[i];
    } else {
        for (int i = threadIdx.x; i < nv; i += blockDim.x) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    }
}

// skip-masked form: the rows without loss weight are not multiplied at all; their log-prob reads NaN
__global__ void __launch_bounds__(256)
fill_nan_rows_kernel(const int32_t* __restrict__ idx, const int* __restrict__ count, float* __restrict__ logp_out) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < *count) logp_out[idx[r]] = __int_as_float(0x7fc00000);
}

// combine_kernel for a launch over gathered rows: row r of the launch (partials part[r][.]) is token
// idx[off + r]; logp goes to the token's place, lse / coefficient / target id to the gathered place.
//
// With ref_g (the sweep stored e = exp(z - rho_r), rho_r = ref_g[off + r]) the kernel also finishes the
// row for the gradient contractions: scale_g = c_t exp(rho - lse), the per-row factor that turns the
// stored exponentials into dZ, and the target column of the scratch is overwritten with
// (p_y - 1) exp(lse - rho) (formed in fp32 from the fp32 target logit), so that factor x entry is
// c_t (p_y - 1) to bf16 rounding even when p_y is close to one.  The reference is usable while the
// factor and the entries stay normal numbers: a row with a non-finite sum or lse - rho above
// kRefWindow raises *fallback instead of a status bit, and the chunk is redone with per-tile maxima.
// Without ref_g, scale_g (if given) is set to one: the scratch will hold dZ itself.
constexpr float kRefWindow = 46.0f;
__global__ void __launch_bounds__(256)
combine_rows_kernel(const float2* __restrict__ part, int nsplit, int rows_max, const int32_t* __restrict__ idx,
                    const int* __restrict__ count, int off, const float* __restrict__ zy,
                    const float4* __restrict__ rec, const long long* __restrict__ denom, float eps_clip, float eps_hi,
                    const float* __restrict__ wtok, float beta, float* __restrict__ logp_out, float* __restrict__ lse_g,
                    float* __restrict__ coef_g, int32_t* __restrict__ y_g, int32_t* __restrict__ dev_status,
                    const float* __restrict__ ref_g, float* __restrict__ scale_g, __nv_bfloat16* __restrict__ dz,
                    int dz_nc, int V, int* __restrict__ fallback, const int* __restrict__ run_flag, int run_want) {
    if (run_flag && *run_flag != run_want) return;
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    const int n = max(0, min(*count - off, rows_max));
    if (r >= n) return;
    const int t = idx[off + r];
    const float4 rc = rec[t];
    const TokenStats ts = token_stats(part + (long long)r * nsplit, nsplit, zy[t], rc, wtok, t, denom, eps_clip, eps_hi,
                                      beta);
    logp_out[t] = ts.finite ? ts.logp : __int_as_float(0x7fc00000);
    const int y = __float_as_int(rc.w) & 0x7fffffff;
    if (lse_g) {
        lse_g[off + r] = ts.finite ? ts.lse : 0.0f;
        coef_g[off + r] = ts.coef;
        y_g[off + r] = y;
    }
    if (ref_g) {
        const float rho = ref_g[off + r];
        const bool usable = ts.finite && (ts.lse - rho <= kRefWindow);
        if (!usable) {
            atomicOr(fallback, 1);
            scale_g[off + r] = 0.0f;
            return;
        }
        scale_g[off + r] = ts.coef * expf(rho - ts.lse);
        if (ts.coef != 0.0f && y < V) dz[dz_offset(r, y, dz_nc)] = __float2bfloat16_rn(expm1f(ts.logp) * expf(ts.lse - rho));
        return;
    }
    if (scale_g) scale_g[off + r] = 1.0f;
    if (!ts.finite && dev_status) atomicOr(dev_status, RLF_DEV_NONFINITE);
}

// Hs[r, :] = bf16(scale[off + r] * Hl[r, :]) for the rows of one chunk: the token-side operand of
// grad_W = e^T (scale H) when the scratch holds exponentials against a per-row reference.  Rows from
// the live extent up to the next multiple of 256 become zeros.
__global__ void __launch_bounds__(128)
scale_rows_kernel(const __nv_bfloat16* __restrict__ Hl, int D, int rows_max, const int* __restrict__ count, int off,
                  const float* __restrict__ scale_g, __nv_bfloat16* __restrict__ Hs) {
    const int n = max(0, min(*count - off, rows_max));
    const int r = blockIdx.x;
    if (r >= ((n + 255) & ~255)) return;
    uint4* dst = reinterpret_cast<uint4*>(Hs + (long long)r * D);
    const int nv = D / 8;
    if (r >= n) {
        for (int i = threadIdx.x; i < nv; i += blockDim.x) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    const float f = scale_g[off + r];
    const uint4* src = reinterpret_cast<const uint4*>(Hl + (long long)r * D);
    for (int i = threadIdx.x; i < nv; i += blockDim.x) {
        const uint4 z = src[i];
        const uint32_t w[4] = {z.x, z.y, z.z, z.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[k])
                : "f"(__uint_as_float(w[k] & 0xffff0000u) * f), "f"(__uint_as_float(w[k] << 16) * f));
        dst[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// in place over one chunk of stored exponentials e = exp(z - tile max): dZ = coef (e exp(tile max - lse)
// - [v == y]) as bf16; the target column takes the fp32 target logit.  Rows from the live extent up
// to the next multiple of 256 become zeros.  A work item is one (token tile, 256-column tile): four adjacent
// blocks of the scratch, 64 KB of contiguous memory; the CTAs stride over the items (the launch is
// usually one that a device flag turns into a no-op, which a small grid makes cheap).
__global__ void __launch_bounds__(256)
dz_from_e_kernel(__nv_bfloat16* __restrict__ ebuf, int V, int n_tiles, const float* __restrict__ tmax, int rows_max,
                 const int* __restrict__ count, int off, const float* __restrict__ lse_g,
                 const float* __restrict__ coef_g, const int32_t* __restrict__ y_g, const int32_t* __restrict__ idx,
                 const float* __restrict__ zy, const int* __restrict__ run_flag, int run_want) {
    __shared__ float f_s[kDzBlockRows];          // signed scale of each row for this column tile
    if (run_flag && *run_flag != run_want) return;
    __shared__ int live_s[kDzBlockRows];
    const int n = max(0, min(*count - off, rows_max));
    const int nc = 4 * n_tiles;
    const long long items = (long long)(((n + 255) & ~255) / kDzBlockRows) * n_tiles;
    for (long long item = blockIdx.x; item < items; item += gridDim.x) {
    const int tt = (int)(item / n_tiles), jt = (int)(item - (long long)tt * n_tiles);
    __syncthreads();                             // the previous item's readers of f_s / live_s are done
    if (threadIdx.x < kDzBlockRows) {
        const int r = tt * kDzBlockRows + threadIdx.x;
        const float coef = r < n ? coef_g[off + r] : 0.0f;
        float f = 0.0f;
        if (coef != 0.0f) {
            const float c2 = lg2_approx(fabsf(coef)) - lse_g[off + r] * kLog2e;
            f = copysignf(ex2_approx(fmaf(tmax[(long long)r * n_tiles + jt], kLog2e, c2)), coef);
        }
        f_s[threadIdx.x] = f;
        live_s[threadIdx.x] = coef != 0.0f;
    }
    __syncthreads();
    uint4* base = reinterpret_cast<uint4*>(ebuf + dz_offset((long long)tt * kDzBlockRows, jt * BN, nc));
    // 4 blocks x 128 rows x 8 vectors of 16 bytes
    for (int i = threadIdx.x; i < 4 * kDzBlockRows * 8; i += 256) {
        const int rr = (i >> 3) & (kDzBlockRows - 1);
        if (!live_s[rr]) {
            base[i] = make_uint4(0u, 0u, 0u, 0u);
            continue;
        }
        const float f = f_s[rr];
        const uint4 z = base[i];
        const uint32_t w[4] = {z.x, z.y, z.z, z.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(o[k])
                : "f"(__uint_as_float(w[k] & 0xffff0000u) * f), "f"(__uint_as_float(w[k] << 16) * f));
        base[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
    __syncthreads();
    if (threadIdx.x < kDzBlockRows && live_s[threadIdx.x]) {
        const int r = tt * kDzBlockRows + threadIdx.x;
        const int y = y_g[off + r];
        if (y >= jt * BN && y < jt * BN + BN && y < V) {
            const float coef = coef_g[off + r];
            const float py = ex2_approx((zy[idx[off + r]] - lse_g[off + r]) * kLog2e);
            ebuf[dz_offset(r, y, nc)] = __float2bfloat16_rn(fmaf(coef, py, -coef));
        }
    }
    }
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static std::mutex mu;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 row-major matrix [rows][cols] (cols contiguous); box = box_cols x box_rows, 128-byte swizzle
static bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_elems,
                     uint32_t box_cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_elems * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int sm_count_lm() {
    int dev = 0, v = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    return v > 0 ? v : 148;
}

static std::atomic<int> g_pair{1};       // 1: cta_group::2 pair form, 0: single-CTA form
static std::atomic<int> g_m_block{0};    // row units per scheduling block of the sweep; 0: automatic
static std::atomic<int> g_max_workers{0};   // persistent CTAs (or pairs) per launch; 0: one per SM (pair of SMs)
static std::atomic<int> g_chunk_tiles{0};   // token tiles per backward chunk; 0: the most the workspace holds
static std::atomic<int> g_pace{1};          // pacing of the workers' loads (see GemmParams::pace): 1 on, 0 off
static std::atomic<int> g_row_ref{1};       // backward scratch: 1 exponentials against a per-row reference, 0 per-tile maxima

template <bool PAIR, bool ACC2>
static rlf_status launch_gemm_t(const CUtensorMap& ma, const CUtensorMap& mb, const GemmParams& p, cudaStream_t s) {
    static std::mutex mu;
    static bool opted[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (dev >= 0 && dev < 64 && !opted[dev]) {
            if (cudaFuncSetAttribute((const void*)umma_gemm_kernel<PAIR, ACC2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg<PAIR, ACC2>::kSmemBytes) != cudaSuccess) {
                cudaGetLastError();
                return RLF_ERR_CUDA;
            }
            opted[dev] = true;
        }
    }
    const bool sweep = p.mode == kLse;
    constexpr int kTilesPerUnit = (PAIR ? 2 : 1) * (ACC2 ? 2 : 1);
    const int m_units = (p.m_tiles + kTilesPerUnit - 1) / kTilesPerUnit;
    const int units = sweep ? m_units * p.nsplit : m_units * p.n_tiles;
    if (units <= 0) return RLF_OK;
    int workers = PAIR ? sm_count_lm() / 2 : sm_count_lm();
    // Sweep schedule: the CTAs (or pairs) running at one time cover m_block row units x (workers / m_block)
    // splits, in lockstep.  Their token tiles (256 x D bf16 per pair: 1.3 MB at D = 2560, 2 MB at 4096)
    // are re-read for every column tile and must stay in L2 next to the streaming head: with all 74 pairs
    // on different row units (97 MB at D = 2560) they did not, and the same launch drew its 1 kW at
    // 1.06 GHz instead of 1.39 GHz.  So m_block is what keeps about 48 MB of token tiles live, at most half
    // the workers, and a divisor of the worker count (blocks that leave the splits misaligned cost
    // 4 - 10 %): when no nearby divisor exists a few workers are left out instead (D = 4096: 24 row
    // units on 72 of the 74 pairs measured 5 % faster than 37 on 74; D = 2560 keeps 37 on 74).
    if (g_max_workers.load() > 0 && g_max_workers.load() < workers) workers = g_max_workers.load();
    GemmParams q = p;
    q.m_block = workers / 2 > 0 ? workers / 2 : 1;
    if (sweep && g_m_block.load() == 0 && g_max_workers.load() == 0) {
        const double unit_bytes = (double)(PAIR ? 2 : 1) * BM * (double)p.k_slabs * BK * 2.0;
        const double target = 48.0 * 1024 * 1024 / unit_bytes;
        int hi = (int)(target * 1.05);
        if (hi > workers / 2) hi = workers / 2;
        if (hi < 1) hi = 1;
        int lo = (int)(target * 0.6);
        if (lo < 1) lo = 1;
        int best_mb = hi, best_w = workers / hi * hi;
        for (int mb = hi - 1; mb >= lo; --mb) {
            const int w = workers / mb * mb;
            if (w > best_w) { best_w = w; best_mb = mb; }
        }
        q.m_block = best_mb;
        workers = best_w;
    }
    if (g_m_block.load() > 0) q.m_block = g_m_block.load();
    if (workers > units) workers = units;
    // Pacing, measured at full size with one-pass ncu counts: grad_hidden 32 -> 10 GB of HBM reads and
    // 9.6 -> 8.5 ms per launch, grad_W 35 -> 11 GB and 10.3 -> 9.1 ms (D = 2560); the sweep at D = 4096
    // 71 -> 61 ms.  Meeting points inside a unit were tried too and cost more than they return.
    if (q.pace && g_pace.load() != 0) {
        if (cudaMemsetAsync(q.pace, 0, sizeof(int), s) != cudaSuccess) return RLF_ERR_CUDA;
    } else {
        q.pace = nullptr;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(PAIR ? 2 * workers : workers);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Cfg<PAIR, ACC2>::kSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = PAIR ? 2 : 1;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, umma_gemm_kernel<PAIR, ACC2>, ma, mb, q) != cudaSuccess) {
        cudaGetLastError();
        return RLF_ERR_CUDA;
    }
    count_launch();
    return RLF_OK;
}

static std::atomic<int> g_acc2{1};          // gradient contractions in pair form: 1 two accumulators per CTA, 0 one
static rlf_status launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const GemmParams& p, bool pair,
                              cudaStream_t s) {
    if (!pair) return launch_gemm_t<false, false>(ma, mb, p, s);
    if (p.mode != kLse && g_acc2.load() != 0) return launch_gemm_t<true, true>(ma, mb, p, s);
    return launch_gemm_t<true, false>(ma, mb, p, s);
}

// Rows of dZ held in scratch at a time: up to 148 token tiles = 37 units of the two-accumulator
// gradient contractions (37 x D/256 = 370 units at D = 2560: five whole waves on 74 CTA pairs) = two
// scheduling blocks of the sweep; 5.8 GB at V = 151936.  Larger chunks mean fewer passes over the head
// in grad_hidden and fewer accumulations into grad_W.
constexpr int kChunkTokens = 148 * BM;
constexpr int kMaxSplit = 64;               // most vocabulary splits a sweep may use (sizes the partials)

// Number of vocabulary splits of a sweep.  A work unit is (pair of token tiles, split); the units are
// dealt round-robin to the persistent CTAs, which keep their load / multiply / drain pipelines
// running across units, so small units cost nothing, while large ones leave a ragged last wave
// (the number of rows that take part is only known on the device).  Splits of at least 8 column
// tiles, at most kMaxSplit of them; concurrently running CTAs still work on the same few splits, so
// the head's rows are shared in L2.
static int pick_split(int n_tiles) {
    int per = (n_tiles + kMaxSplit - 1) / kMaxSplit;
    if (per < 8) per = 8;
    return (n_tiles + per - 1) / per;
}

struct LmWs {
    size_t n_count, partial, rec, zy, lse, coef, wtok, seqcnt, part, idx_live, idx_dead, lse_g, coef_g, y_g, ref_g, scale_g,
        hidden_g, hidden_s, tmax, dz, total;
};
static size_t up1k(size_t x) { return (x + 1023) & ~(size_t)1023; }
static LmWs lm_workspace(int64_t T, int32_t V, int32_t D) {
    LmWs w;
    size_t o = 0;
    const size_t Tn = (size_t)(T > 0 ? T : 0);
    const size_t Tp = (Tn + 255) & ~(size_t)255;     // compact arrays are padded to whole tile pairs
    w.n_count = o; o += 1024;                        // [0] mask count, [64] live / other row counts, [128] chunk flag, [256] pacing counter
    w.partial = o; o += up1k(token_loss_partial_bytes());
    w.rec = o;     o += up1k(16 * Tn);
    w.zy = o;      o += up1k(4 * Tn);
    w.lse = o;     o += up1k(4 * Tn);
    w.coef = o;    o += up1k(4 * Tn);
    w.wtok = o;    o += up1k(4 * Tn);                // sequence-mean aggregation: per-token weights
    w.seqcnt = o;  o += up1k(4 * (Tn + 1));          //   and unmasked tokens per response (B <= T + 1)
    w.part = o;    o += up1k(8 * Tn * kMaxSplit);
    w.idx_live = o; o += up1k(4 * Tp);
    w.idx_dead = o; o += up1k(4 * Tp);
    w.lse_g = o;   o += up1k(4 * Tp);
    w.coef_g = o;  o += up1k(4 * Tp);
    w.y_g = o;     o += up1k(4 * Tp);
    w.ref_g = o;   o += up1k(4 * Tp);                // per-row reference of the stored exponentials
    w.scale_g = o; o += up1k(4 * Tp);                // per-row factor exponentials -> dZ
    w.hidden_g = o; o += 2 * up1k(Tp * (size_t)(D > 0 ? D : 0) * 2);   // live rows, then the others
    const size_t chunk = Tp < (size_t)kChunkTokens ? Tp : (size_t)kChunkTokens;
    w.hidden_s = o; o += up1k(chunk * (size_t)(D > 0 ? D : 0) * 2);    // one chunk of live rows times their factors
    w.tmax = o;    o += up1k(4 * chunk * (size_t)((V + BN - 1) / BN));
    w.dz = o;
    o += up1k(chunk * (size_t)((V + BN - 1) / BN) * BN * 2);     // blocked: whole 256-column tiles
    w.total = o + 1024;
    return w;
}

}  // namespace lm

size_t lmhead_logp_workspace_bytes(int64_t T) {
    const size_t Tn = (size_t)(T > 0 ? T : 0);
    return 1024 + lm::up1k(4 * Tn) + lm::up1k(8 * Tn * lm::kMaxSplit) + lm::up1k(4 * Tn * lm::kMaxSplit) + 1024;
}

size_t lmhead_workspace_bytes(int64_t T, int32_t V, int32_t D) {
    if (V < 1 || D < 1) return 0;
    return lm::lm_workspace(T, V, D).total;
}

}  // namespace rlf

namespace rlf {
namespace lm {

// eps_clip is the lower clip width, eps_hi the upper one; aggregation 0 = token mean (denom counts
// tokens), 1 = sequence mean (denom counts responses); skip_masked: rows without loss weight are not
// multiplied at all and their log-prob reads NaN
static rlf_status fused_lmhead_impl(const void* hidden, const void* W, int64_t T, int32_t D, int32_t V,
                                    const int32_t* ids, const int32_t* seq_id, const float* adv, int32_t B,
                                    const float* old_logp, const float* ref_logp, const uint8_t* mask,
                                    float eps_clip, float eps_hi, float beta_kl, int aggregation, int skip_masked,
                                    const int64_t* denom, float* logp_out,
                                    double* loss_out, void* grad_hidden, float* grad_W,
                                    int accumulate_grad_W, void* workspace, size_t workspace_bytes,
                                    int32_t* dev_status, rlf_stream_t stream) {
    if (T < 0 || V < 1 || D < 1 || B < 0) return RLF_ERR_SHAPE;
    if (aggregation != 0 && aggregation != 1) return RLF_ERR_SHAPE;
    if (aggregation == 1 && (int64_t)B > T + 1) return RLF_ERR_SHAPE;
    if (D % 64 != 0 || V % 8 != 0) return RLF_ERR_SHAPE;
    if (T >= (1ll << 30)) return RLF_ERR_UNSUPPORTED;
    if (!loss_out) return RLF_ERR_NULL;
    if (T > 0 && (!hidden || !W || !ids || !seq_id || !adv || !old_logp || !ref_logp || !mask || !logp_out))
        return RLF_ERR_NULL;
    if (T > 0 && B == 0) return RLF_ERR_SHAPE;
    if (!aligned(hidden, 16) || !aligned(W, 16) || !aligned(grad_hidden, 16) || !aligned(grad_W, 16))
        return RLF_ERR_ALIGN;
    const LmWs w = lm_workspace(T, V, D);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < w.total) return RLF_ERR_WORKSPACE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    // 1 KB alignment of the scratch pieces that TMA reads
    char* ws = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(workspace) + 1023) & ~(uintptr_t)1023);
    long long* n_count = reinterpret_cast<long long*>(ws + w.n_count);
    double* partial = reinterpret_cast<double*>(ws + w.partial);
    float4* rec = reinterpret_cast<float4*>(ws + w.rec);
    float* zy = reinterpret_cast<float*>(ws + w.zy);
    float* lse = reinterpret_cast<float*>(ws + w.lse);
    float* coef = reinterpret_cast<float*>(ws + w.coef);
    float2* part = reinterpret_cast<float2*>(ws + w.part);
    __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(ws + w.dz);
    const __nv_bfloat16* H = static_cast<const __nv_bfloat16*>(hidden);
    const __nv_bfloat16* Wm = static_cast<const __nv_bfloat16*>(W);

    // token mean: dn is the token count (given, or counted by the record kernel); sequence mean: the
    // per-token weights carry the whole normalisation and dn is only a valid address to read
    const long long* dn = aggregation == 0 ? reinterpret_cast<const long long*>(denom) : nullptr;
    const bool count_here = dn == nullptr;
    if (count_here) {
        if (cudaMemsetAsync(n_count, 0, sizeof(long long), s) != cudaSuccess) return RLF_ERR_CUDA;
        dn = n_count;
    }
    float* wtok = nullptr;
    auto token_loss = [&](int64_t rows) {
        return launch_token_loss_w(logp_out, rec, rows, eps_clip, eps_hi, beta_kl, wtok, partial, dn, loss_out, s);
    };
    if (T == 0) return token_loss(0);

    st = launch_token_prep(ids, seq_id, adv, old_logp, ref_logp, mask, T, V, B, rec, count_here ? n_count : nullptr,
                           dev_status, s);
    if (st != RLF_OK) return st;
    if (aggregation == 1) {
        wtok = reinterpret_cast<float*>(ws + w.wtok);
        st = launch_seq_weights(rec, seq_id, T, B, reinterpret_cast<const long long*>(denom),
                                reinterpret_cast<int*>(ws + w.seqcnt), n_count + 4, wtok, s);
        if (st != RLF_OK) return st;
    }
    target_logit_kernel<<<(unsigned)((T + 7) / 8), 256, 0, s>>>(H, Wm, rec, T, D, zy);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;

    const bool pair = g_pair.load() != 0;
    const uint32_t b_rows = pair ? BN / 2 : BN;       // rows of a K-major B tile that one CTA stages
    CUtensorMap mapW;
    if (!make_map(&mapW, Wm, (uint64_t)V, (uint64_t)D, (uint64_t)D, BK, b_rows)) return RLF_ERR_CUDA;
    GemmParams g = {};
    g.mode = kLse;
    g.N = V;
    g.n_tiles = (V + BN - 1) / BN;
    g.k_slabs = D / BK;
    g.part = part;
    g.dev_status = dev_status;
    g.pace = reinterpret_cast<int*>(ws + w.n_count + 256);
    auto set_rows = [&](GemmParams& q, int64_t rows) {
        q.M = (int)rows;
        q.m_tiles = (int)((rows + BM - 1) / BM);
        q.nsplit = pick_split(q.n_tiles);
        q.n_tiles_per_split = (q.n_tiles + q.nsplit - 1) / q.nsplit;
    };

    if (!grad_hidden && !grad_W && !skip_masked) {
        // forward only: one sweep over all rows, running (max, sum exp) per token and vocabulary split
        CUtensorMap mapH;
        if (!make_map(&mapH, H, (uint64_t)T, (uint64_t)D, (uint64_t)D, BK, BM)) return RLF_ERR_CUDA;
        set_rows(g, T);
        st = launch_gemm(mapH, mapW, g, pair, s);
        if (st != RLF_OK) return st;
        combine_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(part, g.nsplit, zy, rec, T, dn, eps_clip, eps_hi, wtok,
                                                                    beta_kl, logp_out, lse, coef, dev_status);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
        return token_loss(T);
    }

    // forward + backward.  The tokens are partitioned (stably) into unmasked rows and the others;
    // their numbers stay on the device (no host sync), so every chunk is launched and the kernels
    // size themselves.  Unmasked rows, by chunks: forward sweep that also keeps the chunk's
    // exponentials (relative to tile maxima) as bf16 -> lse, logp, coefficient -> dZ in place -> grad_hidden rows, grad_W += chunk's part.
    // The other rows only need their log-prob: one forward sweep.
    int* counts = reinterpret_cast<int*>(ws + w.n_count + 64);
    int32_t* idx_live = reinterpret_cast<int32_t*>(ws + w.idx_live);
    int32_t* idx_dead = reinterpret_cast<int32_t*>(ws + w.idx_dead);
    float* lse_g = reinterpret_cast<float*>(ws + w.lse_g);
    float* coef_g = reinterpret_cast<float*>(ws + w.coef_g);
    int32_t* y_g = reinterpret_cast<int32_t*>(ws + w.y_g);
    const int64_t Tp = (T + 255) & ~(int64_t)255;
    __nv_bfloat16* Hl = reinterpret_cast<__nv_bfloat16*>(ws + w.hidden_g);
    __nv_bfloat16* Hd = reinterpret_cast<__nv_bfloat16*>(ws + w.hidden_g + up1k((size_t)Tp * D * 2));
    const bool bwd = grad_hidden || grad_W;
    // backward scratch: exponentials against a per-row reference (no rescaling pass; the per-tile-maximum
    // path stays queued behind a device flag for chunks whose reference turns out unusable), or the
    // per-tile-maximum path alone
    const bool row_ref = bwd && g_row_ref.load() != 0;
    float* ref_g = reinterpret_cast<float*>(ws + w.ref_g);
    float* scale_g = reinterpret_cast<float*>(ws + w.scale_g);
    __nv_bfloat16* Hs = reinterpret_cast<__nv_bfloat16*>(ws + w.hidden_s);
    int* chunk_flag = reinterpret_cast<int*>(ws + w.n_count + 128);
    partition_rows_kernel<<<1, 1024, 0, s>>>(rec, (int)T, idx_live, idx_dead, counts);
    gather_rows_kernel<<<(unsigned)Tp, 128, 0, s>>>(H, D, idx_live, counts, Hl, zy, row_ref ? ref_g : nullptr);
    if (!skip_masked) gather_rows_kernel<<<(unsigned)Tp, 128, 0, s>>>(H, D, idx_dead, counts + 1, Hd, nullptr, nullptr);
    count_launch(skip_masked ? 2 : 3);
    if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    if (grad_hidden && cudaMemsetAsync(grad_hidden, 0, (size_t)T * D * 2, s) != cudaSuccess) return RLF_ERR_CUDA;

    const int tuned_tiles = g_chunk_tiles.load();
    const int64_t chunk_tokens = (tuned_tiles > 0 && tuned_tiles * BM < kChunkTokens) ? tuned_tiles * BM : kChunkTokens;
    for (int64_t t0 = 0; t0 < T; t0 += chunk_tokens) {
        const int64_t tc = (T - t0) < chunk_tokens ? (T - t0) : chunk_tokens;
        CUtensorMap mapHc;
        if (!make_map(&mapHc, Hl + t0 * D, (uint64_t)tc, (uint64_t)D, (uint64_t)D, BK, BM)) return RLF_ERR_CUDA;
        GemmParams z = g;
        set_rows(z, tc);
        if (bwd) {
            z.dz = dz;
            z.dz_nc = 4 * z.n_tiles;
            z.tmax = reinterpret_cast<float*>(ws + w.tmax);
        }
        z.live_count = counts;
        z.live_off = (int)t0;
        auto combine = [&](bool with_ref, const int* run_flag) {
            combine_rows_kernel<<<(unsigned)((tc + 255) / 256), 256, 0, s>>>(
                part, z.nsplit, (int)tc, idx_live, counts, (int)t0, zy, rec, dn, eps_clip, eps_hi, wtok, beta_kl, logp_out,
                lse_g, coef_g, y_g, dev_status, with_ref ? ref_g : nullptr, row_ref ? scale_g : nullptr, dz, z.dz_nc, V,
                chunk_flag, run_flag, 1);
            count_launch();
        };
        const int64_t tcp = (tc + 255) & ~(int64_t)255;
        auto dz_pass = [&](const int* run_flag) {
            const long long dz_items = (tcp / kDzBlockRows) * (long long)z.n_tiles;
            dz_from_e_kernel<<<(unsigned)(dz_items < 148 * 8 ? dz_items : 148 * 8), 256, 0, s>>>(
                dz, V, z.n_tiles, z.tmax, (int)tc, counts, (int)t0, lse_g, coef_g, y_g, idx_live, zy, run_flag, 1);
            count_launch();
        };
        if (row_ref) {
            if (cudaMemsetAsync(chunk_flag, 0, sizeof(int), s) != cudaSuccess) return RLF_ERR_CUDA;
            z.ref = ref_g + t0;
            st = launch_gemm(mapHc, mapW, z, pair, s);
            if (st != RLF_OK) return st;
            combine(true, nullptr);
            // queued always, run only if some row of the chunk raised the flag: the chunk again with
            // per-tile maxima, rescaled in place into dZ (every row's factor becomes one)
            GemmParams zf = z;
            zf.ref = nullptr;
            zf.run_flag = chunk_flag;
            zf.run_want = 1;
            st = launch_gemm(mapHc, mapW, zf, pair, s);
            if (st != RLF_OK) return st;
            combine(false, chunk_flag);
            dz_pass(chunk_flag);
            scale_rows_kernel<<<(unsigned)tcp, 128, 0, s>>>(Hl + t0 * D, D, (int)tc, counts, (int)t0, scale_g, Hs);
            count_launch();
        } else {
            st = launch_gemm(mapHc, mapW, z, pair, s);
            if (st != RLF_OK) return st;
            combine(false, nullptr);
            if (!bwd) continue;
            dz_pass(nullptr);
        }
        // the scratch as the contractions see it: rows of 64 columns, 128 rows per block
        const uint64_t dz_rows = (uint64_t)(tcp / kDzBlockRows) * (uint64_t)(4 * z.n_tiles) * kDzBlockRows;
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
        if (grad_hidden) {
            // grad_hidden[token of gathered row] = (row factor) dZ[chunk, V] W[V, D]
            CUtensorMap mapDzK, mapWn;
            if (!make_map(&mapDzK, dz, dz_rows, kDzBlockCols, kDzBlockCols, BK, BM)) return RLF_ERR_CUDA;
            if (!make_map(&mapWn, Wm, (uint64_t)V, (uint64_t)D, (uint64_t)D, 64, BK)) return RLF_ERR_CUDA;
            GemmParams h = {};
            h.mode = kGradHidden;
            h.M = (int)tc;
            h.N = D;
            h.m_tiles = (int)((tc + BM - 1) / BM);
            h.n_tiles = (D + BN - 1) / BN;
            h.k_slabs = 4 * z.n_tiles;                     // every block of the scratch (zeros past the vocabulary)
            h.dz_nc = 4 * z.n_tiles;
            h.out_bf16 = static_cast<__nv_bfloat16*>(grad_hidden);
            h.out_stride = D;
            h.dev_status = dev_status;
            h.live_count = counts;
            h.live_off = (int)t0;
            h.row_index = idx_live;
            h.row_scale = row_ref ? scale_g + t0 : nullptr;
            h.pace = g.pace;
            st = launch_gemm(mapDzK, mapWn, h, pair, s);
            if (st != RLF_OK) return st;
        }
        if (grad_W) {
            // grad_W[V, D] (+)= dZ[chunk, V]^T hidden[chunk, D]  (hidden rows times their factors)
            CUtensorMap mapDzM, mapHn;
            if (!make_map(&mapDzM, dz, dz_rows, kDzBlockCols, kDzBlockCols, 64, BK)) return RLF_ERR_CUDA;
            if (!make_map(&mapHn, row_ref ? Hs : Hl + t0 * D, (uint64_t)tc, (uint64_t)D, (uint64_t)D, 64, BK))
                return RLF_ERR_CUDA;
            GemmParams q = {};
            q.mode = kGradW;
            q.M = V;
            q.N = D;
            q.m_tiles = (V + BM - 1) / BM;
            q.n_tiles = (D + BN - 1) / BN;
            q.k_slabs = (int)((tc + BK - 1) / BK);
            q.dz_nc = 4 * z.n_tiles;
            q.out_f32 = grad_W;
            q.out_stride = D;
            q.accumulate = (accumulate_grad_W || t0 > 0) ? 1 : 0;
            q.dev_status = dev_status;
            q.live_count = counts;
            q.live_off = (int)t0;
            q.pace = g.pace;
            st = launch_gemm(mapDzM, mapHn, q, pair, s);
            if (st != RLF_OK) return st;
        }
    }

    // the masked rows: log-prob only
    if (skip_masked) {
        fill_nan_rows_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(idx_dead, counts + 1, logp_out);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    } else {
        CUtensorMap mapHd;
        if (!make_map(&mapHd, Hd, (uint64_t)T, (uint64_t)D, (uint64_t)D, BK, BM)) return RLF_ERR_CUDA;
        GemmParams d = g;
        set_rows(d, T);
        d.live_count = counts + 1;
        d.live_off = 0;
        st = launch_gemm(mapHd, mapW, d, pair, s);
        if (st != RLF_OK) return st;
        combine_rows_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(part, d.nsplit, (int)T, idx_dead, counts + 1, 0, zy,
                                                                         rec, dn, eps_clip, eps_hi, wtok, beta_kl, logp_out,
                                                                         nullptr, nullptr, nullptr, dev_status, nullptr,
                                                                         nullptr, nullptr, 0, V, nullptr, nullptr, 0);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    }
    return token_loss(T);
}

}  // namespace lm
}  // namespace rlf

extern "C" rlf_status rlf_fused_lmhead_grpo(const void* hidden, const void* W, int64_t T, int32_t D, int32_t V,
                                            const int32_t* ids, const int32_t* seq_id, const float* adv, int32_t B,
                                            const float* old_logp, const float* ref_logp, const uint8_t* mask,
                                            float eps_clip, float beta_kl, const int64_t* denom, float* logp_out,
                                            double* loss_out, void* grad_hidden, float* grad_W,
                                            int accumulate_grad_W, void* workspace, size_t workspace_bytes,
                                            int32_t* dev_status, rlf_stream_t stream) {
    return rlf::lm::fused_lmhead_impl(hidden, W, T, D, V, ids, seq_id, adv, B, old_logp, ref_logp, mask, eps_clip,
                                      eps_clip, beta_kl, 0, 0, denom, logp_out, loss_out, grad_hidden, grad_W,
                                      accumulate_grad_W, workspace, workspace_bytes, dev_status, stream);
}

extern "C" rlf_status rlf_fused_lmhead_grpo_obj(const void* hidden, const void* W, int64_t T, int32_t D, int32_t V,
                                                const int32_t* ids, const int32_t* seq_id, const float* adv, int32_t B,
                                                const float* old_logp, const float* ref_logp, const uint8_t* mask,
                                                float eps_clip_low, float eps_clip_high, float beta_kl, int aggregation,
                                                int skip_masked, const int64_t* denom, float* logp_out,
                                                double* loss_out, void* grad_hidden, float* grad_W,
                                                int accumulate_grad_W, void* workspace, size_t workspace_bytes,
                                                int32_t* dev_status, rlf_stream_t stream) {
    if (skip_masked != 0 && skip_masked != 1) return RLF_ERR_SHAPE;
    return rlf::lm::fused_lmhead_impl(hidden, W, T, D, V, ids, seq_id, adv, B, old_logp, ref_logp, mask, eps_clip_low,
                                      eps_clip_high, beta_kl, aggregation, skip_masked, denom, logp_out, loss_out,
                                      grad_hidden, grad_W, accumulate_grad_W, workspace, workspace_bytes, dev_status,
                                      stream);
}


extern "C" rlf_status rlf_fused_lmhead_logp_entropy(const void* hidden, const void* W, int64_t T, int32_t D, int32_t V,
                                                    const int32_t* ids, float* logp_out, float* entropy_out,
                                                    void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                                    rlf_stream_t stream) {
    using namespace rlf;
    using namespace rlf::lm;
    if (T < 0 || V < 1 || D < 1) return RLF_ERR_SHAPE;
    if (D % 64 != 0 || V % 8 != 0) return RLF_ERR_SHAPE;
    if (T >= (1ll << 30)) return RLF_ERR_UNSUPPORTED;
    if (T == 0) return RLF_OK;
    if (!hidden || !W || !ids || !logp_out) return RLF_ERR_NULL;
    if (!aligned(hidden, 16) || !aligned(W, 16)) return RLF_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < lmhead_logp_workspace_bytes(T))
        return RLF_ERR_WORKSPACE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    char* ws = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(workspace) + 1023) & ~(uintptr_t)1023);
    float* zy = reinterpret_cast<float*>(ws);
    float2* part = reinterpret_cast<float2*>(ws + up1k(4 * (size_t)T));
    float* part_u = reinterpret_cast<float*>(ws + up1k(4 * (size_t)T) + up1k(8 * (size_t)T * kMaxSplit));
    const __nv_bfloat16* H = static_cast<const __nv_bfloat16*>(hidden);
    const __nv_bfloat16* Wm = static_cast<const __nv_bfloat16*>(W);
    target_logit_ids_kernel<<<(unsigned)((T + 7) / 8), 256, 0, s>>>(H, Wm, ids, T, D, V, zy, dev_status);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    const bool pair = g_pair.load() != 0;
    CUtensorMap mapH, mapW;
    if (!make_map(&mapH, H, (uint64_t)T, (uint64_t)D, (uint64_t)D, BK, BM)) return RLF_ERR_CUDA;
    if (!make_map(&mapW, Wm, (uint64_t)V, (uint64_t)D, (uint64_t)D, BK, pair ? BN / 2 : BN)) return RLF_ERR_CUDA;
    GemmParams g = {};
    g.mode = kLse;
    g.M = (int)T;
    g.N = V;
    g.m_tiles = (int)((T + BM - 1) / BM);
    g.n_tiles = (V + BN - 1) / BN;
    g.k_slabs = D / BK;
    g.nsplit = pick_split(g.n_tiles);
    g.n_tiles_per_split = (g.n_tiles + g.nsplit - 1) / g.nsplit;
    g.part = part;
    g.part_u = entropy_out ? part_u : nullptr;
    g.dev_status = dev_status;
    // the pacing counter sits in the kilobyte that closes the workspace
    g.pace = reinterpret_cast<int*>(ws + up1k(4 * (size_t)T) + up1k(8 * (size_t)T * kMaxSplit) + up1k(4 * (size_t)T * kMaxSplit));
    st = launch_gemm(mapH, mapW, g, pair, s);
    if (st != RLF_OK) return st;
    combine_logp_entropy_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(part, g.part_u, g.nsplit, zy, T, logp_out,
                                                                             entropy_out, dev_status);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

extern "C" rlf_status rlf_tune_lmhead(int pair_ctas) {
    if (pair_ctas != 0 && pair_ctas != 1) return RLF_ERR_SHAPE;
    rlf::lm::g_pair = pair_ctas;
    return RLF_OK;
}

extern "C" rlf_status rlf_tune_lmhead_backward(int row_reference, int two_accumulators) {
    if ((row_reference != 0 && row_reference != 1) || (two_accumulators != 0 && two_accumulators != 1)) return RLF_ERR_SHAPE;
    rlf::lm::g_row_ref = row_reference;
    rlf::lm::g_acc2 = two_accumulators;
    return RLF_OK;
}

extern "C" rlf_status rlf_tune_lmhead_pacing(int on) {
    if (on != 0 && on != 1) return RLF_ERR_SHAPE;
    rlf::lm::g_pace = on;
    return RLF_OK;
}

extern "C" rlf_status rlf_tune_lmhead_schedule(int m_block, int max_workers, int chunk_tiles) {
    if (m_block < 0 || m_block > (1 << 20) || max_workers < 0 || chunk_tiles < 0 || (chunk_tiles & 1)) return RLF_ERR_SHAPE;
    rlf::lm::g_m_block = m_block;
    rlf::lm::g_max_workers = max_workers;
    rlf::lm::g_chunk_tiles = chunk_tiles;
    return RLF_OK;
}
