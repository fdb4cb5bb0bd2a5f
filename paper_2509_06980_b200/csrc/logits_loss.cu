// Fused log-prob + clipped-ratio + k3-KL loss, forward and backward, over materialised logits.
//
// Kernels, in launch order:
//   token_prep_kernel   packs each token's scalars into one 16-byte record {old_logp, ref_logp,
//                       advantage, target id | live bit}, validates ids, and (when the caller gives
//                       no denominator) counts the mask.
//   row kernel          reads every logits row once, writes logp[t] and grad_logits[t, :].
//   token_loss_kernel + finalize_loss_kernel
//                       scalar loss from logp in fp64, added in a fixed order (run-to-run identical).
//
// Fast row kernel (bf16, 16-byte aligned rows).  A thread-block cluster owns one logits row at a
// time and keeps the WHOLE row in registers as packed bf16 (NV 16-byte vectors per thread), so the
// row crosses HBM exactly once in each direction:
//   1. cp.async brings each thread's NV coalesced 16-byte vectors into its own slots of a
//      shared-memory staging buffer (no registers held, no barrier: a thread only reads back what
//      it copied itself); the thread pulls them into registers, takes the packed bf16x2 max, and
//      immediately re-queues the same slots with the cluster's NEXT row, so HBM reads of row r+1
//      run under the rest of row r;
//   2. one exp2 per element against the WARP's max, fp32 sum, warp sum by shuffles; in the
//      one-exp variant the exponentials replace the logits in the registers (packed bf16);
//   3. every warp stores its (max, sum) into every CTA of the cluster and the owner of the target
//      column likewise sends z_target, as asynchronous distributed-shared-memory stores that credit
//      an mbarrier in the receiving CTA; each warp then waits (bounded) on its own CTA's mbarrier
//      for the row's byte count.  There is no thread barrier and no memory fence in the loop, so
//      a row's exchange never waits for the previous row's gradient stores to drain;
//   4. every warp merges all pairs of the row (lanes in parallel), forms lse, logp and the loss
//      coefficient c_t, and writes grad = c_t (softmax - onehot) from the registers it still
//      holds, either as exp2(z log2e + log2|c_t| - lse log2e) (two-exp) or as e * 2^(...) (one-exp).
// In the training variants the target column stays out of the warps' (max, sum): its owner replaces
// it by -inf in its staging slot before loading its registers, and every warp folds z_target back in
// after the merge.  The sum over the other columns, S', gives the target's gradient as -c S' / S, which
// keeps its digits when p_y rounds to one (c p_y - c does not).
// Exponents are formed by one FFMA per element; rows whose maximum is huge in magnitude switch to
// a subtract-first form so that the result stays accurate for any finite logits.
// Token records ride the same cp.async groups two rows ahead, so no scalar input costs a register
// across the passes.
//
// General row kernel (fp32 logits, odd V, unaligned rows): one CTA per row, three sweeps with
// scalar loads (max, sum, gradient); later sweeps of a row are served by L2 when the row fits.
#include <atomic>
#include <type_traits>
#include <mutex>

#include "common.cuh"

namespace rlf {

// workspace layout: [0] int64 sum of mask (used when no denominator is given); [256 ..) fp64
// partial sums of the token-loss kernel, 4 per block; then T 16-byte token records.
constexpr int kMaxPartials = 1024;
constexpr size_t kWsPartialOff = 256;
constexpr size_t kWsRecordOff = kWsPartialOff + sizeof(double) * 4 * kMaxPartials;

// the skip-masked variant adds, after the records: compacted records (16 B per token), the list of
// live rows (4 B per token); its live-row counter sits at byte 128 of the workspace
constexpr size_t ws_tokens(int64_t T) { return (size_t)(T > 0 ? T : 0); }
constexpr size_t ws_compact_rec_off(int64_t T) { return kWsRecordOff + 16 * ws_tokens(T) + 256; }
constexpr size_t ws_row_list_off(int64_t T) { return ws_compact_rec_off(T) + 16 * ws_tokens(T) + 256; }
// then per-token weights (4 B per token) and per-sequence counters (4 B x (T + 1)) of the
// sequence-mean aggregation
constexpr size_t ws_wtok_off(int64_t T) { return ws_row_list_off(T) + 4 * ws_tokens(T) + 256; }
constexpr size_t ws_seqcnt_off(int64_t T) { return ws_wtok_off(T) + 4 * ws_tokens(T) + 256; }
constexpr size_t ws_total_bytes(int64_t T) { return ws_seqcnt_off(T) + 4 * (ws_tokens(T) + 1) + 256; }
size_t loss_workspace_bytes(int64_t T) { return ws_total_bytes(T); }

// ---------------------------------------------------------------------------------------------
// token records
constexpr int kPrepThreads = 256;
__global__ void __launch_bounds__(kPrepThreads)
token_prep_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ seq_id,
                  const float* __restrict__ adv, const float* __restrict__ old_logp,
                  const float* __restrict__ ref_logp, const uint8_t* __restrict__ mask, int64_t T,
                  int32_t V, int32_t B, float4* __restrict__ rec, unsigned long long* __restrict__ n_count,
                  int32_t* __restrict__ dev_status) {
    const int64_t t = (int64_t)blockIdx.x * kPrepThreads + threadIdx.x;
    int live = 0, bad = 0;
    if (t < T) {
        int32_t y = ids[t];
        const int32_t sid = seq_id[t];
        float A = 0.0f;
        if (y < 0 || y >= V) { bad |= RLF_DEV_BAD_TARGET; y = 0; }
        if (sid < 0 || sid >= B) bad |= RLF_DEV_BAD_SEQ;
        else A = adv[sid];
        const int m = mask[t] != 0;
        live = m && !bad;
        rec[t] = make_float4(old_logp[t], ref_logp[t], A, __int_as_float(y | (live ? (int)0x80000000 : 0)));
        live = m;   // the denominator counts the mask as given
    }
    if (n_count != nullptr) {
        const unsigned c = __popc(__ballot_sync(0xffffffffu, live));
        if ((threadIdx.x & 31) == 0 && c) atomicAdd(n_count, (unsigned long long)c);
    }
    if (bad && dev_status) atomicOr(dev_status, bad);
}

// d(pg + beta kl)/d logp with hardware exp2 (relative error ~1e-6: ample for a bf16 gradient)
__device__ __forceinline__ float grad_coef_fast(float logp, float old_lp, float ref_lp, float A,
                                                float eps_lo, float eps_hi, float beta) {
    const float rho = ex2_approx((logp - old_lp) * kLog2e);
    const bool clipped = ((A > 0.0f) && (rho > 1.0f + eps_hi)) || ((A < 0.0f) && (rho < 1.0f - eps_lo));
    const float dpg = clipped ? 0.0f : -A * rho;
    const float ed = ex2_approx((ref_lp - logp) * kLog2e);
    return fmaf(beta, 1.0f - ed, dpg);
}

// ---------------------------------------------------------------------------------------------
// Fast row kernel
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// order-preserving float <-> int map so that a warp max is one redux instruction
__device__ __forceinline__ int f2ord(float f) {
    int i = __float_as_int(f);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// store a float4 into the same shared-memory location of CTA `rank` of this cluster
__device__ __forceinline__ void st_cluster_f4(uint32_t local_addr, uint32_t rank, float4 v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1,%2,%3,%4};"
                 :: "r"(remote), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" :: "r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async16_cg(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" :: "r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_group1() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

constexpr uint32_t kNegInfPair = 0xFF80FF80u;   // two bf16 -inf

struct FastParams {
    const __nv_bfloat16* logits;
    __nv_bfloat16* grad;        // nullable
    long long stride;           // elements
    int T;
    int nvec;                   // V / 8
    int per_cta_vec;
    const float4* rec;
    const long long* denom;
    float* logp_out;
    float* entropy_out;         // entropy variant only, nullable
    const int* row_list;        // skip-masked variant: rows to process, rec[] is indexed like this list
    const int* n_rows;          // skip-masked variant: device count of listed rows
    const float* wtok;          // per-token loss weights (sequence-mean aggregation) or NULL: 1 / N
    int32_t* dev_status;
    float eps_clip, eps_hi, beta;   // clip range [1 - eps_clip, 1 + eps_hi]
};

// bf16 element e (0..7) of a 16-byte vector, widened
__device__ __forceinline__ float pick_elem(const uint4& v, int e) {
    const int w = e >> 1;
    uint32_t word = w == 0 ? v.x : (w == 1 ? v.y : (w == 2 ? v.z : v.w));
    return (e & 1) ? bf_hi(word) : bf_lo(word);
}
__device__ __forceinline__ void put_elem(uint4& v, int e, float x) {
    const uint32_t gb = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x));
    const uint32_t keep = (e & 1) ? 0x0000ffffu : 0xffff0000u;
    const uint32_t ins = (e & 1) ? (gb << 16) : gb;
    const int w = e >> 1;
    if (w == 0) v.x = (v.x & keep) | ins;
    if (w == 1) v.y = (v.y & keep) | ins;
    if (w == 2) v.z = (v.z & keep) | ins;
    if (w == 3) v.w = (v.w & keep) | ins;
}

// exponent of one element.  Fast form: one FFMA, z log2e + off with off = -m log2e rounded to fp32,
// accurate while |m| is moderate (the rounding of off is an absolute error of |m| 2^-24 log2e in
// the exponent).  Robust form for rows with a huge maximum: (z - m) log2e + add, subtraction first.
constexpr float kRobustAbove = 2048.0f;
template <bool ROBUST>
__device__ __forceinline__ float expo(float z, float m, float off) {
    return ROBUST ? fmaf(z - m, kLog2e, off) : fmaf(z, kLog2e, off);
}

// sum of 2^expo over this thread's registers; ONE_EXP keeps the exponentials in place as bf16
template <int NV, bool ONE_EXP, bool ROBUST>
__device__ __forceinline__ float exp_sum_pass(uint4 (&d)[NV], float m, float off) {
    float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        uint32_t* w = reinterpret_cast<uint32_t*>(&d[i]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float e0 = ex2_approx(expo<ROBUST>(bf_lo(w[k]), m, off));
            const float e1 = ex2_approx(expo<ROBUST>(bf_hi(w[k]), m, off));
            s0 += e0;
            s1 += e1;
            if (ONE_EXP) w[k] = pack_bf16x2(e0, e1);
        }
    }
    return s0 + s1;
}

// forward-only variant with entropy: besides s = sum 2^x it accumulates u = sum 2^x * x, where
// x = (z - m) log2e is the element's exponent (clamped below so that a vanishing term contributes
// 0 * finite instead of 0 * inf); the entropy is ln S - ln2 * U / S once merged over the row
template <int NV, bool ROBUST>
__device__ __forceinline__ float2 exp_sum_ent_pass(const uint4 (&d)[NV], float m, float off) {
    float s0 = 0.0f, s1 = 0.0f, u0 = 0.0f, u1 = 0.0f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const uint32_t w[4] = {d[i].x, d[i].y, d[i].z, d[i].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float x0 = fmaxf(expo<ROBUST>(bf_lo(w[k]), m, off), -1e30f);
            const float x1 = fmaxf(expo<ROBUST>(bf_hi(w[k]), m, off), -1e30f);
            const float e0 = ex2_approx(x0), e1 = ex2_approx(x1);
            s0 += e0;
            s1 += e1;
            u0 = fmaf(e0, x0, u0);
            u1 = fmaf(e1, x1, u1);
        }
    }
    return make_float2(s0 + s1, u0 + u1);
}

template <bool ROBUST>
__device__ __forceinline__ uint4 grad_vec_two_exp(const uint4& v, float m, float off, uint32_t sgn) {
    uint4 o;
    o.x = pack_bf16x2(ex2_approx(expo<ROBUST>(bf_lo(v.x), m, off)), ex2_approx(expo<ROBUST>(bf_hi(v.x), m, off))) ^ sgn;
    o.y = pack_bf16x2(ex2_approx(expo<ROBUST>(bf_lo(v.y), m, off)), ex2_approx(expo<ROBUST>(bf_hi(v.y), m, off))) ^ sgn;
    o.z = pack_bf16x2(ex2_approx(expo<ROBUST>(bf_lo(v.z), m, off)), ex2_approx(expo<ROBUST>(bf_hi(v.z), m, off))) ^ sgn;
    o.w = pack_bf16x2(ex2_approx(expo<ROBUST>(bf_lo(v.w), m, off)), ex2_approx(expo<ROBUST>(bf_hi(v.w), m, off))) ^ sgn;
    return o;
}

// Resident CTAs per SM: bounded by registers (64 per thread) and by the staging buffer.
constexpr int kSmemBudget = 220 * 1024;
constexpr int stage_bytes(int threads, int nv) { return nv * threads * 16; }
constexpr int ctas_per_sm(int threads, int nv) {
    const int by_regs = 65536 / (64 * threads);
    const int by_smem = kSmemBudget / (stage_bytes(threads, nv) + 4096);
    const int m = by_regs < by_smem ? by_regs : by_smem;
    return m < 1 ? 1 : m;
}

// Asynchronous stores into the shared memory of CTA `rank` of this cluster: the data is written to
// the peer's copy of `local_addr` and its byte count is credited to the peer's copy of the mbarrier
// at `local_mbar`, which is how the peer learns that it has arrived (no fence, no thread barrier).
__device__ __forceinline__ void st_async_f2(uint32_t local_addr, uint32_t local_mbar, uint32_t rank, float a, float b) {
    uint32_t raddr, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(local_mbar), "r"(rank));
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 :: "r"(raddr), "f"(a), "f"(b), "r"(rbar) : "memory");
}
__device__ __forceinline__ void st_async_f1(uint32_t local_addr, uint32_t local_mbar, uint32_t rank, float a) {
    uint32_t raddr, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(local_mbar), "r"(rank));
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];"
                 :: "r"(raddr), "f"(a), "r"(rbar) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t mbar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for one phase of an mbarrier: false when it gives up (about a second).
constexpr int kWaitPolls = 1 << 22;
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t mbar, uint32_t parity) {
    for (int i = 0; i < kWaitPolls; ++i)
        if (mbar_try_wait(mbar, parity)) return true;
    return false;
}

__device__ __forceinline__ int ring_read(const int* ring, int slot) { return reinterpret_cast<const volatile int*>(ring)[slot]; }

// SKIP: the rows to process come from a compacted list (rows whose loss weight is zero are
// neither read nor computed); token records are then indexed like the list.
// WT: per-token loss weights from the caller replace the common 1 / N.
// CMAX: the largest cluster the instantiation serves (8 is the portable limit; 16 for rows that 8 CTAs
// of 256 threads cannot hold, e.g. a vocabulary of 262144, launched with the non-portable size allowed).
template <int THREADS, int NV, bool ONE_EXP, bool ENT = false, bool SKIP = false, bool WT = false, int CMAX = 8>
__global__ void __launch_bounds__(THREADS, ctas_per_sm(THREADS, NV))
grpo_row_cluster_kernel(const FastParams p) {
    constexpr int NWARPS = THREADS / 32;
    constexpr int MAXE = CMAX * NWARPS;       // (max, sum) pairs per row: one per warp of the cluster
    // staging: [NV][THREADS] 16-byte slots; a thread only ever touches its own slots, so its own
    // cp.async wait is all the synchronisation the logits data needs
    extern __shared__ __align__(16) uint4 stage[];
    __shared__ __align__(8) float2 pair_slot[2][MAXE];   // per row parity: every warp's (max, sum)
    constexpr int RM = SKIP ? 7 : 3;                     // ring mask of the per-row metadata
    constexpr int AHEAD = SKIP ? 3 : 2;                  // how many rows ahead thread 0 fetches metadata
    __shared__ __align__(16) float4 rec_slot[RM + 1];    // token records, ring over rows
    __shared__ int row_slot[SKIP ? 8 : 1];               // skip variant: row index of each listed row
    __shared__ float w_slot[WT ? RM + 1 : 1];            // per-token loss weight (WT variant)
    __shared__ float zy_slot[2];                         // per row parity: the target logit
    __shared__ float ent_slot[2][ENT ? MAXE : 1];        // entropy variant: every warp's sum 2^x * x
    __shared__ __align__(8) unsigned long long row_bar[2];   // per row parity: "all pairs and z_target are here"

    const int csize = (int)cluster_nctarank();
    const int crank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x / csize;
    const int num_clusters = gridDim.x / csize;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int npairs = csize * NWARPS;

    // this thread's vectors are  vbeg + i * THREADS  for i < NV, live while < vend
    const int vbeg = crank * p.per_cta_vec + tid;
    const int vend = min(p.nvec, (crank + 1) * p.per_cta_vec);
    // number of live vectors of this thread (they are the first nvalid of the NV), same for every row
    const int nvalid = vend > vbeg ? min(NV, (vend - vbeg + THREADS - 1) / THREADS) : 0;

    float inv_n;
    {
        const long long N = *p.denom;
        inv_n = 1.0f / (float)(N > 1 ? N : 1);
    }

    const int nrows = SKIP ? *p.n_rows : p.T;
    // thread 0 fetches the metadata of the row this cluster handles in iteration `j` (its token
    // record; in the skip variant also its row index) into the rings
    auto fetch_meta = [&](int j) {
        const long long k = (long long)cluster_id + (long long)j * num_clusters;
        if (tid == 0 && j >= 0 && k < nrows) {
            cp_async16(&rec_slot[j & RM], p.rec + k);
            if (SKIP) cp_async4(&row_slot[j & RM], p.row_list + k);
            if (WT) cp_async4(&w_slot[j & RM], p.wtok + k);
        }
    };
    // queue this thread's part of a row into the staging buffer (one cp.async group per row; thread
    // 0's group also carries metadata of a later row)
    auto prefetch = [&](int row, bool have, int meta_j) {
        if (have) {
            const uint4* src = reinterpret_cast<const uint4*>(p.logits + (long long)row * p.stride) + vbeg;
            uint4* dst = stage + tid;
#pragma unroll
            for (int i = 0; i < NV; ++i)
                if (i < nvalid) cp_async16_cg(dst + i * THREADS, src + i * THREADS);
        }
        fetch_meta(meta_j);
        cp_async_commit();
    };

    // per row every CTA receives one (max, sum) pair from every warp of the cluster and z_target
    const uint32_t row_bytes = (uint32_t)npairs * (ENT ? 12u : 8u) + 4u;
    if (tid == 0) {
        mbar_init(smem_u32(&row_bar[0]), 1);
        mbar_init(smem_u32(&row_bar[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int j = 0; j < AHEAD; ++j) fetch_meta(j);
    if (SKIP) {
        // the first row's index is needed to start its copy
        cp_async_wait_all();
        __syncthreads();
    }
    {
        const bool have0 = cluster_id < nrows;
        const int row0 = SKIP ? (have0 ? row_slot[0] : 0) : cluster_id;
        prefetch(row0, have0, -1);       // first row of this cluster (no further metadata yet)
    }
    cp_async_wait_all();                 // the first records must be visible CTA-wide below
    // every CTA of the cluster is running before any peer may address its shared memory
    cluster_sync_all();

    int status = 0;
    int it = 0;
    bool gave_up = false;                // a wait ran out: stop waiting, finish the loop, report
    for (int k = cluster_id; k < nrows; k += num_clusters, ++it) {
        const int parity = it & 1;
        // the listed row's index is re-read from its ring slot where it is used (late in the iteration)
        // instead of being held in a register across the passes: the skip variant is at its register
        // budget, and a spill in this loop costs more than a few shared-memory reads
        const int row = SKIP ? 0 : k;
#define RLF_CUR_ROW() (SKIP ? ring_read(row_slot, it & RM) : row)
        const uint32_t bar = smem_u32(&row_bar[parity]);
        cp_async_wait_all();             // this thread's part of the row (and thread 0's metadata) has landed
        // an arrive releases what this thread did before it: the landed metadata becomes visible to
        // every thread that later sees this barrier's phase complete
        if (tid == 0) mbar_arrive_expect_tx(bar, row_bytes);
        // the owner of the target column sends z_target to every CTA of the cluster; the target id is
        // re-read from its ring slot where the gradient needs it again, not held across the passes
#define RLF_TARGET_ID() (ring_read(reinterpret_cast<const int*>(rec_slot), 4 * (it & RM) + 3) & 0x7fffffff)
#define RLF_OWNS(yrel) ((yrel) >= 0 && ((yrel) & (THREADS - 1)) == 0 && ((yrel) / THREADS) < nvalid)
        const int y = RLF_TARGET_ID();
        const int yrel = (y >> 3) - vbeg;             // owner iff a multiple of THREADS below nvalid * THREADS
        if (RLF_OWNS(yrel)) {
            // the target logit sits in this thread's own staging slot
            __nv_bfloat16* sv = reinterpret_cast<__nv_bfloat16*>(&stage[yrel + tid]);
            const float zt = __bfloat162float(sv[y & 7]);
            for (int r = 0; r < csize; ++r) st_async_f1(smem_u32(&zy_slot[parity]), bar, (uint32_t)r, zt);
            // The training variants sum over the OTHER columns: the target becomes -inf in the slot
            // before the registers are loaded, so it drops out of (max, sum) here and comes back in
            // once per row from z_target.  S' = S - 2^(z_y - M) is what the target column's gradient
            // needs, -c S' / S, and summing it directly avoids the cancellation of c (p_y - 1).
            // (stored by an asm statement with a memory clobber: the loads below read the same bytes through
            // another type, and nothing may move them above this store)
            if (!ENT)
                asm volatile("st.shared.b16 [%0], %1;" :: "r"(smem_u32(sv + (y & 7))), "h"((unsigned short)0xff80u) : "memory");
        }
        uint4 d[NV];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            if (i < nvalid) d[i] = stage[i * THREADS + tid];
            else d[i] = make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);
        }

        // max over the registers (packed), then over the warp
        uint32_t mx = kNegInfPair;
#pragma unroll
        for (int i = 0; i < NV; ++i)
            mx = max_bf16x2(mx, max_bf16x2(max_bf16x2(d[i].x, d[i].y), max_bf16x2(d[i].z, d[i].w)));
        // the staging slots have been consumed (the max needed every register): refill them with
        // the cluster's next row while this one is processed
        {
            const bool have_next = k + num_clusters < nrows;
            const int next_row = SKIP ? (have_next ? row_slot[(it + 1) & RM] : 0) : k + num_clusters;
            prefetch(next_row, have_next, it + AHEAD);
        }

        float m_w = fmaxf(bf_lo(mx), bf_hi(mx));
        m_w = ord2f(__reduce_max_sync(0xffffffffu, f2ord(m_w)));
        // exponent base of this warp: 2^((z - m_w) log2e); all lanes agree on the form
        const float m_ws = (m_w == -INFINITY) ? 0.0f : m_w;
        const bool robust_w = fabsf(m_ws) > kRobustAbove;
        float s_t, u_w = 0.0f;
        if (ENT) {
            const float2 su = robust_w ? exp_sum_ent_pass<NV, true>(d, m_ws, 0.0f)
                                       : exp_sum_ent_pass<NV, false>(d, 0.0f, -m_ws * kLog2e);
            s_t = su.x;
            u_w = warp_sum(su.y);
        } else {
            s_t = robust_w ? exp_sum_pass<NV, ONE_EXP, true>(d, m_ws, 0.0f)
                           : exp_sum_pass<NV, ONE_EXP, false>(d, 0.0f, -m_ws * kLog2e);
        }
        const float s_w = warp_sum(s_t);
        // every warp hands its (max, sum) to every CTA of the cluster, then waits until its own CTA
        // has received the whole row's worth (the only synchronisation in the loop)
        if (lane < csize) {
            st_async_f2(smem_u32(&pair_slot[parity][crank * NWARPS + warp]), bar, (uint32_t)lane, m_w, s_w);
            if (ENT) st_async_f1(smem_u32(&ent_slot[parity][crank * NWARPS + warp]), bar, (uint32_t)lane, u_w);
        }
        if (!gave_up && !mbar_wait_bounded(bar, (uint32_t)(it >> 1) & 1u)) {
            gave_up = true;
            status |= RLF_DEV_TIMEOUT;
        }

        // merge all pairs of the row, lanes in parallel, identically in every warp
        float M = -INFINITY;
        float2 e[MAXE / 32 > 0 ? MAXE / 32 : 1];
#pragma unroll
        for (int j = 0; j < (MAXE + 31) / 32; ++j) {
            const int k = lane + 32 * j;
            e[j] = (k < npairs) ? pair_slot[parity][k] : make_float2(-INFINITY, 0.0f);
            M = fmaxf(M, e[j].x);
        }
        M = ord2f(__reduce_max_sync(0xffffffffu, f2ord(M)));
        const float zy = zy_slot[parity];
        if (!ENT) M = fmaxf(M, zy);                  // the pairs of the training variants leave the target out
        float S = 0.0f, U = 0.0f;
#pragma unroll
        for (int j = 0; j < (MAXE + 31) / 32; ++j) {
            if (e[j].x != -INFINITY) {
                const float dx = (e[j].x - M) * kLog2e;          // this warp's base relative to the row's
                const float f = ex2_approx(dx);
                S += e[j].y * f;
                if (ENT) {
                    const int k = lane + 32 * j;
                    // exponents relative to the row maximum are x + dx; a warp whose weight f
                    // vanishes contributes nothing (its dx may be -huge)
                    if (f > 0.0f) U += f * fmaf(e[j].y, dx, ent_slot[parity][k < npairs ? k : 0]);
                }
            }
        }
        S = warp_sum(S);
        if (ENT) U = warp_sum(U);
        const float4 rec = rec_slot[it & RM];
        // the training variants summed without the target column: S' = S here, S = S' + 2^((z_y - M) log2e)
        float others = 0.0f;                         // S' / S = 1 - p_y
        if (!ENT) {
            const float s_all = S + ex2_approx((zy - M) * kLog2e);
            others = __fdividef(S, s_all);
            S = s_all;
        }
        const float lg2s = lg2_approx(S);
        const float logp = (zy - M) - lg2s * kLn2;
        const bool finite = (M > -INFINITY) && (M < INFINITY) && (S > 0.0f) && (S < INFINITY) &&
                            (fabsf(logp) < INFINITY);
        const bool live = (__float_as_int(rec.w) < 0) && finite;
        const float w_row = WT ? w_slot[it & RM] : inv_n;
        const float coef = live ? -w_row * grad_coef_fast(logp, rec.x, rec.y, rec.z, p.eps_clip, p.eps_hi, p.beta) : 0.0f;
        if (crank == 0 && tid == 0) {
            // forward-only variant: a row whose target id was out of range has no log-prob
            const bool has_logp = finite && (!ENT || __float_as_int(rec.w) < 0);
            p.logp_out[RLF_CUR_ROW()] = has_logp ? logp : __int_as_float(0x7fc00000);
            if (!finite) status |= RLF_DEV_NONFINITE;
            // H = ln S - ln2 * U / S  (= lse - E[z])
            if (ENT && p.entropy_out) p.entropy_out[RLF_CUR_ROW()] = finite ? (lg2s - U / S) * kLn2 : __int_as_float(0x7fc00000);
        }

        if (!ENT && p.grad != nullptr) {
            uint4* dst = reinterpret_cast<uint4*>(p.grad + (long long)RLF_CUR_ROW() * p.stride) + vbeg;
            if (coef == 0.0f || !(fabsf(coef) < INFINITY)) {
                const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int i = 0; i < NV; ++i)
                    if (i < nvalid) st_stream(dst + i * THREADS, z4);
            } else {
                // grad = sign(c) 2^((z - M) log2e + lc), lc = log2|c| - log2 S; the target column is written apart
                const float lc = lg2_approx(fabsf(coef)) - lg2s;
                const float gy = -coef * others;                                    // c (p_y - 1) = -c S' / S
                if (ONE_EXP) {
                    // the registers hold 2^((z - m_w) log2e): rescale from the warp's base to the row's
                    const float scale = copysignf(ex2_approx(fmaf(m_ws - M, kLog2e, lc)), coef);
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        if (i < nvalid) {
                            uint4 o;
                            o.x = pack_bf16x2(bf_lo(d[i].x) * scale, bf_hi(d[i].x) * scale);
                            o.y = pack_bf16x2(bf_lo(d[i].y) * scale, bf_hi(d[i].y) * scale);
                            o.z = pack_bf16x2(bf_lo(d[i].z) * scale, bf_hi(d[i].z) * scale);
                            o.w = pack_bf16x2(bf_lo(d[i].w) * scale, bf_hi(d[i].w) * scale);
                            st_stream(dst + i * THREADS, o);
                        }
                    }
                } else {
                    const uint32_t sgn = coef < 0.0f ? 0x80008000u : 0u;
                    const bool robust_r = fabsf(M) > kRobustAbove;
                    const float c2 = lc - M * kLog2e;
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        if (i < nvalid) {
                            uint4 o = robust_r ? grad_vec_two_exp<true>(d[i], M, lc, sgn)
                                               : grad_vec_two_exp<false>(d[i], 0.0f, c2, sgn);
                            st_stream(dst + i * THREADS, o);
                        }
                    }
                }
                // the owner overwrites the target column of the vector it has just stored
                const int yg = RLF_TARGET_ID();
                if (RLF_OWNS((yg >> 3) - vbeg)) p.grad[(long long)RLF_CUR_ROW() * p.stride + yg] = __float2bfloat16_rn(gy);
            }
        }
    }
    if (status && p.dev_status) atomicOr(p.dev_status, status);
    // A warp that gave up has stopped waiting for its rows' exchanges, so peers' asynchronous stores
    // of the last rows may still be on their way into this CTA's shared memory: give them two
    // milliseconds (they take microseconds) before the CTA may be retired.  Every CTA still runs all
    // its iterations and issues all its stores, so the barrier below is always reached by all.
    if (gave_up)
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    // no CTA leaves while a peer could still address its shared memory
    cluster_sync_all();
}

// ---------------------------------------------------------------------------------------------
#undef RLF_CUR_ROW
#undef RLF_TARGET_ID
#undef RLF_OWNS

// General row kernel: one CTA per row, scalar loads, any dtype / V / alignment.
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct GenParams {
    const void* logits;
    void* grad;                 // nullable
    long long stride;
    long long T;
    int V;
    const float4* rec;
    const long long* denom;
    float* logp_out;
    float* entropy_out;         // nullable: also return the row's entropy (forward-only use)
    int fwd_only;               // forward-only entry point: a row with a bad target id gets NaN
    const float* wtok;          // per-token loss weights or NULL: 1 / N
    int32_t* dev_status;
    float eps_clip, eps_hi, beta;
};

constexpr int kGenThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kGenThreads)
grpo_row_general_kernel(const GenParams p) {
    __shared__ float red[kGenThreads / 32];
    __shared__ float red_u[kGenThreads / 32];
    __shared__ float bcast, bcast_u;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long N = *p.denom;
    const float inv_n = 1.0f / (float)(N > 1 ? N : 1);
    int status = 0;

    for (long long row = blockIdx.x; row < p.T; row += gridDim.x) {
        const T* z = static_cast<const T*>(p.logits) + row * p.stride;
        const float4 rec = p.rec[row];
        const int y = __float_as_int(rec.w) & 0x7fffffff;
        const float zy = to_f32<T>(z[y]);

        float m = -INFINITY;
        for (int v = tid; v < p.V; v += kGenThreads) m = fmaxf(m, to_f32<T>(z[v]));
        m = warp_max(m);
        if (lane == 0) red[warp] = m;
        __syncthreads();
        if (tid == 0) {
            float mm = red[0];
            for (int w = 1; w < kGenThreads / 32; ++w) mm = fmaxf(mm, red[w]);
            bcast = mm;
        }
        __syncthreads();
        const float M = bcast;
        const float Ms = (M == -INFINITY) ? 0.0f : M;
        float s = 0.0f, u = 0.0f;
        // the sums leave the target column out; it comes back in once per row below.  S' = sum over the
        // other columns gives the target's gradient as -c S' / S without the cancellation of c (p_y - 1)
        for (int v = tid; v < p.V; v += kGenThreads) {
            const float x = fmaxf((to_f32<T>(z[v]) - Ms) * kLog2e, -1e30f);
            const float e = (v == y) ? 0.0f : ex2_approx(x);
            s += e;
            u = fmaf(e, x, u);                 // for the entropy: sum 2^x * x
        }
        s = warp_sum(s);
        u = warp_sum(u);
        __syncthreads();
        if (lane == 0) { red[warp] = s; red_u[warp] = u; }
        __syncthreads();
        if (tid == 0) {
            float ss = 0.0f, uu = 0.0f;
            for (int w = 0; w < kGenThreads / 32; ++w) { ss += red[w]; uu += red_u[w]; }
            bcast = ss;
            bcast_u = uu;
        }
        __syncthreads();
        const float S_others = bcast;
        const float x_y = fmaxf((zy - Ms) * kLog2e, -1e30f);
        const float e_y = ex2_approx(x_y);
        const float S = S_others + e_y;
        const float U = fmaf(e_y, x_y, bcast_u);
        __syncthreads();

        const float lg2s = lg2_approx(S);
        const float logp = (zy - M) - lg2s * kLn2;
        const bool finite = (M > -INFINITY) && (M < INFINITY) && (S > 0.0f) && (S < INFINITY) &&
                            (fabsf(logp) < INFINITY);
        const bool live = (__float_as_int(rec.w) < 0) && finite;
        const float w_row = p.wtok ? p.wtok[row] : inv_n;
        const float coef = live ? -w_row * grad_coef_fast(logp, rec.x, rec.y, rec.z, p.eps_clip, p.eps_hi, p.beta) : 0.0f;
        if (tid == 0) {
            const bool has_logp = finite && (!p.fwd_only || __float_as_int(rec.w) < 0);
            p.logp_out[row] = has_logp ? logp : __int_as_float(0x7fc00000);
            if (!finite) status |= RLF_DEV_NONFINITE;
            if (p.entropy_out) p.entropy_out[row] = finite ? (lg2s - U / S) * kLn2 : __int_as_float(0x7fc00000);
        }
        if (p.grad != nullptr) {
            T* g = static_cast<T*>(p.grad) + row * p.stride;
            if (coef == 0.0f || !(fabsf(coef) < INFINITY)) {
                for (int v = tid; v < p.V; v += kGenThreads) g[v] = from_f32<T>(0.0f);
            } else {
                for (int v = tid; v < p.V; v += kGenThreads) {
                    const float pv = ex2_approx(fmaf(to_f32<T>(z[v]) - M, kLog2e, -lg2s));
                    const float gv = (v == y) ? -coef * (S_others / S) : coef * pv;
                    g[v] = from_f32<T>(gv);
                }
            }
        }
    }
    if (tid == 0 && status && p.dev_status) atomicOr(p.dev_status, status);
}

// ---------------------------------------------------------------------------------------------
// Token terms from logp in fp64.  Each block adds its tokens in a fixed order and writes one slot.
// A token counts when its record is live and its logp is finite (the row kernels write NaN for a
// non-finite row).
constexpr int kLossThreads = 256;
__global__ void __launch_bounds__(kLossThreads)
token_loss_kernel(const float* __restrict__ logp, const float4* __restrict__ rec, int64_t T,
                  float eps_clip, float eps_hi, const float* __restrict__ wtok, double* __restrict__ partial) {
    __shared__ double red[kLossThreads / 32][3];
    double a_pg = 0.0, a_kl = 0.0, a_cl = 0.0;
    for (int64_t t = (int64_t)blockIdx.x * kLossThreads + threadIdx.x; t < T;
         t += (int64_t)gridDim.x * kLossThreads) {
        const float4 r = rec[t];
        const double lp = (double)logp[t];
        if (__float_as_int(r.w) >= 0 || !isfinite(lp)) continue;
        const double A = (double)r.z;
        const double rho = exp(lp - (double)r.x);
        const double lo = 1.0 - (double)eps_clip, hi = 1.0 + (double)eps_hi;
        const double rc = fmin(fmax(rho, lo), hi);
        const double w = wtok ? (double)wtok[t] : 1.0;      // token mean: divided by N at the end
        a_pg += w * -fmin(rho * A, rc * A);
        a_cl += ((A > 0.0 && rho > hi) || (A < 0.0 && rho < lo)) ? w : 0.0;
        const double d = (double)r.y - lp;
        a_kl += w * (expm1(d) - d);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a_pg += __shfl_xor_sync(0xffffffffu, a_pg, o);
        a_kl += __shfl_xor_sync(0xffffffffu, a_kl, o);
        a_cl += __shfl_xor_sync(0xffffffffu, a_cl, o);
    }
    if ((threadIdx.x & 31) == 0) {
        red[threadIdx.x >> 5][0] = a_pg;
        red[threadIdx.x >> 5][1] = a_kl;
        red[threadIdx.x >> 5][2] = a_cl;
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        double a = 0.0;
        for (int w = 0; w < kLossThreads / 32; ++w) a += red[w][threadIdx.x];
        partial[4 * (int64_t)blockIdx.x + threadIdx.x] = a;
    }
}

// per-block partial sums -> loss_out[4].  One warp per quantity: each lane adds its partials (stride 32,
// index order), then a fixed shuffle tree: the same order on every launch, so results are run-to-run
// identical.  Launched with 96 threads.
__global__ void __launch_bounds__(96)
finalize_loss_kernel(const double* __restrict__ partial, int num_partials, const long long* __restrict__ denom,
                     float beta, int weighted, double* __restrict__ loss_out) {
    __shared__ double s[3];
    const int q = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double a = 0.0;
    for (int i = lane; i < num_partials; i += 32) a += partial[4 * i + q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) s[q] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long N = *denom;
        const double nd = weighted ? 1.0 : (double)(N > 1 ? N : 1);   // weighted sums are already means
        loss_out[0] = (s[0] + (double)beta * s[1]) / nd;
        loss_out[1] = s[0] / nd;
        loss_out[2] = s[1] / nd;
        loss_out[3] = s[2] / nd;
    }
}

// ---------------------------------------------------------------------------------------------
// host side
static std::atomic<int> g_tune_cluster{0};
static std::atomic<int> g_tune_threads{0};
static std::atomic<int> g_tune_one_exp{-1};
static std::atomic<int> g_rows_per_cluster{0};    // 0: built-in
static std::atomic<int> g_units_per_cta{0};       // streaming forward pass; 0: built-in

struct FastShape { int cluster, threads, nv, one_exp; };

static const int kNvChoices[] = {1, 2, 3, 4, 5, 6, 7, 8, 9, 10};

static int round_nv(int need) {
    for (int c : kNvChoices) if (c >= need) return c;
    return 0;
}

// 16-byte vectors of a row per CTA of a cluster: an even split rounded up to whole 128-byte lines, so
// that every CTA's piece of a (line-aligned) row starts on a line.  Pieces that start in the middle of
// a 32-byte sector cost 10 - 20 % of the bandwidth (V = 200000 over 16 CTAs: 1563 vectors each).
static int per_cta_vectors(int nvec, int cluster) {
    return (((nvec + cluster - 1) / cluster) + 7) & ~7;
}

// launch shape that holds a row of nvec 16-byte vectors in registers
static bool pick_shape(int nvec, FastShape* out, bool allow_wide_cluster = false) {
    const int tc = g_tune_cluster.load(), tt = g_tune_threads.load();
    const int oe = g_tune_one_exp.load() < 0 ? 1 : g_tune_one_exp.load();
    if (tc > 0 && tt > 0) {
        // clusters beyond the portable 8 exist for the plain training kernel with 256-thread CTAs only
        if (tc > 8 && (!allow_wide_cluster || tt != 256 || !oe)) return false;
        const int per = per_cta_vectors(nvec, tc);
        int nv = round_nv((per + tt - 1) / tt);
        if (nv == 0) return false;
        if (tc > 8 && nv < 6) nv = 6;                 // the smallest instantiation for those clusters
        *out = {tc, tt, nv, oe};
        return true;
    }
    // built-in choice: 256-thread CTAs holding up to 10 vectors per thread (four CTAs per SM), in
    // the smallest cluster that covers the row; wider CTAs only for rows beyond 8 x 256 x 10 vectors
    for (int th = 256; th <= 1024; th *= 2) {
        for (int c = 1; c <= 8; c *= 2) {
            const int per = per_cta_vectors(nvec, c);
            const int need = (per + th - 1) / th;
            if (need <= 10 && stage_bytes(th, round_nv(need)) <= kSmemBudget) {
                *out = {c, th, round_nv(need), oe};
                return true;
            }
        }
        // rows beyond 8 x 256 x 10 vectors: a cluster of 16 such CTAs (four per SM, every register
        // holding a piece of a row) before CTAs of 512 threads (two per SM): V = 262144 ran at 0.80 of
        // the copy rate as 8 x 512 threads
        // (10 CTAs where they hold the row, V <= 204800, else 16: V = 200000 runs at 6.09 TB/s over 10 CTAs
        // with 10 vectors per thread, 5.51 over 16 with 7; between 10 and 16 nothing beat 16 where 10 is too few)
        if (th == 256 && allow_wide_cluster && oe) {
            for (int c = 10; c <= 16; c += 6) {
                const int need = (per_cta_vectors(nvec, c) + th - 1) / th;
                if (need <= 10) {
                    *out = {c, th, round_nv(need), oe};
                    return true;
                }
            }
        }
    }
    return false;
}

typedef void (*FastKernel)(const FastParams);

// the row kernel's instantiation for a launch shape: vectors per thread (1 .. 10) and the
// variant flags (one exponential per element, entropy output, skip-masked row list, per-token weights)
template <int THREADS, bool ONE_EXP, bool ENT = false, bool SKIP = false, bool WT = false>
static FastKernel row_kernel_for_nv(int nv) {
    switch (nv) {
        case 1: return grpo_row_cluster_kernel<THREADS, 1, ONE_EXP, ENT, SKIP, WT>;
        case 2: return grpo_row_cluster_kernel<THREADS, 2, ONE_EXP, ENT, SKIP, WT>;
        case 3: return grpo_row_cluster_kernel<THREADS, 3, ONE_EXP, ENT, SKIP, WT>;
        case 4: return grpo_row_cluster_kernel<THREADS, 4, ONE_EXP, ENT, SKIP, WT>;
        case 5: return grpo_row_cluster_kernel<THREADS, 5, ONE_EXP, ENT, SKIP, WT>;
        case 6: return grpo_row_cluster_kernel<THREADS, 6, ONE_EXP, ENT, SKIP, WT>;
        case 7: return grpo_row_cluster_kernel<THREADS, 7, ONE_EXP, ENT, SKIP, WT>;
        case 8: return grpo_row_cluster_kernel<THREADS, 8, ONE_EXP, ENT, SKIP, WT>;
        case 9: return grpo_row_cluster_kernel<THREADS, 9, ONE_EXP, ENT, SKIP, WT>;
        case 10: return grpo_row_cluster_kernel<THREADS, 10, ONE_EXP, ENT, SKIP, WT>;
    }
    return nullptr;
}
// the training kernels for clusters of 9 to 16 CTAs of 256 threads (rows beyond 8 x 256 x 10 vectors):
// plain, skip-masked and weighted variants, one exponential per element
template <bool SKIP = false, bool WT = false>
static FastKernel wide_cluster_kernel(int nv) {
    switch (nv) {
        case 6: return grpo_row_cluster_kernel<256, 6, true, false, SKIP, WT, 16>;
        case 7: return grpo_row_cluster_kernel<256, 7, true, false, SKIP, WT, 16>;
        case 8: return grpo_row_cluster_kernel<256, 8, true, false, SKIP, WT, 16>;
        case 9: return grpo_row_cluster_kernel<256, 9, true, false, SKIP, WT, 16>;
        case 10: return grpo_row_cluster_kernel<256, 10, true, false, SKIP, WT, 16>;
    }
    return nullptr;
}
// ... for a thread count known at run time
template <bool ONE_EXP, bool ENT = false, bool SKIP = false, bool WT = false>
static FastKernel row_kernel_for(int threads, int nv) {
    if (threads == 256) return row_kernel_for_nv<256, ONE_EXP, ENT, SKIP, WT>(nv);
    if (threads == 512) return row_kernel_for_nv<512, ONE_EXP, ENT, SKIP, WT>(nv);
    if (threads == 1024) return row_kernel_for_nv<1024, ONE_EXP, ENT, SKIP, WT>(nv);
    return nullptr;
}
static FastKernel weighted_kernel(const FastShape& sh) {
    if (sh.cluster > 8) return wide_cluster_kernel<false, true>(sh.nv);
    return row_kernel_for<true, false, false, true>(sh.threads, sh.nv);
}
static FastKernel skip_kernel(const FastShape& sh) {
    if (sh.cluster > 8) return wide_cluster_kernel<true, false>(sh.nv);
    return row_kernel_for<true, false, true>(sh.threads, sh.nv);
}
static FastKernel fast_kernel(const FastShape& sh) {
    if (sh.cluster > 8) return wide_cluster_kernel<>(sh.nv);
    return sh.one_exp ? row_kernel_for<true>(sh.threads, sh.nv) : row_kernel_for<false>(sh.threads, sh.nv);
}

static int sm_count() {
    static std::atomic<int> n{0};
    if (n.load() == 0) {
        int dev = 0, v = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        n = v > 0 ? v : 148;
    }
    return n.load();
}

static void cluster_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* at, int grid, const FastShape& sh,
                           cudaStream_t s) {
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3(grid);
    cfg->blockDim = dim3(sh.threads);
    cfg->dynamicSmemBytes = (size_t)stage_bytes(sh.threads, sh.nv);
    cfg->stream = s;
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = sh.cluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg->attrs = at;
    cfg->numAttrs = 1;
}

// how many clusters of this shape can be resident at once; also opts the kernel in to its staging
// buffer.  Cached per device, kernel and cluster size.
static int max_clusters(FastKernel k, const FastShape& sh) {
    static std::mutex mu;
    static struct { int dev; FastKernel k; int cluster; int n; } cache[128];
    static int ncache = 0;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < ncache; ++i)
        if (cache[i].dev == dev && cache[i].k == k && cache[i].cluster == sh.cluster) return cache[i].n;
    if (cudaFuncSetAttribute((const void*)k, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             stage_bytes(sh.threads, sh.nv)) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    if (sh.cluster > 8 &&
        cudaFuncSetAttribute((const void*)k, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute at[1];
    cluster_config(&cfg, at, sh.cluster * sm_count() * 8, sh, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, (void*)k, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return -1;
    }
    if (ncache < 128) cache[ncache++] = {dev, k, sh.cluster, n};
    return n;
}

// Clusters to launch for `rows` rows.  At least as many as fit on the device at once; beyond that,
// enough that a cluster handles only a couple of dozen rows before it retires and the hardware
// scheduler starts the next one, in whole generations (multiples of what fits at once).  With exactly
// one resident generation of persistent clusters, all of them load, then all of them store, in step
// for the whole launch, and the memory system sees the traffic in synchronised bursts; short-lived
// clusters drift apart.  Measured on one GPU (copy rate 6.5 TB/s), TB/s by rows per cluster:
//   32768 rows, 100 launches each:  one generation 5.87;  56: 6.14;  40: 6.20;  28: 6.14;  16: 6.15;  8: 6.07
//   133010 rows in place:           one generation 5.83;  112: 6.50;  28: 6.62;  14: 6.67;  7: 6.61
//   8192 rows:                      one generation 5.66;  56: 5.88;  28: 6.12;  14: 6.16;  7: 6.15
// and one row per cluster 4.99 (start-up and the two cluster barriers of every cluster dominate).
// A plain copy written the same way shows the same: persistent CTAs 6.1 TB/s, one CTA per 40 KB unit 6.9.
constexpr int kRowsPerCluster = 24;
static int clusters_for(int resident, int64_t rows) {
    const int rpc = g_rows_per_cluster.load() > 0 ? g_rows_per_cluster.load() : kRowsPerCluster;
    // whole generations: a multiple of what fits at once
    const int64_t per_generation = (int64_t)resident * rpc;
    int64_t nc = (rows + per_generation - 1) / per_generation * resident;
    if (nc > rows) nc = rows;
    if (nc > (1 << 26)) nc = 1 << 26;          // grid.x stays far below 2^31 - 1 for any cluster size
    return (int)nc;
}

// CTAs of the general (one CTA per row) kernel: a few rows per CTA, for the same reason
static int general_grid(int64_t rows) {
    int64_t g = (rows + 3) / 4;
    if (g < (int64_t)sm_count() * 8) g = (int64_t)sm_count() * 8;
    if (g > rows) g = rows;
    if (g > (1 << 30)) g = 1 << 30;
    return (int)g;
}

struct LossArgs {
    const void* logits;
    void* grad;
    rlf_dtype dt;
    int64_t T;
    int32_t V;
    int64_t stride;
    const int32_t* ids;
    const int32_t* seq_id;
    const float* adv;
    int32_t B;
    const float* old_logp;
    const float* ref_logp;
    const uint8_t* mask;
    float eps_clip, beta;
    float eps_hi;               // upper clip width (the lower one is eps_clip)
    int aggregation;            // 0 token mean, 1 sequence mean (per-token weights built in the workspace)
    const int64_t* denom;
    float* logp_out;
    double* loss_out;
    int32_t* dev_status;
};

// sequence-mean aggregation: w_t = live_t / (n_b * S), n_b = live tokens of the token's sequence,
// S = *denom if given else the number of sequences with n_b > 0
__global__ void __launch_bounds__(256)
seq_count_kernel(const float4* __restrict__ rec, const int32_t* __restrict__ seq_id, int64_t T, int* __restrict__ cnt) {
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t < T && __float_as_int(rec[t].w) < 0) atomicAdd(&cnt[seq_id[t]], 1);
}
__global__ void __launch_bounds__(1024)
seq_live_kernel(const int* __restrict__ cnt, int32_t B, const long long* __restrict__ denom, long long* __restrict__ s_out) {
    __shared__ int red[32];
    int c = 0;
    for (int b = threadIdx.x; b < B; b += 1024) c += cnt[b] > 0 ? 1 : 0;
    c = __reduce_add_sync(0xffffffffu, c);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int w = 0; w < 32; ++w) s += red[w];
        *s_out = denom ? *denom : (long long)s;
    }
}
__global__ void __launch_bounds__(256)
seq_weight_kernel(const float4* __restrict__ rec, const int32_t* __restrict__ seq_id, int64_t T,
                  const int* __restrict__ cnt, const long long* __restrict__ s_in, float* __restrict__ wtok) {
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= T) return;
    float w = 0.0f;
    if (__float_as_int(rec[t].w) < 0) {
        const long long S = *s_in;
        w = (float)(1.0 / ((double)cnt[seq_id[t]] * (double)(S > 1 ? S : 1)));
    }
    wtok[t] = w;
}

static rlf_status launch_logits_loss(const LossArgs& a, bool fast_ok, void* workspace, cudaStream_t s) {
    char* ws = static_cast<char*>(workspace);
    long long* n_count = reinterpret_cast<long long*>(ws);
    double* partial = reinterpret_cast<double*>(ws + kWsPartialOff);
    float4* rec = reinterpret_cast<float4*>(ws + kWsRecordOff);
    const long long* denom = reinterpret_cast<const long long*>(a.denom);
    if (denom == nullptr) {
        if (cudaMemsetAsync(n_count, 0, sizeof(long long), s) != cudaSuccess) return RLF_ERR_CUDA;
        denom = n_count;
    }
    int num_partials = 0;
    float* wtok = nullptr;
    if (a.T > 0) {
        const int64_t prep_blocks = (a.T + kPrepThreads - 1) / kPrepThreads;
        token_prep_kernel<<<(unsigned)prep_blocks, kPrepThreads, 0, s>>>(
            a.ids, a.seq_id, a.adv, a.old_logp, a.ref_logp, a.mask, a.T, a.V, a.B, rec,
            a.denom == nullptr ? reinterpret_cast<unsigned long long*>(n_count) : nullptr, a.dev_status);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
        if (a.aggregation == 1) {
            // per-token weights of the sequence mean; here `denom`, if given, counts sequences
            int* cnt = reinterpret_cast<int*>(ws + ws_seqcnt_off(a.T));
            long long* s_slot = reinterpret_cast<long long*>(ws + 64);
            wtok = reinterpret_cast<float*>(ws + ws_wtok_off(a.T));
            if (cudaMemsetAsync(cnt, 0, sizeof(int) * (size_t)a.B, s) != cudaSuccess) return RLF_ERR_CUDA;
            seq_count_kernel<<<(unsigned)prep_blocks, 256, 0, s>>>(rec, a.seq_id, a.T, cnt);
            seq_live_kernel<<<1, 1024, 0, s>>>(cnt, a.B, reinterpret_cast<const long long*>(a.denom), s_slot);
            seq_weight_kernel<<<(unsigned)prep_blocks, 256, 0, s>>>(rec, a.seq_id, a.T, cnt, s_slot, wtok);
            count_launch(3);
            if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
        }

        FastShape sh;
        const bool tuned = g_tune_cluster.load() > 0;
        if (fast_ok && a.T < (1ll << 31) && pick_shape(a.V >> 3, &sh, /*allow_wide_cluster=*/true)) {
            FastKernel k = wtok ? weighted_kernel(sh) : fast_kernel(sh);
            int nc = k ? max_clusters(k, sh) : -1;
            if (nc <= 0 && sh.cluster > 8 && !tuned && pick_shape(a.V >> 3, &sh)) {
                // the device does not take a cluster of 16: the portable shape instead
                k = wtok ? weighted_kernel(sh) : fast_kernel(sh);
                nc = k ? max_clusters(k, sh) : -1;
            }
            if (!k) return RLF_ERR_UNSUPPORTED;
            if (nc <= 0) return RLF_ERR_UNSUPPORTED;      // this shape does not fit on the device
            nc = clusters_for(nc, a.T);
            FastParams p;
            p.logits = static_cast<const __nv_bfloat16*>(a.logits);
            p.grad = static_cast<__nv_bfloat16*>(a.grad);
            p.stride = a.stride;
            p.T = (int)a.T;
            p.nvec = a.V >> 3;
            p.per_cta_vec = per_cta_vectors(p.nvec, sh.cluster);
            p.rec = rec;
            p.denom = denom;
            p.logp_out = a.logp_out;
            p.dev_status = a.dev_status;
            p.eps_clip = a.eps_clip;
            p.eps_hi = a.eps_hi;
            p.beta = a.beta;
            p.wtok = wtok;
            p.entropy_out = nullptr;
            p.row_list = nullptr;
            p.n_rows = nullptr;
            cudaLaunchConfig_t cfg;
            cudaLaunchAttribute at[1];
            cluster_config(&cfg, at, nc * sh.cluster, sh, s);
            if (cudaLaunchKernelEx(&cfg, k, p) != cudaSuccess) {
                cudaGetLastError();
                return RLF_ERR_CUDA;
            }
            count_launch();
        } else if (fast_ok && tuned) {
            return RLF_ERR_UNSUPPORTED;
        } else {
            GenParams p;
            p.logits = a.logits; p.grad = a.grad; p.stride = a.stride; p.T = a.T; p.V = a.V;
            p.rec = rec; p.denom = denom; p.logp_out = a.logp_out; p.dev_status = a.dev_status;
            p.eps_clip = a.eps_clip; p.eps_hi = a.eps_hi; p.beta = a.beta; p.entropy_out = nullptr; p.fwd_only = 0;
            p.wtok = wtok;
            int grid = general_grid(a.T);
            if (a.dt == RLF_BF16) grpo_row_general_kernel<__nv_bfloat16><<<grid, kGenThreads, 0, s>>>(p);
            else grpo_row_general_kernel<float><<<grid, kGenThreads, 0, s>>>(p);
            count_launch();
            if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
        }
        const int64_t blocks = (a.T + kLossThreads - 1) / kLossThreads;
        num_partials = (int)(blocks < kMaxPartials ? blocks : kMaxPartials);
        token_loss_kernel<<<num_partials, kLossThreads, 0, s>>>(a.logp_out, rec, a.T, a.eps_clip, a.eps_hi, wtok, partial);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    }
    finalize_loss_kernel<<<1, 96, 0, s>>>(partial, num_partials, denom, a.beta, wtok != nullptr, a.loss_out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

}  // namespace rlf

extern "C" rlf_status rlf_tune_logits_kernel(int cluster_ctas, int threads_per_cta, int one_exp) {
    rlf::g_tune_one_exp = one_exp;
    if (cluster_ctas == 0 || threads_per_cta == 0) {
        rlf::g_tune_cluster = 0;
        rlf::g_tune_threads = 0;
        return RLF_OK;
    }
    const bool c_ok = cluster_ctas >= 1 && cluster_ctas <= 16;
    const bool t_ok = threads_per_cta == 256 || threads_per_cta == 512 || threads_per_cta == 1024;
    if (!c_ok || !t_ok) return RLF_ERR_SHAPE;
    rlf::g_tune_cluster = cluster_ctas;
    rlf::g_tune_threads = threads_per_cta;
    return RLF_OK;
}

extern "C" rlf_status rlf_tune_logits_grid(int rows_per_cluster, int units_per_cta) {
    if (rows_per_cluster < 0 || units_per_cta < 0) return RLF_ERR_SHAPE;
    rlf::g_rows_per_cluster = rows_per_cluster;
    rlf::g_units_per_cta = units_per_cta;
    return RLF_OK;
}

extern "C" rlf_status rlf_grpo_logp_loss_fwd_bwd(
    const void* logits, rlf_dtype dt, int64_t T, int32_t V, int64_t row_stride, const int32_t* ids,
    const int32_t* seq_id, const float* adv, int32_t B, const float* old_logp, const float* ref_logp,
    const uint8_t* mask, float eps_clip, float beta_kl, const int64_t* denom, float* logp_out,
    double* loss_out, void* grad_logits, void* workspace, size_t workspace_bytes,
    int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (dt != RLF_BF16 && dt != RLF_F32) return RLF_ERR_DTYPE;
    if (T < 0 || V < 1 || B < 0 || row_stride < V) return RLF_ERR_SHAPE;
    if (!loss_out) return RLF_ERR_NULL;
    if (T > 0 && (!logits || !ids || !seq_id || !adv || !old_logp || !ref_logp || !mask || !logp_out))
        return RLF_ERR_NULL;
    if (T > 0 && B == 0) return RLF_ERR_SHAPE;
    const size_t esz = dt == RLF_BF16 ? 2 : 4;
    if (!aligned(logits, esz) || !aligned(grad_logits, esz)) return RLF_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < loss_workspace_bytes(T))
        return RLF_ERR_WORKSPACE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;

    LossArgs a;
    a.logits = logits; a.grad = grad_logits; a.dt = dt; a.T = T; a.V = V; a.stride = row_stride;
    a.ids = ids; a.seq_id = seq_id; a.adv = adv; a.B = B; a.old_logp = old_logp; a.ref_logp = ref_logp;
    a.mask = mask; a.eps_clip = eps_clip; a.beta = beta_kl; a.denom = denom; a.logp_out = logp_out;
    a.loss_out = loss_out; a.dev_status = dev_status;
    a.eps_hi = eps_clip; a.aggregation = 0;
    const bool fast_ok = dt == RLF_BF16 && (V % 8 == 0) && (row_stride % 8 == 0) &&
                         aligned(logits, 16) && aligned(grad_logits, 16);
    return launch_logits_loss(a, fast_ok, workspace, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" rlf_status rlf_grpo_logp_loss_fwd_bwd_obj(
    const void* logits, rlf_dtype dt, int64_t T, int32_t V, int64_t row_stride, const int32_t* ids,
    const int32_t* seq_id, const float* adv, int32_t B, const float* old_logp, const float* ref_logp,
    const uint8_t* mask, float eps_clip_low, float eps_clip_high, float beta_kl, int aggregation,
    const int64_t* denom, float* logp_out, double* loss_out, void* grad_logits, void* workspace,
    size_t workspace_bytes, int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (dt != RLF_BF16 && dt != RLF_F32) return RLF_ERR_DTYPE;
    if (T < 0 || V < 1 || B < 0 || row_stride < V) return RLF_ERR_SHAPE;
    if (aggregation != 0 && aggregation != 1) return RLF_ERR_SHAPE;
    if (aggregation == 1 && (int64_t)B > T + 1) return RLF_ERR_SHAPE;
    if (!loss_out) return RLF_ERR_NULL;
    if (T > 0 && (!logits || !ids || !seq_id || !adv || !old_logp || !ref_logp || !mask || !logp_out))
        return RLF_ERR_NULL;
    if (T > 0 && B == 0) return RLF_ERR_SHAPE;
    const size_t esz = dt == RLF_BF16 ? 2 : 4;
    if (!aligned(logits, esz) || !aligned(grad_logits, esz)) return RLF_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < loss_workspace_bytes(T))
        return RLF_ERR_WORKSPACE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    LossArgs a;
    a.logits = logits; a.grad = grad_logits; a.dt = dt; a.T = T; a.V = V; a.stride = row_stride;
    a.ids = ids; a.seq_id = seq_id; a.adv = adv; a.B = B; a.old_logp = old_logp; a.ref_logp = ref_logp;
    a.mask = mask; a.eps_clip = eps_clip_low; a.beta = beta_kl; a.denom = denom; a.logp_out = logp_out;
    a.loss_out = loss_out; a.dev_status = dev_status;
    a.eps_hi = eps_clip_high; a.aggregation = aggregation;
    const bool fast_ok = dt == RLF_BF16 && (V % 8 == 0) && (row_stride % 8 == 0) &&
                         aligned(logits, 16) && aligned(grad_logits, 16);
    return launch_logits_loss(a, fast_ok, workspace, reinterpret_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------
// Forward-only log-prob (+ entropy) of given target ids: the pass that produces old_logp / ref_logp.
namespace rlf {

__global__ void __launch_bounds__(256)
ids_to_record_kernel(const int32_t* __restrict__ ids, int64_t T, int32_t V, float4* __restrict__ rec,
                     long long* __restrict__ one, int32_t* __restrict__ dev_status) {
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t == 0) *one = 1;                       // the row kernels read a denominator; unused here
    if (t >= T) return;
    int32_t y = ids[t];
    const bool bad = y < 0 || y >= V;
    if (bad) {
        y = 0;
        if (dev_status) atomicOr(dev_status, RLF_DEV_BAD_TARGET);
    }
    rec[t] = make_float4(0.0f, 0.0f, 0.0f, __int_as_float(bad ? y : (y | (int)0x80000000)));
}

// Streaming form of the forward-only pass.  Log-sum-exp statistics are associative, so a row need not
// be owned by anyone: a work unit is one CHUNK of one row (up to 256 x 10 vectors), every WARP turns
// its share of a unit into a partial (max, sum 2^x, sum 2^x x) in global memory and a second kernel
// merges the partials of a row and gathers the target logit.  No cluster, no exchange and no CTA
// barrier: a thread only ever reads the staging slots it filled itself (cp.async, refilled with the
// CTA's next unit as soon as they are in registers), so the warps of a CTA drift freely and the
// exponential unit, the busiest pipe of this pass, is kept fed while other warps wait on loads.
constexpr int kStreamThreads = 256;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kStreamNV = 10;
constexpr int kStreamCtasPerSm = 4;
constexpr int kStreamUnitsPerCta = 8;     // units a CTA handles before it retires (when there are that many)

// Packed fp32 pairs (one instruction, two lanes of arithmetic): with one instruction per element
// for each of the multiply-adds around the exponential the pass is bound by instruction issue.
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
constexpr uint32_t kFloorPair = 0xFE96FE96u;   // two bf16 -9.97e37: keeps x finite, so that 2^x * x is 0, not NaN

// (sum 2^x, sum 2^x x) with x = z log2e + off over this thread's registers; WANT_U = false drops the
// second sum.  Only for moderate |max| (the caller takes the subtract-first form otherwise).
template <int NV, bool WANT_U>
__device__ __forceinline__ float2 stream_exp_pass(const uint4 (&d)[NV], float off) {
    const uint64_t c2 = f32x2(kLog2e, kLog2e), off2 = f32x2(off, off);
    uint64_t s2a = 0, s2b = 0, u2a = 0, u2b = 0;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const uint32_t w[4] = {d[i].x, d[i].y, d[i].z, d[i].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t wc = WANT_U ? max_bf16x2(w[k], kFloorPair) : w[k];
            const uint64_t x2 = fma_f32x2(f32x2(bf_lo(wc), bf_hi(wc)), c2, off2);
            float x0, x1;
            f32x2_split(x2, x0, x1);
            const uint64_t e2 = f32x2(ex2_approx(x0), ex2_approx(x1));
            if (k & 1) {
                s2b = add_f32x2(s2b, e2);
                if (WANT_U) u2b = fma_f32x2(e2, x2, u2b);
            } else {
                s2a = add_f32x2(s2a, e2);
                if (WANT_U) u2a = fma_f32x2(e2, x2, u2a);
            }
        }
    }
    float a, b, c, e;
    f32x2_split(add_f32x2(s2a, s2b), a, b);
    f32x2_split(add_f32x2(u2a, u2b), c, e);
    return make_float2(a + b, c + e);
}

struct StreamParams {
    const __nv_bfloat16* logits;
    long long stride;
    long long units;            // T * chunks
    int chunks;                 // chunks per row
    int per_chunk_vec;          // vectors per chunk (the last chunk of a row may hold fewer)
    int nvec;                   // V / 8
    float4* partial;            // [units][kStreamWarps] (max, sum, usum, -)
};

template <bool WANT_U, int NV>
__global__ void __launch_bounds__(kStreamThreads, kStreamCtasPerSm)
logp_entropy_stream_kernel(const StreamParams p) {
    constexpr int THREADS = kStreamThreads;
    extern __shared__ __align__(16) uint4 stage[];      // [NV][THREADS], slot (i, tid) private to thread tid
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    auto unit_geometry = [&](long long u, const uint4*& src, int& nvalid) {
        const long long row = u / p.chunks;
        const int chunk = (int)(u - row * p.chunks);
        const int vbeg = chunk * p.per_chunk_vec + tid;
        const int vend = min(p.nvec, (chunk + 1) * p.per_chunk_vec);
        nvalid = vend > vbeg ? min(NV, (vend - vbeg + THREADS - 1) / THREADS) : 0;
        src = reinterpret_cast<const uint4*>(p.logits + row * p.stride) + vbeg;
    };
    auto prefetch = [&](long long u) {
        if (u < p.units) {
            const uint4* src;
            int nvalid;
            unit_geometry(u, src, nvalid);
#pragma unroll
            for (int i = 0; i < NV; ++i)
                if (i < nvalid) cp_async16_cg(stage + i * THREADS + tid, src + i * THREADS);
        }
        cp_async_commit();
    };

    prefetch(blockIdx.x);
    for (long long u = blockIdx.x; u < p.units; u += gridDim.x) {
        const uint4* src_unused;
        int nvalid;
        unit_geometry(u, src_unused, nvalid);
        cp_async_wait_all();
        uint4 d[NV];
        if (nvalid == NV) {
#pragma unroll
            for (int i = 0; i < NV; ++i) d[i] = stage[i * THREADS + tid];
        } else {
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                if (i < nvalid) d[i] = stage[i * THREADS + tid];
                else d[i] = make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);
            }
        }
        prefetch(u + gridDim.x);          // the slots are in registers: refill them with the next unit
        uint32_t mx = kNegInfPair;
#pragma unroll
        for (int i = 0; i < NV; ++i)
            mx = max_bf16x2(mx, max_bf16x2(max_bf16x2(d[i].x, d[i].y), max_bf16x2(d[i].z, d[i].w)));
        float m_w = fmaxf(bf_lo(mx), bf_hi(mx));
        m_w = ord2f(__reduce_max_sync(0xffffffffu, f2ord(m_w)));
        const float m_ws = (m_w == -INFINITY) ? 0.0f : m_w;
        const float2 su = fabsf(m_ws) > kRobustAbove ? exp_sum_ent_pass<NV, true>(d, m_ws, 0.0f)
                                                     : stream_exp_pass<NV, WANT_U>(d, -m_ws * kLog2e);
        const float s_w = warp_sum(su.x), u_w = WANT_U ? warp_sum(su.y) : 0.0f;
        if (lane == 0) p.partial[u * kStreamWarps + warp] = make_float4(m_w, s_w, u_w, 0.0f);
    }
    cp_async_wait_all();
}

// merge the warp partials of every row: one warp per row
__global__ void __launch_bounds__(256)
logp_entropy_merge_kernel(const float4* __restrict__ partial, int per_row, const __nv_bfloat16* __restrict__ logits,
                          long long stride, const int32_t* __restrict__ ids, int64_t T, int32_t V,
                          float* __restrict__ logp_out, float* __restrict__ entropy_out,
                          int32_t* __restrict__ dev_status) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    const float4* row = partial + t * per_row;
    float M = -INFINITY;
    for (int c = lane; c < per_row; c += 32) M = fmaxf(M, row[c].x);
    M = ord2f(__reduce_max_sync(0xffffffffu, f2ord(M)));
    float S = 0.0f, U = 0.0f;
    for (int c = lane; c < per_row; c += 32) {
        const float4 e = row[c];
        if (e.x == -INFINITY) continue;
        const float dx = (e.x - M) * kLog2e;
        const float f = ex2_approx(dx);
        S += e.y * f;
        if (f > 0.0f) U += f * fmaf(e.y, dx, e.z);
    }
    S = warp_sum(S);
    U = warp_sum(U);
    if (lane != 0) return;
    const int32_t y = ids[t];
    const bool bad = y < 0 || y >= V;
    const float zy = bad ? 0.0f : __bfloat162float(logits[t * stride + y]);
    const float lg2s = lg2_approx(S);
    const float logp = (zy - M) - lg2s * kLn2;
    const bool finite = (M > -INFINITY) && (M < INFINITY) && (S > 0.0f) && (S < INFINITY) && (fabsf(logp) < INFINITY);
    const float nan = __int_as_float(0x7fc00000);
    logp_out[t] = (finite && !bad) ? logp : nan;
    if (entropy_out) entropy_out[t] = finite ? (lg2s - U / S) * kLn2 : nan;
    const int st = (bad ? RLF_DEV_BAD_TARGET : 0) | (finite ? 0 : RLF_DEV_NONFINITE);
    if (st && dev_status) atomicOr(dev_status, st);
}

// Vectors per thread of a unit.  A row is cut into equal chunks of at most 256 x NV vectors; with NV = 10
// a row of 1024 vectors (V = 8192) would fill 40 % of its unit's staging slots and leave the rest of the
// in-flight capacity unused.  The largest NV among 10, 8, 6, 5, 4 that fills at least 85 % of the slots
// is taken (large units have the least per-unit overhead), else the one that fills the most.
static int stream_nv(int nvec) {
    static const int choices[] = {10, 8, 6, 5, 4};
    int best = kStreamNV;
    double best_fill = -1.0;
    for (int nv : choices) {
        const int chunks = (nvec + kStreamThreads * nv - 1) / (kStreamThreads * nv);
        const double fill = (double)nvec / ((double)chunks * kStreamThreads * nv);
        if (fill >= 0.85) return nv;
        if (fill > best_fill) { best_fill = fill; best = nv; }
    }
    return best;
}
static int stream_chunks(int nvec) {
    const int nv = stream_nv(nvec);
    return (nvec + kStreamThreads * nv - 1) / (kStreamThreads * nv);
}
size_t entropy_workspace_bytes(int64_t T, int32_t V) {
    const size_t chunks = V >= 8 ? (size_t)stream_chunks(V >> 3) : 1;
    return loss_workspace_bytes(T) + 16 * ws_tokens(T) * chunks * kStreamWarps + 256;
}


}  // namespace rlf

extern "C" rlf_status rlf_logp_entropy_fwd(const void* logits, rlf_dtype dt, int64_t T, int32_t V,
                                           int64_t row_stride, const int32_t* ids, float* logp_out,
                                           float* entropy_out, void* workspace, size_t workspace_bytes,
                                           int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (dt != RLF_BF16 && dt != RLF_F32) return RLF_ERR_DTYPE;
    if (T < 0 || V < 1 || row_stride < V) return RLF_ERR_SHAPE;
    if (T == 0) return RLF_OK;
    if (!logits || !ids || !logp_out) return RLF_ERR_NULL;
    const size_t esz = dt == RLF_BF16 ? 2 : 4;
    if (!aligned(logits, esz)) return RLF_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < loss_workspace_bytes(T)) return RLF_ERR_WORKSPACE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    const bool fast_ok = dt == RLF_BF16 && (V % 8 == 0) && (row_stride % 8 == 0) && aligned(logits, 16) &&
                         T < (1ll << 30);
    if (fast_ok && workspace_bytes >= entropy_workspace_bytes(T, V)) {
        // streaming form: chunk partials, then a per-row merge
        const int snv = stream_nv(V >> 3);
        const int smem = snv * kStreamThreads * 16;         // at most 40 KB: below the default dynamic limit
        StreamParams sp;
        sp.logits = static_cast<const __nv_bfloat16*>(logits);
        sp.stride = row_stride;
        sp.nvec = V >> 3;
        sp.chunks = stream_chunks(sp.nvec);
        sp.per_chunk_vec = (sp.nvec + sp.chunks - 1) / sp.chunks;
        sp.units = (long long)T * sp.chunks;
        sp.partial = reinterpret_cast<float4*>(ws + ((loss_workspace_bytes(T) + 255) & ~(size_t)255));
        // as for the row kernel: CTAs that retire after a few units instead of one resident generation
        const int upc = g_units_per_cta.load() > 0 ? g_units_per_cta.load() : kStreamUnitsPerCta;
        long long grid = (long long)sm_count() * kStreamCtasPerSm;
        if ((sp.units + upc - 1) / upc > grid) grid = (sp.units + upc - 1) / upc;
        if (grid > sp.units) grid = sp.units;
        if (grid > (1ll << 30)) grid = 1ll << 30;
        auto launch = [&](auto want_u) {
            constexpr bool U = decltype(want_u)::value;
            switch (snv) {
                case 4: logp_entropy_stream_kernel<U, 4><<<(unsigned)grid, kStreamThreads, smem, s>>>(sp); break;
                case 5: logp_entropy_stream_kernel<U, 5><<<(unsigned)grid, kStreamThreads, smem, s>>>(sp); break;
                case 6: logp_entropy_stream_kernel<U, 6><<<(unsigned)grid, kStreamThreads, smem, s>>>(sp); break;
                case 8: logp_entropy_stream_kernel<U, 8><<<(unsigned)grid, kStreamThreads, smem, s>>>(sp); break;
                default: logp_entropy_stream_kernel<U, 10><<<(unsigned)grid, kStreamThreads, smem, s>>>(sp); break;
            }
        };
        if (entropy_out) launch(std::true_type{});
        else launch(std::false_type{});
        logp_entropy_merge_kernel<<<(unsigned)((T + 7) / 8), 256, 0, s>>>(
            sp.partial, sp.chunks * kStreamWarps, sp.logits, row_stride, ids, T, V, logp_out, entropy_out, dev_status);
        count_launch(2);
        return cuda_ok(cudaGetLastError());
    }
    long long* one = reinterpret_cast<long long*>(ws);
    float4* rec = reinterpret_cast<float4*>(ws + kWsRecordOff);
    ids_to_record_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(ids, T, V, rec, one, dev_status);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;

    FastShape sh;
    if (fast_ok && pick_shape(V >> 3, &sh)) {
        FastKernel k = row_kernel_for<false, true>(sh.threads, sh.nv);
        if (!k) return RLF_ERR_UNSUPPORTED;
        int nc = max_clusters(k, sh);
        if (nc <= 0) return RLF_ERR_UNSUPPORTED;
        nc = clusters_for(nc, T);
        FastParams p;
        p.logits = static_cast<const __nv_bfloat16*>(logits);
        p.grad = nullptr;
        p.stride = row_stride;
        p.T = (int)T;
        p.nvec = V >> 3;
        p.per_cta_vec = per_cta_vectors(p.nvec, sh.cluster);
        p.rec = rec;
        p.denom = one;
        p.logp_out = logp_out;
        p.entropy_out = entropy_out;
        p.row_list = nullptr;
        p.n_rows = nullptr;
        p.dev_status = dev_status;
        p.eps_clip = 0.0f;
        p.eps_hi = 0.0f;
        p.wtok = nullptr;
        p.beta = 0.0f;
        cudaLaunchConfig_t cfg;
        cudaLaunchAttribute at[1];
        cluster_config(&cfg, at, nc * sh.cluster, sh, s);
        if (cudaLaunchKernelEx(&cfg, k, p) != cudaSuccess) {
            cudaGetLastError();
            return RLF_ERR_CUDA;
        }
        count_launch();
        return RLF_OK;
    }
    GenParams g;
    g.logits = logits; g.grad = nullptr; g.stride = row_stride; g.T = T; g.V = V; g.rec = rec; g.denom = one;
    g.logp_out = logp_out; g.entropy_out = entropy_out; g.dev_status = dev_status; g.eps_clip = 0.0f; g.beta = 0.0f;
    g.eps_hi = 0.0f; g.wtok = nullptr;
    g.fwd_only = 1;
    int grid = general_grid(T);
    if (dt == RLF_BF16) grpo_row_general_kernel<__nv_bfloat16><<<grid, kGenThreads, 0, s>>>(g);
    else grpo_row_general_kernel<float><<<grid, kGenThreads, 0, s>>>(g);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Skip-masked variant: rows with zero loss weight are neither read nor computed.
namespace rlf {

// live rows (record's live bit) -> compacted list of row indices and of their records, in arbitrary
// order (rows are independent, so the order does not affect any result)
__global__ void __launch_bounds__(256)
compact_live_kernel(const float4* __restrict__ rec, int64_t T, int* __restrict__ row_list,
                    float4* __restrict__ rec_c, int* __restrict__ counter) {
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    bool live = false;
    if (t < T) {
        r = rec[t];
        live = __float_as_int(r.w) < 0;
    }
    const unsigned m = __ballot_sync(0xffffffffu, live);
    if (m == 0) return;
    const int lane = threadIdx.x & 31;
    int base = 0;
    if (lane == 0) base = atomicAdd(counter, __popc(m));
    base = __shfl_sync(0xffffffffu, base, 0);
    if (live) {
        const int k = base + __popc(m & ((1u << lane) - 1u));
        row_list[k] = (int)t;
        rec_c[k] = r;
    }
}

// rows that are not live: log-prob NaN and (optionally) an all-zero gradient row
template <typename T>
__global__ void __launch_bounds__(256)
fill_dead_rows_kernel(const float4* __restrict__ rec, int64_t Tn, int32_t V, long long stride, T* __restrict__ grad,
                      int zero_grad, float* __restrict__ logp_out) {
    for (int64_t row = blockIdx.x; row < Tn; row += gridDim.x) {
        if (__float_as_int(rec[row].w) < 0) continue;
        if (threadIdx.x == 0) logp_out[row] = __int_as_float(0x7fc00000);
        if (grad == nullptr || !zero_grad) continue;
        T* g = grad + row * stride;
        const bool vec = (sizeof(T) * V) % 16 == 0 && (reinterpret_cast<uintptr_t>(g) % 16) == 0;
        if (vec) {
            uint4* g4 = reinterpret_cast<uint4*>(g);
            const int n4 = (int)(sizeof(T) * V / 16);
            for (int i = threadIdx.x; i < n4; i += 256) st_stream(g4 + i, make_uint4(0u, 0u, 0u, 0u));
        } else {
            for (int v = threadIdx.x; v < V; v += 256) g[v] = from_f32<T>(0.0f);
        }
    }
}


}  // namespace rlf

extern "C" rlf_status rlf_grpo_logp_loss_fwd_bwd_skip_masked(
    const void* logits, rlf_dtype dt, int64_t T, int32_t V, int64_t row_stride, const int32_t* ids,
    const int32_t* seq_id, const float* adv, int32_t B, const float* old_logp, const float* ref_logp,
    const uint8_t* mask, float eps_clip, float beta_kl, const int64_t* denom, float* logp_out,
    double* loss_out, void* grad_logits, int zero_masked_grad, void* workspace, size_t workspace_bytes,
    int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (dt != RLF_BF16 && dt != RLF_F32) return RLF_ERR_DTYPE;
    if (T < 0 || V < 1 || B < 0 || row_stride < V) return RLF_ERR_SHAPE;
    if (!loss_out) return RLF_ERR_NULL;
    if (T > 0 && (!logits || !ids || !seq_id || !adv || !old_logp || !ref_logp || !mask || !logp_out))
        return RLF_ERR_NULL;
    if (T > 0 && B == 0) return RLF_ERR_SHAPE;
    const size_t esz = dt == RLF_BF16 ? 2 : 4;
    if (!aligned(logits, esz) || !aligned(grad_logits, esz)) return RLF_ERR_ALIGN;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < loss_workspace_bytes(T)) return RLF_ERR_WORKSPACE;
    const bool fast_ok = dt == RLF_BF16 && (V % 8 == 0) && (row_stride % 8 == 0) && aligned(logits, 16) &&
                         aligned(grad_logits, 16) && T < (1ll << 30);
    FastShape sh;
    if (T == 0 || !fast_ok || !pick_shape(V >> 3, &sh, /*allow_wide_cluster=*/true)) {
        // nothing to gain on the general path: process every row, then mark the dead rows' log-probs
        rlf_status st0 = rlf_grpo_logp_loss_fwd_bwd(logits, dt, T, V, row_stride, ids, seq_id, adv, B, old_logp, ref_logp,
                                                    mask, eps_clip, beta_kl, denom, logp_out, loss_out, grad_logits,
                                                    workspace, workspace_bytes, dev_status, stream);
        if (st0 != RLF_OK || T == 0) return st0;
        const float4* rec0 = reinterpret_cast<const float4*>(static_cast<char*>(workspace) + kWsRecordOff);
        fill_dead_rows_kernel<float><<<general_grid(T), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
            rec0, T, V, row_stride, nullptr, 0, logp_out);
        count_launch();
        return cuda_ok(cudaGetLastError());
    }
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    long long* n_count = reinterpret_cast<long long*>(ws);
    int* n_live = reinterpret_cast<int*>(ws + 128);
    double* partial = reinterpret_cast<double*>(ws + kWsPartialOff);
    float4* rec = reinterpret_cast<float4*>(ws + kWsRecordOff);
    float4* rec_c = reinterpret_cast<float4*>(ws + ws_compact_rec_off(T));
    int* row_list = reinterpret_cast<int*>(ws + ws_row_list_off(T));
    if (cudaMemsetAsync(ws, 0, 256, s) != cudaSuccess) return RLF_ERR_CUDA;
    const long long* dn = denom ? reinterpret_cast<const long long*>(denom) : n_count;
    st = launch_token_prep(ids, seq_id, adv, old_logp, ref_logp, mask, T, V, B, rec, denom ? nullptr : n_count,
                           dev_status, s);
    if (st != RLF_OK) return st;
    compact_live_kernel<<<(unsigned)((T + 255) / 256), 256, 0, s>>>(rec, T, row_list, rec_c, n_live);
    count_launch();
    fill_dead_rows_kernel<__nv_bfloat16><<<general_grid(T), 256, 0, s>>>(
        rec, T, V, row_stride, static_cast<__nv_bfloat16*>(grad_logits), zero_masked_grad, logp_out);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;

    FastKernel k = skip_kernel(sh);
    int nc = k ? max_clusters(k, sh) : -1;
    if (nc <= 0 && sh.cluster > 8 && g_tune_cluster.load() == 0 && pick_shape(V >> 3, &sh)) {
        k = skip_kernel(sh);             // the device does not take the wide cluster: the portable shape
        nc = k ? max_clusters(k, sh) : -1;
    }
    if (!k || nc <= 0) return RLF_ERR_UNSUPPORTED;
    nc = clusters_for(nc, T);            // T bounds the listed rows, whose number is only known on the device
    FastParams p;
    p.logits = static_cast<const __nv_bfloat16*>(logits);
    p.grad = static_cast<__nv_bfloat16*>(grad_logits);
    p.stride = row_stride;
    p.T = (int)T;
    p.nvec = V >> 3;
    p.per_cta_vec = per_cta_vectors(p.nvec, sh.cluster);
    p.rec = rec_c;
    p.denom = dn;
    p.logp_out = logp_out;
    p.entropy_out = nullptr;
    p.row_list = row_list;
    p.n_rows = n_live;
    p.dev_status = dev_status;
    p.eps_clip = eps_clip;
    p.eps_hi = eps_clip;
    p.wtok = nullptr;
    p.beta = beta_kl;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute at[1];
    cluster_config(&cfg, at, nc * sh.cluster, sh, s);
    if (cudaLaunchKernelEx(&cfg, k, p) != cudaSuccess) {
        cudaGetLastError();
        return RLF_ERR_CUDA;
    }
    count_launch();
    return launch_token_loss(logp_out, rec, T, eps_clip, beta_kl, partial, dn, loss_out, s);
}

// ---------------------------------------------------------------------------------------------
// Token-record and scalar-loss stages, shared with the fused LM-head path.
namespace rlf {

rlf_status launch_token_prep(const int32_t* ids, const int32_t* seq_id, const float* adv, const float* old_logp,
                             const float* ref_logp, const uint8_t* mask, int64_t T, int32_t V, int32_t B,
                             void* rec, long long* n_count_or_null, int32_t* dev_status, cudaStream_t s) {
    if (T <= 0) return RLF_OK;
    const int64_t blocks = (T + kPrepThreads - 1) / kPrepThreads;
    token_prep_kernel<<<(unsigned)blocks, kPrepThreads, 0, s>>>(
        ids, seq_id, adv, old_logp, ref_logp, mask, T, V, B, static_cast<float4*>(rec),
        reinterpret_cast<unsigned long long*>(n_count_or_null), dev_status);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

rlf_status launch_token_loss(const float* logp, const void* rec, int64_t T, float eps_clip, float beta,
                             double* partial, const long long* denom, double* loss_out, cudaStream_t s) {
    int num_partials = 0;
    if (T > 0) {
        const int64_t blocks = (T + kLossThreads - 1) / kLossThreads;
        num_partials = (int)(blocks < kMaxPartials ? blocks : kMaxPartials);
        token_loss_kernel<<<num_partials, kLossThreads, 0, s>>>(logp, static_cast<const float4*>(rec), T, eps_clip,
                                                               eps_clip, nullptr, partial);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    }
    finalize_loss_kernel<<<1, 96, 0, s>>>(partial, num_partials, denom, beta, 0, loss_out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

rlf_status launch_token_loss_w(const float* logp, const void* rec, int64_t T, float eps_lo, float eps_hi, float beta,
                               const float* wtok, double* partial, const long long* denom, double* loss_out,
                               cudaStream_t s) {
    int num_partials = 0;
    if (T > 0) {
        const int64_t blocks = (T + kLossThreads - 1) / kLossThreads;
        num_partials = (int)(blocks < kMaxPartials ? blocks : kMaxPartials);
        token_loss_kernel<<<num_partials, kLossThreads, 0, s>>>(logp, static_cast<const float4*>(rec), T, eps_lo,
                                                               eps_hi, wtok, partial);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    }
    finalize_loss_kernel<<<1, 96, 0, s>>>(partial, num_partials, denom, beta, wtok != nullptr, loss_out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

rlf_status launch_seq_weights(const void* rec, const int32_t* seq_id, int64_t T, int32_t B,
                              const long long* denom_or_null, int* cnt, long long* s_slot, float* wtok,
                              cudaStream_t s) {
    if (T <= 0) return RLF_OK;
    const int64_t blocks = (T + 255) / 256;
    if (cudaMemsetAsync(cnt, 0, sizeof(int) * (size_t)B, s) != cudaSuccess) return RLF_ERR_CUDA;
    seq_count_kernel<<<(unsigned)blocks, 256, 0, s>>>(static_cast<const float4*>(rec), seq_id, T, cnt);
    seq_live_kernel<<<1, 1024, 0, s>>>(cnt, B, denom_or_null, s_slot);
    seq_weight_kernel<<<(unsigned)blocks, 256, 0, s>>>(static_cast<const float4*>(rec), seq_id, T, cnt, s_slot, wtok);
    count_launch(3);
    return cuda_ok(cudaGetLastError());
}

size_t token_loss_partial_bytes() { return sizeof(double) * 4 * kMaxPartials; }

}  // namespace rlf

// ---------------------------------------------------------------------------------------------
// Variant for callers that cannot allocate: the scratch lives in the library's device image.
namespace rlf {

// The array is sized by the same layout function that the workspace check of the forwarded call
// uses, so a batch of RLF_STATIC_MAX_TOKENS tokens always fits (about 2.9 MB per device).
constexpr size_t kStaticScratchBytes = (ws_total_bytes(RLF_STATIC_MAX_TOKENS) + 255) & ~(size_t)255;
static_assert(kStaticScratchBytes >= ws_total_bytes(RLF_STATIC_MAX_TOKENS) &&
              ws_total_bytes(RLF_STATIC_MAX_TOKENS) >= ws_total_bytes(RLF_STATIC_MAX_TOKENS - 1),
              "the built-in scratch must hold the workspace of the largest batch the entry point accepts");
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the scratch array on the current device.  In host code the array's name only
// stands for the symbol; the address a kernel can use comes from the runtime, per device.
static rlf_status static_scratch_ptr(void** out) {
    static std::mutex mu;
    static void* ptr_of_device[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RLF_ERR_CUDA;
    if (dev < 0 || dev >= 64) return RLF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (ptr_of_device[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return RLF_ERR_CUDA;
        }
        ptr_of_device[dev] = ptr;
    }
    *out = ptr_of_device[dev];
    return RLF_OK;
}

}  // namespace rlf

extern "C" rlf_status rlf_grpo_logp_loss_fwd_bwd_static(
    const void* logits, rlf_dtype dt, int64_t T, int32_t V, int64_t row_stride, const int32_t* ids,
    const int32_t* seq_id, const float* adv, int32_t B, const float* old_logp, const float* ref_logp,
    const uint8_t* mask, float eps_clip, float beta_kl, const int64_t* denom, float* logp_out,
    double* loss_out, void* grad_logits, int32_t* dev_status, rlf_stream_t stream) {
    if (T > RLF_STATIC_MAX_TOKENS) return RLF_ERR_TOO_LARGE;
    rlf_status st = rlf::check_arch();
    if (st != RLF_OK) return st;
    void* scratch = nullptr;
    st = rlf::static_scratch_ptr(&scratch);
    if (st != RLF_OK) return st;
    return rlf_grpo_logp_loss_fwd_bwd(logits, dt, T, V, row_stride, ids, seq_id, adv, B, old_logp, ref_logp,
                                      mask, eps_clip, beta_kl, denom, logp_out, loss_out, grad_logits,
                                      scratch, rlf::kStaticScratchBytes, dev_status, stream);
}
