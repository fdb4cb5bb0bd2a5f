// Loss mask from observation markers: a segmented scan over the two-state machine
// {outside, inside} whose transitions are "open marker: set inside", "close marker: set outside",
// "anything else: keep".  Because both markers SET the state, the state before a token is decided
// by the nearest marker before it in the same response ("last marker wins"), which a warp resolves
// with two ballots and a count-leading-zeros; carries cross warps through shared memory and cross
// 1024-token chunks of a response through a register.  One CTA per response.
#include "common.cuh"

namespace rlf {

constexpr int kMaskThreads = 1024;

__global__ void __launch_bounds__(kMaskThreads)
mask_scan_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ cu_seqlens, int32_t B,
                 int64_t T, int32_t open_id, int32_t close_id, const uint8_t* __restrict__ valid,
                 uint8_t* __restrict__ mask_out, int32_t* __restrict__ seq_id_out,
                 unsigned long long* __restrict__ n_out, int32_t* __restrict__ dev_status) {
    __shared__ int warp_tr[kMaskThreads / 32];   // 0 keep, 1 set inside, 2 set outside
    __shared__ int chunk_carry;
    __shared__ unsigned int cta_count;
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t s0 = cu_seqlens[b], s1 = cu_seqlens[b + 1];
    if (threadIdx.x == 0) {
        bool bad = (s0 < 0) || (s1 > T) || (s1 < s0) || (b == 0 && s0 != 0) || (b == B - 1 && s1 != T);
        if (bad && dev_status) atomicOr(dev_status, RLF_DEV_BAD_SEQ);
        chunk_carry = 0;
        cta_count = 0;
    }
    s0 = s0 < 0 ? 0 : (s0 > T ? T : s0);
    s1 = s1 < s0 ? s0 : (s1 > T ? T : s1);
    __syncthreads();

    unsigned int my_count = 0;
    for (int64_t base = s0; base < s1; base += kMaskThreads) {
        const int64_t t = base + threadIdx.x;
        const bool live = t < s1;
        const int32_t id = live ? ids[t] : -1;
        const bool is_open = live && (id == open_id);
        const bool is_close = live && (id == close_id) && !is_open;
        const unsigned O = __ballot_sync(0xffffffffu, is_open);
        const unsigned C = __ballot_sync(0xffffffffu, is_close);
        const unsigned M = O | C;
        if (lane == 0) warp_tr[warp] = M ? (((O >> (31 - __clz(M))) & 1u) ? 1 : 2) : 0;
        const int carry_in_chunk = chunk_carry;
        __syncthreads();
        // state entering this warp: nearest earlier warp of the chunk that saw a marker, else the chunk carry
        int tr = (lane < warp) ? warp_tr[lane] : 0;
        const unsigned has = __ballot_sync(0xffffffffu, tr != 0);
        int inside_warp_in = carry_in_chunk;
        if (has) inside_warp_in = (__shfl_sync(0xffffffffu, tr, 31 - __clz(has)) == 1);
        // state before this token: nearest earlier marker in the warp, else the warp's entry state
        const unsigned before = M & ((1u << lane) - 1u);
        const int inside_before = before ? (int)((O >> (31 - __clz(before))) & 1u) : inside_warp_in;
        if (live) {
            uint8_t m = (is_open || inside_before) ? 0 : 1;
            if (valid && !valid[t]) m = 0;
            mask_out[t] = m;
            if (seq_id_out) seq_id_out[t] = b;
            my_count += m;
        }
        __syncthreads();
        if (threadIdx.x == kMaskThreads - 1) {
            // carry leaving the chunk = state after the last warp
            chunk_carry = M ? (int)((O >> (31 - __clz(M))) & 1u) : inside_warp_in;
        }
        __syncthreads();
    }
    my_count = __reduce_add_sync(0xffffffffu, my_count);
    if (lane == 0 && my_count) atomicAdd(&cta_count, my_count);
    __syncthreads();
    if (threadIdx.x == 0 && cta_count) atomicAdd(n_out, (unsigned long long)cta_count);
}

}  // namespace rlf

extern "C" rlf_status rlf_build_loss_mask(const int32_t* ids, const int32_t* cu_seqlens, int32_t B,
                                          int64_t T, int32_t open_id, int32_t close_id,
                                          const uint8_t* valid, uint8_t* mask_out,
                                          int32_t* seq_id_out, int64_t* n_out, int32_t* dev_status,
                                          rlf_stream_t stream) {
    using namespace rlf;
    if (B < 0 || T < 0) return RLF_ERR_SHAPE;
    if (!n_out || !cu_seqlens) return RLF_ERR_NULL;
    if (T > 0 && (!ids || !mask_out)) return RLF_ERR_NULL;
    if (T > 0 && B == 0) return RLF_ERR_SHAPE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(n_out, 0, sizeof(int64_t), s) != cudaSuccess) return RLF_ERR_CUDA;
    if (T > 0) {
        // tokens that no response covers keep mask 0 / seq_id -1
        if (cudaMemsetAsync(mask_out, 0, (size_t)T, s) != cudaSuccess) return RLF_ERR_CUDA;
        if (seq_id_out && cudaMemsetAsync(seq_id_out, 0xFF, (size_t)T * 4, s) != cudaSuccess)
            return RLF_ERR_CUDA;
    }
    if (B > 0) {
        mask_scan_kernel<<<B, kMaskThreads, 0, s>>>(ids, cu_seqlens, B, T, open_id, close_id, valid,
                                                    mask_out, seq_id_out,
                                                    reinterpret_cast<unsigned long long*>(n_out),
                                                    dev_status);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    }
    return RLF_OK;
}

// ---------------------------------------------------------------------------------------------
// Number of responses that carry loss: those with at least one token of mask 1.  The denominator of
// the sequence-mean aggregation; a rank of a sharded batch counts its own responses and the counts
// are summed.  One CTA per response; integer atomics (exact).
namespace rlf {
__global__ void __launch_bounds__(256)
count_live_responses_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ cu_seqlens, int64_t T,
                            unsigned long long* __restrict__ count_out, int32_t* __restrict__ dev_status) {
    long long lo = cu_seqlens[blockIdx.x], hi = cu_seqlens[blockIdx.x + 1];
    if (lo < 0 || hi < lo || hi > T) {
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, RLF_DEV_BAD_SEQ);
        lo = lo < 0 ? 0 : (lo > T ? T : lo);
        hi = hi < lo ? lo : (hi > T ? T : hi);
    }
    int any = 0;
    for (long long t = lo + threadIdx.x; t < hi; t += 256) any |= mask[t] != 0;
    any = __syncthreads_or(any);
    if (threadIdx.x == 0 && any) atomicAdd(count_out, 1ull);
}
}  // namespace rlf

extern "C" rlf_status rlf_count_live_responses(const uint8_t* mask, const int32_t* cu_seqlens, int32_t B, int64_t T,
                                               int64_t* count_out, int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (B < 0 || T < 0) return RLF_ERR_SHAPE;
    if (!count_out || (B > 0 && !cu_seqlens) || (T > 0 && B > 0 && !mask)) return RLF_ERR_NULL;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(count_out, 0, sizeof(int64_t), s) != cudaSuccess) return RLF_ERR_CUDA;
    if (B > 0) {
        count_live_responses_kernel<<<B, 256, 0, s>>>(mask, cu_seqlens, T, reinterpret_cast<unsigned long long*>(count_out),
                                                      dev_status);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return RLF_ERR_CUDA;
    }
    return RLF_OK;
}
