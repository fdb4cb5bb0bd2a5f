// Group-relative outcome advantage: A_i = (r_i - mean_g) / (std_g + eps).
// One warp per group.  Members are visited in index order, lane-strided, and the fp64 partial
// sums are combined by a fixed shuffle tree, so results are run-to-run identical.  B is the number
// of responses of a micro-batch (tens to thousands): launch latency is all this costs.
#include "common.cuh"

namespace rlf {

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(128)
group_advantage_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_id,
                       int32_t B, int32_t g_or_num_groups, int32_t num_groups, float eps,
                       int unbiased, float* __restrict__ adv_out, int32_t* __restrict__ dev_status) {
    const int lane = threadIdx.x & 31;
    const int warps_per_cta = blockDim.x >> 5;
    for (int g = blockIdx.x * warps_per_cta + (threadIdx.x >> 5); g < num_groups;
         g += gridDim.x * warps_per_cta) {
        int lo = 0, hi = B;
        if (!group_id) {
            lo = g * g_or_num_groups;
            hi = min(B, lo + g_or_num_groups);
        }
        double sum = 0.0;
        int n = 0;
        for (int i = lo + lane; i < hi; i += 32) {
            if (!group_id || group_id[i] == g) { sum += (double)rewards[i]; ++n; }
        }
        sum = warp_sum_f64(sum);
        n = __reduce_add_sync(0xffffffffu, n);
        if (n == 0) continue;
        const double mean = sum / (double)n;
        double ss = 0.0;
        for (int i = lo + lane; i < hi; i += 32) {
            if (!group_id || group_id[i] == g) { double d = (double)rewards[i] - mean; ss += d * d; }
        }
        ss = warp_sum_f64(ss);
        const double div = unbiased ? (double)(n - 1) : (double)n;
        const double sd = div > 0.0 ? sqrt(ss / div) : 0.0;
        // zero spread (or a single member) with eps = 0 would be 0 * inf: such a group carries no
        // signal and gets A = 0 like every other degenerate group
        const double den = sd + (double)eps;
        const double inv = den > 0.0 ? 1.0 / den : 0.0;
        for (int i = lo + lane; i < hi; i += 32) {
            if (!group_id || group_id[i] == g) adv_out[i] = (float)(((double)rewards[i] - mean) * inv);
        }
    }
    // responses whose group id is out of range: advantage 0 and a status bit
    if (group_id && blockIdx.x == 0) {
        for (int i = threadIdx.x; i < B; i += blockDim.x) {
            int gi = group_id[i];
            if (gi < 0 || gi >= num_groups) {
                adv_out[i] = 0.0f;
                if (dev_status) atomicOr(dev_status, RLF_DEV_BAD_SEQ);
            }
        }
    }
}

}  // namespace rlf

extern "C" rlf_status rlf_group_advantage(const float* rewards, const int32_t* group_id, int32_t B,
                                          int32_t g_or_num_groups, float eps, int unbiased_std,
                                          float* adv_out, int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (B < 0 || g_or_num_groups <= 0) return RLF_ERR_SHAPE;
    if (B == 0) return RLF_OK;
    if (!rewards || !adv_out) return RLF_ERR_NULL;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    const int num_groups = group_id ? g_or_num_groups : (B + g_or_num_groups - 1) / g_or_num_groups;
    const int ctas = (num_groups + 3) / 4 < 592 ? (num_groups + 3) / 4 : 592;
    group_advantage_kernel<<<ctas, 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        rewards, group_id, B, g_or_num_groups, num_groups, eps, unbiased_std, adv_out, dev_status);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// Rule reward (paper Eq. 1): R_b = sum_i w_i r_{b,i}.  One thread per response, fp64 accumulation in
// index order (n is a handful of rule dimensions).
namespace rlf {
__global__ void __launch_bounds__(128)
rule_reward_kernel(const float* __restrict__ scores, const float* __restrict__ weights, int32_t B, int32_t n,
                   float* __restrict__ reward_out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    double acc = 0.0;
    for (int i = 0; i < n; ++i) acc += (double)weights[i] * (double)scores[(long long)b * n + i];
    reward_out[b] = (float)acc;
}
}  // namespace rlf

extern "C" rlf_status rlf_rule_reward(const float* scores, const float* weights, int32_t B, int32_t n,
                                      float* reward_out, rlf_stream_t stream) {
    using namespace rlf;
    if (B < 0 || n < 0) return RLF_ERR_SHAPE;
    if (B == 0) return RLF_OK;
    if (!reward_out || (n > 0 && (!scores || !weights))) return RLF_ERR_NULL;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    rule_reward_kernel<<<(B + 127) / 128, 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(scores, weights, B, n,
                                                                                          reward_out);
    count_launch();
    return cuda_ok(cudaGetLastError());
}

// ---------------------------------------------------------------------------------------------
// KL penalty folded into the outcome reward: R'_b = R_b - beta * sum_{t in b} mask_t k(old_t, ref_t),
// d = old_logp - ref_logp; kind 0: k = d, kind 1: k = d^2 / 2, kind 2: k = exp(-d) + d - 1.
// One CTA per response; every thread sums its tokens (stride 256, index order) in fp64 and the
// partial sums are combined by a fixed shuffle tree and a fixed loop over warps, so results are
// run-to-run identical.  10 bytes per token: launch latency is what this costs.
namespace rlf {
__global__ void __launch_bounds__(256)
kl_in_reward_kernel(const float* __restrict__ rewards, const float* __restrict__ old_logp,
                    const float* __restrict__ ref_logp, const uint8_t* __restrict__ mask,
                    const int32_t* __restrict__ cu_seqlens, int64_t T, float beta, int kind,
                    float* __restrict__ reward_out, float* __restrict__ kl_seq_out, int32_t* __restrict__ dev_status) {
    __shared__ double warp_part[8];
    const int b = blockIdx.x;
    long long lo = cu_seqlens[b], hi = cu_seqlens[b + 1];
    if (lo < 0 || hi < lo || hi > T) {
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, RLF_DEV_BAD_SEQ);
        lo = lo < 0 ? 0 : (lo > T ? T : lo);
        hi = hi < lo ? lo : (hi > T ? T : hi);
    }
    double acc = 0.0;
    for (long long t = lo + threadIdx.x; t < hi; t += 256) {
        if (!mask[t]) continue;
        const double d = (double)old_logp[t] - (double)ref_logp[t];
        acc += kind == 0 ? d : kind == 1 ? 0.5 * d * d : exp(-d) + d - 1.0;
    }
    acc = warp_sum_f64(acc);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += warp_part[w];
        if (kl_seq_out) kl_seq_out[b] = (float)s;
        reward_out[b] = (float)((double)rewards[b] - (double)beta * s);
    }
}
}  // namespace rlf

extern "C" rlf_status rlf_kl_in_reward(const float* rewards, const float* old_logp, const float* ref_logp,
                                       const uint8_t* mask, const int32_t* cu_seqlens, int32_t B, int64_t T,
                                       float beta, int kl_kind, float* reward_out, float* kl_seq_out,
                                       int32_t* dev_status, rlf_stream_t stream) {
    using namespace rlf;
    if (B < 0 || T < 0) return RLF_ERR_SHAPE;
    if (kl_kind < 0 || kl_kind > 2) return RLF_ERR_UNSUPPORTED;
    if (B == 0) return RLF_OK;
    if (!rewards || !reward_out || !cu_seqlens) return RLF_ERR_NULL;
    if (T > 0 && (!old_logp || !ref_logp || !mask)) return RLF_ERR_NULL;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    kl_in_reward_kernel<<<B, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        rewards, old_logp, ref_logp, mask, cu_seqlens, T, beta, kl_kind, reward_out, kl_seq_out, dev_status);
    count_launch();
    return cuda_ok(cudaGetLastError());
}
