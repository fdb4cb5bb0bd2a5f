// Shared host/device helpers of the CUDA library (status codes, launch accounting, small
// device utilities).  Nothing here is used by, or shared with, the CPU oracle.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/rlf.h"

namespace rlf {

// counts kernels launched by this library (host side, relaxed)
void count_launch(int n = 1);

// RLF_OK iff the current device is compute capability 10.x
rlf_status check_arch();

// token-record and scalar-loss stages (logits_loss.cu), also used by the fused LM-head path
rlf_status launch_token_prep(const int32_t* ids, const int32_t* seq_id, const float* adv, const float* old_logp,
                             const float* ref_logp, const uint8_t* mask, int64_t T, int32_t V, int32_t B,
                             void* rec, long long* n_count_or_null, int32_t* dev_status, cudaStream_t s);
rlf_status launch_token_loss(const float* logp, const void* rec, int64_t T, float eps_clip, float beta,
                             double* partial, const long long* denom, double* loss_out, cudaStream_t s);
size_t token_loss_partial_bytes();
// the same with an asymmetric clip range and optional per-token weights (weighted sums are already means)
rlf_status launch_token_loss_w(const float* logp, const void* rec, int64_t T, float eps_lo, float eps_hi, float beta,
                               const float* wtok, double* partial, const long long* denom, double* loss_out,
                               cudaStream_t s);
// sequence-mean aggregation: wtok[t] = live_t / (n_b * S); cnt [B] ints and s_slot [1] are scratch
rlf_status launch_seq_weights(const void* rec, const int32_t* seq_id, int64_t T, int32_t B,
                              const long long* denom_or_null, int* cnt, long long* s_slot, float* wtok,
                              cudaStream_t s);

inline rlf_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? RLF_OK : RLF_ERR_CUDA; }

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace rlf
