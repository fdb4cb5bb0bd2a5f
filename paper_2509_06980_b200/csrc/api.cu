// Entry points that are not tied to one kernel: device check, accounting, workspace sizes, status
// strings, and the whole-step call that takes host buffers.
#include <atomic>

#include "common.cuh"

namespace rlf {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

rlf_status check_arch() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RLF_ERR_CUDA;
    static std::atomic<int> cached[64];   // 0 unknown, 1 ok, 2 wrong arch
    if (dev >= 0 && dev < 64) {
        int c = cached[dev].load();
        if (c) return c == 1 ? RLF_OK : RLF_ERR_ARCH;
    }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return RLF_ERR_CUDA;
    const bool ok = major == 10;
    if (dev >= 0 && dev < 64) cached[dev] = ok ? 1 : 2;
    return ok ? RLF_OK : RLF_ERR_ARCH;
}

size_t loss_workspace_bytes(int64_t T);                          // logits_loss.cu
size_t lmhead_workspace_bytes(int64_t T, int32_t V, int32_t D);  // lmhead.cu
size_t entropy_workspace_bytes(int64_t T, int32_t V);             // logits_loss.cu
size_t lmhead_logp_workspace_bytes(int64_t T);                    // lmhead.cu

static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

struct StepArena {
    size_t logits, ids, cu, rewards, old_lp, ref_lp, mask, seq_id, adv, n, logp, loss, status, ws, total;
};
static StepArena step_arena(int64_t T, int32_t V, int32_t B, rlf_dtype dt) {
    StepArena a;
    size_t o = 0;
    const size_t esz = dt == RLF_BF16 ? 2 : 4;
    a.logits = o;  o += up256((size_t)T * (size_t)V * esz);
    a.ids = o;     o += up256((size_t)T * 4);
    a.cu = o;      o += up256((size_t)(B + 1) * 4);
    a.rewards = o; o += up256((size_t)B * 4);
    a.old_lp = o;  o += up256((size_t)T * 4);
    a.ref_lp = o;  o += up256((size_t)T * 4);
    a.mask = o;    o += up256((size_t)T);
    a.seq_id = o;  o += up256((size_t)T * 4);
    a.adv = o;     o += up256((size_t)B * 4);
    a.n = o;       o += 256;
    a.logp = o;    o += up256((size_t)T * 4);
    a.loss = o;    o += 256;
    a.status = o;  o += 256;
    a.ws = o;      o += up256(loss_workspace_bytes(T));
    a.total = o;
    return a;
}

}  // namespace rlf

extern "C" int64_t rlf_launch_count(void) { return rlf::g_launches.load(); }

extern "C" int rlf_version(void) { return 100; }

extern "C" const char* rlf_status_string(rlf_status s) {
    switch (s) {
        case RLF_OK: return "ok";
        case RLF_ERR_NULL: return "a required pointer is NULL";
        case RLF_ERR_SHAPE: return "invalid or inconsistent size";
        case RLF_ERR_ALIGN: return "pointer or stride misaligned";
        case RLF_ERR_DTYPE: return "unknown dtype";
        case RLF_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case RLF_ERR_ARCH: return "device is not sm_100";
        case RLF_ERR_CUDA: return "CUDA runtime error";
        case RLF_ERR_UNSUPPORTED: return "request outside what this library implements";
        case RLF_ERR_TOO_LARGE: return "more tokens than the built-in scratch holds (RLF_STATIC_MAX_TOKENS)";
    }
    return "unknown status";
}

extern "C" size_t rlf_workspace_bytes(int which_fn, int64_t T, int32_t V, int32_t D, rlf_dtype dt) {
    (void)dt;
    if (which_fn == RLF_FN_LOGP_LOSS) return rlf::loss_workspace_bytes(T);
    if (which_fn == RLF_FN_FUSED_LMHEAD) return rlf::lmhead_workspace_bytes(T, V, D);
    if (which_fn == RLF_FN_LOGP_ENTROPY) return rlf::entropy_workspace_bytes(T, V);
    if (which_fn == RLF_FN_FUSED_LOGP_ENTROPY) return rlf::lmhead_logp_workspace_bytes(T);
    return 0;
}

extern "C" size_t rlf_step_arena_bytes(int64_t T, int32_t V, int32_t B, rlf_dtype dt) {
    if (T < 0 || V < 1 || B < 0) return 0;
    return rlf::step_arena(T, V, B, dt).total;
}

extern "C" rlf_status rlf_grpo_step_host(const void* h_logits, rlf_dtype dt, int64_t T, int32_t V,
                                         const int32_t* h_ids, const int32_t* h_cu_seqlens, int32_t B,
                                         int32_t G, const float* h_rewards, const float* h_old_logp,
                                         const float* h_ref_logp, int32_t open_id, int32_t close_id,
                                         float adv_eps, float eps_clip, float beta_kl,
                                         double* h_loss_out, float* h_logp_out, uint8_t* h_mask_out,
                                         int32_t* h_dev_status, void* d_arena, size_t arena_bytes,
                                         rlf_stream_t stream) {
    using namespace rlf;
    if (dt != RLF_BF16 && dt != RLF_F32) return RLF_ERR_DTYPE;
    if (T < 1 || V < 1 || B < 1 || G < 1) return RLF_ERR_SHAPE;
    if (!h_logits || !h_ids || !h_cu_seqlens || !h_rewards || !h_old_logp || !h_ref_logp || !h_loss_out)
        return RLF_ERR_NULL;
    const StepArena a = step_arena(T, V, B, dt);
    if (!d_arena || !aligned(d_arena, 256) || arena_bytes < a.total) return RLF_ERR_WORKSPACE;
    rlf_status st = check_arch();
    if (st != RLF_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(d_arena);
    const size_t esz = dt == RLF_BF16 ? 2 : 4;
    auto h2d = [&](size_t off, const void* src, size_t bytes) {
        return cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
    };
    bool ok = true;
    ok = ok && h2d(a.ids, h_ids, (size_t)T * 4);
    ok = ok && h2d(a.cu, h_cu_seqlens, (size_t)(B + 1) * 4);
    ok = ok && h2d(a.rewards, h_rewards, (size_t)B * 4);
    ok = ok && h2d(a.old_lp, h_old_logp, (size_t)T * 4);
    ok = ok && h2d(a.ref_lp, h_ref_logp, (size_t)T * 4);
    ok = ok && h2d(a.logits, h_logits, (size_t)T * (size_t)V * esz);
    ok = ok && cudaMemsetAsync(base + a.status, 0, 4, s) == cudaSuccess;
    if (!ok) return RLF_ERR_CUDA;

    int32_t* d_status = reinterpret_cast<int32_t*>(base + a.status);
    st = rlf_build_loss_mask(reinterpret_cast<int32_t*>(base + a.ids), reinterpret_cast<int32_t*>(base + a.cu),
                             B, T, open_id, close_id, nullptr, reinterpret_cast<uint8_t*>(base + a.mask),
                             reinterpret_cast<int32_t*>(base + a.seq_id),
                             reinterpret_cast<int64_t*>(base + a.n), d_status, stream);
    if (st != RLF_OK) return st;
    st = rlf_group_advantage(reinterpret_cast<float*>(base + a.rewards), nullptr, B, G, adv_eps, 1,
                             reinterpret_cast<float*>(base + a.adv), d_status, stream);
    if (st != RLF_OK) return st;
    st = rlf_grpo_logp_loss_fwd_bwd(base + a.logits, dt, T, V, V, reinterpret_cast<int32_t*>(base + a.ids),
                                    reinterpret_cast<int32_t*>(base + a.seq_id),
                                    reinterpret_cast<float*>(base + a.adv), B,
                                    reinterpret_cast<float*>(base + a.old_lp),
                                    reinterpret_cast<float*>(base + a.ref_lp),
                                    reinterpret_cast<uint8_t*>(base + a.mask), eps_clip, beta_kl,
                                    reinterpret_cast<int64_t*>(base + a.n),
                                    reinterpret_cast<float*>(base + a.logp),
                                    reinterpret_cast<double*>(base + a.loss), base + a.logits,
                                    base + a.ws, loss_workspace_bytes(T), d_status, stream);
    if (st != RLF_OK) return st;
    auto d2h = [&](void* dst, size_t off, size_t bytes) {
        return cudaMemcpyAsync(dst, base + off, bytes, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    };
    ok = d2h(h_loss_out, a.loss, 4 * sizeof(double));
    if (h_logp_out) ok = ok && d2h(h_logp_out, a.logp, (size_t)T * 4);
    if (h_mask_out) ok = ok && d2h(h_mask_out, a.mask, (size_t)T);
    if (h_dev_status) ok = ok && d2h(h_dev_status, a.status, 4);
    if (!ok) return RLF_ERR_CUDA;
    return cuda_ok(cudaStreamSynchronize(s));
}
