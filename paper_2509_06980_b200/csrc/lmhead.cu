// Fused LM-head variant (placeholder until the tcgen05 kernels land).
#include "common.cuh"

namespace rlf {
size_t lmhead_workspace_bytes(int64_t, int32_t, int32_t) { return 0; }
}  // namespace rlf

extern "C" rlf_status rlf_fused_lmhead_grpo(const void*, const void*, int64_t, int32_t, int32_t,
                                            const int32_t*, const int32_t*, const float*, int32_t,
                                            const float*, const float*, const uint8_t*, float, float,
                                            const int64_t*, float*, double*, void*, float*, int,
                                            void*, size_t, int32_t*, rlf_stream_t) {
    return RLF_ERR_UNSUPPORTED;
}
