// Tensor-core attention kernel (placeholder until the tcgen05 path lands): reports "not supported" so that the
// dispatcher uses the CUDA-core kernel.
#include "common.cuh"

namespace hippo {

bool attn_tc_supported(const AttnParams &, int) { return false; }

int32_t launch_attn_tc(const AttnParams &, bool, cudaStream_t) {
    return fail(HIPPO_ERR_UNIMPLEMENTED, "tensor-core attention not built");
}

}  // namespace hippo
