// Read-only streaming probe: sums a buffer with 16-byte loads, one pass, nothing written but one word per CTA.
// It measures what a kernel that only READS device memory can reach on this part (the attention kernels are such
// kernels: K and V are read once, the outputs are tiny), next to the copy figure that counts a read and a write.
#include "common.cuh"

namespace hippo {

constexpr int kProbeThreads = 512;
constexpr int kProbeUnroll = 8;

__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const uint4 *__restrict__ src, size_t n16, unsigned int *sink) {
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    unsigned int acc = 0;
    for (; i + (kProbeUnroll - 1) * stride < n16; i += kProbeUnroll * stride) {
        uint4 v[kProbeUnroll];
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) v[u] = __ldcs(src + i + u * stride);   // streaming: do not keep in cache
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) acc += v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldcs(src + i);
        acc += v.x ^ v.y ^ v.z ^ v.w;
    }
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) atomicAdd(sink + (blockIdx.x & 63), acc);
}

}  // namespace hippo

extern "C" int32_t hippo_read_probe(const void *buffer, size_t bytes, void *sink, void *stream) {
    using namespace hippo;
    if (!buffer || !sink) return fail(HIPPO_ERR_INVALID_ARG, "hippo_read_probe: null pointer");
    if (((uintptr_t)buffer & 15) || ((uintptr_t)sink & 255)) return fail(HIPPO_ERR_INVALID_ARG, "hippo_read_probe: buffer must be 16-byte, sink 256-byte aligned");
    if (bytes < 16) return fail(HIPPO_ERR_INVALID_ARG, "hippo_read_probe: fewer than 16 bytes");
    read_probe_kernel<<<kNumSMs * 4, kProbeThreads, 0, (cudaStream_t)stream>>>((const uint4 *)buffer, bytes / 16, (unsigned int *)sink);
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}
