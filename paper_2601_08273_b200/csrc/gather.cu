// hippo_gather_kv: compacts the kept rows of the draft model's KV cache, all layers in one launch.
//
// "One-time pruning of the draft model's KV cache during the prefill stage" (Limitations (i)): after selection the
// draft keeps only the chosen visual tokens plus the always-kept positions.  A pure copy, bound by HBM bandwidth:
// per kept token and layer 2 * n_kv_heads * head_dim elements are read and written once.
//
// One work item moves 16 bytes; a thread takes four items per round, all four loads issued before the first store.
// Items are ordered (chunk within row, destination token, head) inside a (layer, K|V) plane given by blockIdx.y, so
// that consecutive threads write consecutive addresses of one destination (page, head) block; reads are whole rows of
// head_dim elements (128 B for head_dim 64 bf16) scattered over the source pages.  Index arithmetic is 32-bit.
#include "common.cuh"

namespace hippo {

struct GatherParams {
    const char *src_k, *src_v;
    char *dst_k, *dst_v;
    const int32_t *src_table, *dst_table, *keep_idx, *keep_offsets;
    size_t src_layer_stride, dst_layer_stride;
    int n_layers, batch, total_keep, n_kv_heads, row_chunks, src_mpps, dst_mpps;
};

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;

__global__ void __launch_bounds__(kGatherThreads) gather_kv_kernel(const GatherParams p) {
    const uint32_t per_plane = (uint32_t)p.total_keep * (uint32_t)p.n_kv_heads * (uint32_t)p.row_chunks;
    const int l = blockIdx.y >> 1, is_v = blockIdx.y & 1;
    const char *src = (is_v ? p.src_v : p.src_k) + (size_t)l * p.src_layer_stride;
    char *dst = (is_v ? p.dst_v : p.dst_k) + (size_t)l * p.dst_layer_stride;
    const uint32_t row_bytes = (uint32_t)p.row_chunks * 16u;
    const uint32_t stride = gridDim.x * kGatherThreads;
    for (uint32_t w0 = blockIdx.x * kGatherThreads + threadIdx.x; w0 < per_plane; w0 += stride * kGatherUnroll) {
        size_t so[kGatherUnroll], dof[kGatherUnroll];
        bool live[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const uint32_t w = w0 + u * stride;
            live[u] = w < per_plane;
            const uint32_t x = live[u] ? w : 0u;
            const uint32_t c = x % (uint32_t)p.row_chunks, y = x / (uint32_t)p.row_chunks;
            const int i = (int)(y % (uint32_t)p.total_keep), h = (int)(y / (uint32_t)p.total_keep);
            // sequence of flat keep index i: largest b with keep_offsets[b] <= i
            int lo = 0, hi = p.batch;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (__ldg(p.keep_offsets + mid) <= i) lo = mid; else hi = mid;
            }
            const int src_tok = __ldg(p.keep_idx + i);
            const int dst_tok = i - __ldg(p.keep_offsets + lo);
            const int sp = page_of(p.src_table, p.src_mpps, lo, src_tok / kPageSize);
            const int dp = page_of(p.dst_table, p.dst_mpps, lo, dst_tok / kPageSize);
            so[u] = (((size_t)sp * p.n_kv_heads + h) * kPageSize + (src_tok % kPageSize)) * row_bytes + c * 16u;
            dof[u] = (((size_t)dp * p.n_kv_heads + h) * kPageSize + (dst_tok % kPageSize)) * row_bytes + c * 16u;
        }
        uint4 v[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u)
            if (live[u]) v[u] = __ldg(reinterpret_cast<const uint4 *>(src + so[u]));
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u)
            if (live[u]) *reinterpret_cast<uint4 *>(dst + dof[u]) = v[u];
    }
}

static int32_t check(const hippo_kv_cache_t *kv, const char *name) {
    if (!kv) return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: null %s descriptor", name);
    if (kv->struct_size != sizeof(hippo_kv_cache_t)) return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: %s struct_size", name);
    if (!kv->k_pages || !kv->v_pages) return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: null %s pool", name);
    if (kv->n_kv_heads <= 0 || kv->head_dim <= 0 || kv->n_pages <= 0 || kv->max_pages_per_seq <= 0)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: non-positive %s dimension", name);
    if (((uintptr_t)kv->k_pages | (uintptr_t)kv->v_pages) & 127)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: %s pools must be 128-byte aligned", name);
    return HIPPO_OK;
}

}  // namespace hippo

extern "C" int32_t hippo_gather_kv(int32_t n_layers, const hippo_kv_cache_t *src, size_t src_layer_stride_bytes,
                                   const hippo_kv_cache_t *dst, size_t dst_layer_stride_bytes, int32_t batch,
                                   const int32_t *keep_idx, const int32_t *keep_offsets, int32_t total_keep,
                                   void *stream) {
    using namespace hippo;
    int32_t rc = check(src, "src");
    if (rc != HIPPO_OK) return rc;
    rc = check(dst, "dst");
    if (rc != HIPPO_OK) return rc;
    if (n_layers <= 0 || batch <= 0 || total_keep < 0) return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: bad sizes");
    if (src->dtype != dst->dtype || src->n_kv_heads != dst->n_kv_heads || src->head_dim != dst->head_dim)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: src and dst disagree in dtype / heads / head_dim");
    if (src->dtype != HIPPO_DTYPE_FP32 && src->dtype != HIPPO_DTYPE_BF16)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: unknown dtype");
    const size_t esize = src->dtype == HIPPO_DTYPE_FP32 ? 4 : 2;
    const size_t row_bytes = (size_t)src->head_dim * esize;
    if (row_bytes % 16) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_gather_kv: head_dim*elem_size must be a multiple of 16 bytes");
    if ((src_layer_stride_bytes | dst_layer_stride_bytes) & 127)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: layer strides must be multiples of 128 bytes");
    if (total_keep == 0) return HIPPO_OK;
    if (!keep_idx || !keep_offsets) return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: null index arrays");

    GatherParams p;
    p.src_k = (const char *)src->k_pages; p.src_v = (const char *)src->v_pages;
    p.dst_k = (char *)dst->k_pages; p.dst_v = (char *)dst->v_pages;
    p.src_table = src->page_table; p.dst_table = dst->page_table;
    p.keep_idx = keep_idx; p.keep_offsets = keep_offsets;
    p.src_layer_stride = src_layer_stride_bytes; p.dst_layer_stride = dst_layer_stride_bytes;
    p.n_layers = n_layers; p.batch = batch; p.total_keep = total_keep; p.n_kv_heads = src->n_kv_heads;
    p.row_chunks = (int)(row_bytes / 16); p.src_mpps = src->max_pages_per_seq; p.dst_mpps = dst->max_pages_per_seq;
    const long long per_plane = (long long)total_keep * p.n_kv_heads * p.row_chunks;
    if (per_plane > 0x7fffffffLL) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_gather_kv: more than 2^31 16-byte items per layer");
    if (2 * n_layers > 65535) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_gather_kv: too many layers for one launch");
    // blocks per (layer, K|V) plane: enough rounds of kGatherUnroll items per thread, at most ~16 blocks per SM in total
    long long bx = (per_plane + kGatherThreads * kGatherUnroll - 1) / (kGatherThreads * kGatherUnroll);
    const long long cap = (long long)kNumSMs * 16 / (2 * n_layers) + 1;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    gather_kv_kernel<<<dim3((unsigned)bx, (unsigned)(2 * n_layers)), kGatherThreads, 0, (cudaStream_t)stream>>>(p);
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}
