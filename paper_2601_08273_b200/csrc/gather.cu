// hippo_gather_kv: compacts the kept rows of the draft model's KV cache, all layers in one launch.
//
// The draft model's cache is pruned once, during prefill (Limitations (i)): after selection the draft keeps only the
// chosen visual tokens plus the always-kept positions.  A pure copy, bound by HBM bandwidth: per kept token and layer
// 2 * n_kv_heads * head_dim elements are read and written once.
//
// One work item is a 16-byte piece of one kept row: (chunk within row, destination token, head).  Its offsets inside a
// (layer, K|V) plane are the same for every plane - the page tables are shared by all layers - so a thread resolves
// its item once (keep index, source and destination page) and then copies that piece in plane after plane, eight
// loads in flight before the first store.  blockIdx.y splits the planes into groups when there are too few items to
// fill the machine.  Items are ordered so that consecutive threads write consecutive addresses of one destination
// (page, head) block; reads are whole rows of head_dim elements (128 B for head_dim 64 bf16) scattered over the
// source pages.
//
// Indices come from device memory (a selector's output, an engine's page tables), so every address formed from them is
// checked first: a source position beyond the sequence's page capacity, a destination position beyond the destination's,
// or a page id outside its pool skips the item and raises the caller's flag word instead of touching memory.
#include <initializer_list>

#include "common.cuh"

namespace hippo {

struct GatherParams {
    const char *src_k, *src_v;
    char *dst_k, *dst_v;
    const int32_t *src_table, *dst_table, *keep_idx, *keep_offsets;
    int32_t *bad_index;          // may be null: set to 1 when an item was skipped
    size_t src_layer_stride, dst_layer_stride;
    int n_layers, batch, total_keep, n_kv_heads, row_chunks, src_mpps, dst_mpps, planes_per_group;
    int src_pages, dst_pages;    // pool sizes
};

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 8;

__global__ void __launch_bounds__(kGatherThreads) gather_kv_kernel(const GatherParams p) {
    const uint32_t per_plane = (uint32_t)p.total_keep * (uint32_t)p.n_kv_heads * (uint32_t)p.row_chunks;
    const uint32_t x = blockIdx.x * kGatherThreads + threadIdx.x;
    if (x >= per_plane) return;
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
    // positions must lie inside the page-table rows before the tables are read, page ids inside the pools before
    // the pools are
    bool ok = src_tok >= 0 && src_tok < p.src_mpps * kPageSize && dst_tok >= 0 && dst_tok < p.dst_mpps * kPageSize;
    int sp = 0, dp = 0;
    if (ok) {
        sp = page_of(p.src_table, p.src_mpps, lo, src_tok / kPageSize);
        dp = page_of(p.dst_table, p.dst_mpps, lo, dst_tok / kPageSize);
        ok = sp >= 0 && sp < p.src_pages && dp >= 0 && dp < p.dst_pages;
    }
    if (!ok) {
        if (p.bad_index) *p.bad_index = 1;
        return;
    }
    const size_t row_bytes = (size_t)p.row_chunks * 16;
    const size_t so = (((size_t)sp * p.n_kv_heads + h) * kPageSize + (src_tok % kPageSize)) * row_bytes + c * 16u;
    const size_t dof = (((size_t)dp * p.n_kv_heads + h) * kPageSize + (dst_tok % kPageSize)) * row_bytes + c * 16u;
    // planes: 2*l + (0 = K, 1 = V)
    const int pl0 = blockIdx.y * p.planes_per_group, pl1 = min(2 * p.n_layers, pl0 + p.planes_per_group);
    for (int pl = pl0; pl < pl1; pl += kGatherUnroll) {
        uint4 v[kGatherUnroll];
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int q = pl + u;
            if (q < pl1) v[u] = __ldg(reinterpret_cast<const uint4 *>(((q & 1) ? p.src_v : p.src_k) + (size_t)(q >> 1) * p.src_layer_stride + so));
        }
#pragma unroll
        for (int u = 0; u < kGatherUnroll; ++u) {
            const int q = pl + u;
            if (q < pl1) *reinterpret_cast<uint4 *>(((q & 1) ? p.dst_v : p.dst_k) + (size_t)(q >> 1) * p.dst_layer_stride + dof) = v[u];
        }
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
                                   int32_t *bad_index, void *stream) {
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
    if ((long long)total_keep > (long long)batch * dst->max_pages_per_seq * kPageSize)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: total_keep %d exceeds the destination's capacity (%d sequences x %d pages)",
                    total_keep, batch, dst->max_pages_per_seq);
    for (const hippo_kv_cache_t *kv : {src, dst})
        if (!kv->page_table && (long long)batch * kv->max_pages_per_seq > kv->n_pages)
            return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: identity page mapping needs batch*max_pages_per_seq <= n_pages");
    if (total_keep == 0) return HIPPO_OK;
    if (!keep_idx || !keep_offsets) return fail(HIPPO_ERR_INVALID_ARG, "hippo_gather_kv: null index arrays");

    GatherParams p;
    p.src_k = (const char *)src->k_pages; p.src_v = (const char *)src->v_pages;
    p.dst_k = (char *)dst->k_pages; p.dst_v = (char *)dst->v_pages;
    p.src_table = src->page_table; p.dst_table = dst->page_table;
    p.keep_idx = keep_idx; p.keep_offsets = keep_offsets; p.bad_index = bad_index;
    p.src_pages = src->n_pages; p.dst_pages = dst->n_pages;
    p.src_layer_stride = src_layer_stride_bytes; p.dst_layer_stride = dst_layer_stride_bytes;
    p.n_layers = n_layers; p.batch = batch; p.total_keep = total_keep; p.n_kv_heads = src->n_kv_heads;
    p.row_chunks = (int)(row_bytes / 16); p.src_mpps = src->max_pages_per_seq; p.dst_mpps = dst->max_pages_per_seq;
    const long long per_plane = (long long)total_keep * p.n_kv_heads * p.row_chunks;
    if (per_plane > 0x7fffffffLL) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_gather_kv: more than 2^31 16-byte items per layer");
    if (2 * n_layers > 65535) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_gather_kv: too many layers for one launch");
    // plane groups: all planes in one thread when the items alone fill the machine (8 blocks per SM), else split
    const long long bx = (per_plane + kGatherThreads - 1) / kGatherThreads;
    long long gy = ((long long)kNumSMs * 8 + bx - 1) / bx;
    if (gy > 2 * n_layers) gy = 2 * n_layers;
    if (gy < 1) gy = 1;
    p.planes_per_group = (int)((2 * n_layers + gy - 1) / gy);
    gy = (2 * n_layers + p.planes_per_group - 1) / p.planes_per_group;
    if (bx > 0x7fffffffLL || gy > 65535) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_gather_kv: grid too large");
    gather_kv_kernel<<<dim3((unsigned)bx, (unsigned)gy), kGatherThreads, 0, (cudaStream_t)stream>>>(p);
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}
