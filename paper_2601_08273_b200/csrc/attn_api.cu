// hippo_verify_attention / hippo_draft_attention: argument checks and kernel selection.
#include <math.h>

#include "common.cuh"

namespace hippo {

static int32_t check_cache(const hippo_kv_cache_t *kv, const char *who) {
    if (!kv) return fail(HIPPO_ERR_INVALID_ARG, "%s: null kv cache descriptor", who);
    if (kv->struct_size != sizeof(hippo_kv_cache_t))
        return fail(HIPPO_ERR_INVALID_ARG, "%s: kv struct_size %u != %zu", who, kv->struct_size, sizeof(hippo_kv_cache_t));
    if (kv->dtype != HIPPO_DTYPE_FP32 && kv->dtype != HIPPO_DTYPE_BF16)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: unknown dtype %d", who, kv->dtype);
    if (!kv->k_pages || !kv->v_pages) return fail(HIPPO_ERR_INVALID_ARG, "%s: null page pool", who);
    if (kv->n_kv_heads <= 0 || kv->head_dim <= 0 || kv->n_pages <= 0 || kv->max_pages_per_seq <= 0)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: non-positive cache dimension", who);
    if (((uintptr_t)kv->k_pages | (uintptr_t)kv->v_pages) & 127)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: page pools must be 128-byte aligned", who);
    return HIPPO_OK;
}

// Shape checks shared by the single-layer and the multi-layer calls; fills the shape part of the kernel arguments.
static int32_t check_shape(const char *who, int32_t batch, int32_t q_len, int32_t n_q_heads, const hippo_kv_cache_t *kv,
                           const int32_t *kv_len, const int32_t *kv_len_host, int32_t max_kv_len, float softmax_scale,
                           int32_t num_splits, AttnParams &p) {
    int32_t rc = check_cache(kv, who);
    if (rc != HIPPO_OK) return rc;
    if (batch <= 0 || q_len <= 0 || n_q_heads <= 0 || max_kv_len <= 0 || num_splits < 0)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: non-positive size", who);
    if (n_q_heads % kv->n_kv_heads) return fail(HIPPO_ERR_INVALID_ARG, "%s: n_q_heads %% n_kv_heads != 0", who);
    if ((long long)batch * kv->n_kv_heads > 16000) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: batch*n_kv_heads > 16000", who);
    p.kv_resident = 0;
    const int G = n_q_heads / kv->n_kv_heads, rows = q_len * G;
    if (rows > kMaxPackedRows)
        return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: q_len*group = %d > %d packed rows", who, rows, kMaxPackedRows);
    if (kv->head_dim % 32 || kv->head_dim > 256)
        return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: head_dim %d (need a multiple of 32, <= 256)", who, kv->head_dim);
    if ((long long)max_kv_len > (long long)kv->max_pages_per_seq * kPageSize)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: max_kv_len %d exceeds max_pages_per_seq*%d", who, max_kv_len, kPageSize);
    if (!kv->page_table && (long long)batch * kv->max_pages_per_seq > kv->n_pages)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: identity page mapping needs batch*max_pages_per_seq <= n_pages", who);
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return fail(HIPPO_ERR_INVALID_ARG, "%s: bad softmax_scale", who);
    if (kv_len_host)
        for (int b = 0; b < batch; ++b)
            if (kv_len_host[b] < 0 || kv_len_host[b] > max_kv_len)
                return fail(HIPPO_ERR_INVALID_ARG, "%s: kv_len_host[%d] = %d outside [0, max_kv_len]", who, b, kv_len_host[b]);
    p.k_pages = kv->k_pages; p.v_pages = kv->v_pages; p.page_table = kv->page_table;
    p.kv_len = kv_len; p.kv_len_host = kv_len_host;
    p.batch = batch; p.q_len = q_len; p.n_q_heads = n_q_heads; p.n_kv_heads = kv->n_kv_heads;
    p.head_dim = kv->head_dim; p.group = G; p.rows = rows;
    p.n_pages = kv->n_pages; p.max_pages_per_seq = kv->max_pages_per_seq; p.max_kv_len = max_kv_len;
    p.num_splits = num_splits;
    p.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kv->head_dim);
    return HIPPO_OK;
}

static int32_t attention_entry(const char *who, bool draft, int32_t batch, int32_t q_len, int32_t n_q_heads,
                               const void *q, const hippo_kv_cache_t *kv, const int32_t *kv_len,
                               const int32_t *kv_len_host, int32_t max_kv_len,
                               float softmax_scale, int32_t num_splits, void *out, float *lse, void *workspace,
                               size_t workspace_bytes, void *stream) {
    AttnParams p;
    int32_t rc = check_shape(who, batch, q_len, n_q_heads, kv, kv_len, kv_len_host, max_kv_len, softmax_scale, num_splits, p);
    if (rc != HIPPO_OK) return rc;
    if (!q || !out || !workspace) return fail(HIPPO_ERR_INVALID_ARG, "%s: null pointer", who);
    AttnWsLayout L = attn_ws_layout(batch, q_len, n_q_heads, kv->n_kv_heads, kv->head_dim);
    if (workspace_bytes < L.total)
        return fail(HIPPO_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu bytes", who, workspace_bytes, L.total);
    if ((uintptr_t)workspace & 255) return fail(HIPPO_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", who);
    p.q = q; p.out = out; p.lse = lse;
    p.kv_resident = draft ? 1 : 0;
    p.header = (WsHeader *)workspace;
    p.counters = (int32_t *)((char *)workspace + L.counters_off);
    p.partials = (float *)((char *)workspace + L.partials_off);
    cudaStream_t s = (cudaStream_t)stream;

    if (attn_small_supported(p, kv->dtype)) return launch_attn_small(p, s);   // few rows, short cache: latency-bound
    if (attn_tc_supported(p, kv->dtype)) return launch_attn_tc(p, s);
    // CUDA-core path: split so that the grid roughly fills the machine, bounded by the slots available.
    const int units = batch * kv->n_kv_heads;
    int max_splits = (int)(L.n_slots / units);
    int tiles = ceil_div(max_kv_len, 32);
    int want = num_splits > 0 ? num_splits : ceil_div(2 * kNumSMs, units);
    if (want > tiles) want = tiles;
    if (want > max_splits) want = max_splits;
    if (want < 1) want = 1;
    p.num_splits = want;
    return launch_attn_generic(p, kv->dtype, s);
}

}  // namespace hippo

extern "C" {

size_t hippo_attention_workspace_bytes(int32_t batch, int32_t q_len, int32_t n_q_heads, int32_t n_kv_heads,
                                       int32_t head_dim) {
    if (batch <= 0 || q_len <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 || n_q_heads % n_kv_heads) return 0;
    return hippo::attn_ws_layout(batch, q_len, n_q_heads, n_kv_heads, head_dim).total;
}

int32_t hippo_verify_attention(int32_t batch, int32_t q_len, int32_t n_q_heads, const void *q,
                               const hippo_kv_cache_t *kv, const int32_t *kv_len, const int32_t *kv_len_host,
                               int32_t max_kv_len, float softmax_scale, int32_t num_splits, void *out, float *lse,
                               void *workspace, size_t workspace_bytes, void *stream) {
    return hippo::attention_entry("hippo_verify_attention", false, batch, q_len, n_q_heads, q, kv, kv_len, kv_len_host, max_kv_len,
                                  softmax_scale, num_splits, out, lse, workspace, workspace_bytes, stream);
}

int32_t hippo_draft_attention(int32_t batch, int32_t q_len, int32_t n_q_heads, const void *q,
                              const hippo_kv_cache_t *kv, const int32_t *kv_len, const int32_t *kv_len_host,
                              int32_t max_kv_len, float softmax_scale, int32_t num_splits, void *out, float *lse,
                              void *workspace, size_t workspace_bytes, void *stream) {
    return hippo::attention_entry("hippo_draft_attention", true, batch, q_len, n_q_heads, q, kv, kv_len, kv_len_host, max_kv_len,
                                  softmax_scale, num_splits, out, lse, workspace, workspace_bytes, stream);
}

size_t hippo_verify_attention_layers_workspace_bytes(int32_t n_layers, int32_t batch, int32_t q_len, int32_t n_q_heads,
                                                     int32_t n_kv_heads, int32_t head_dim) {
    if (n_layers <= 0 || batch <= 0 || q_len <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0 ||
        n_q_heads % n_kv_heads)
        return 0;
    return hippo::attn_layers_ws_layout(n_layers, batch, q_len, n_q_heads, n_kv_heads, head_dim).total;
}

int32_t hippo_verify_attention_layers(int32_t n_layers, int32_t batch, int32_t q_len, int32_t n_q_heads,
                                      const void *const *q_layers, const hippo_kv_cache_t *kv_layers,
                                      const int32_t *kv_len, const int32_t *kv_len_host, int32_t max_kv_len,
                                      float softmax_scale, int32_t max_ctas, void *const *out_layers, float *const *lse_layers,
                                      void *workspace, size_t workspace_bytes, void *stream) {
    using namespace hippo;
    const char *who = "hippo_verify_attention_layers";
    if (n_layers <= 0 || max_ctas < 0) return fail(HIPPO_ERR_INVALID_ARG, "%s: n_layers <= 0 or max_ctas < 0", who);
    if (!q_layers || !kv_layers || !out_layers || !workspace) return fail(HIPPO_ERR_INVALID_ARG, "%s: null pointer", who);
    AttnParams p;
    for (int l = 0; l < n_layers; ++l) {
        AttnParams pl;
        int32_t rc = check_shape(who, batch, q_len, n_q_heads, &kv_layers[l], kv_len, kv_len_host, max_kv_len, softmax_scale, 0, pl);
        if (rc != HIPPO_OK) return rc;
        if (!q_layers[l] || !out_layers[l]) return fail(HIPPO_ERR_INVALID_ARG, "%s: null q or out pointer of layer %d", who, l);
        if (l == 0) { p = pl; continue; }
        const hippo_kv_cache_t &a = kv_layers[0], &b = kv_layers[l];
        if (a.dtype != b.dtype || a.n_kv_heads != b.n_kv_heads || a.head_dim != b.head_dim ||
            a.max_pages_per_seq != b.max_pages_per_seq || a.page_table != b.page_table)
            return fail(HIPPO_ERR_INVALID_ARG, "%s: layer %d differs from layer 0 in dtype, heads, head_dim or page table", who, l);
    }
    const hippo_kv_cache_t *kv = kv_layers;
    const AttnLayersWsLayout L = attn_layers_ws_layout(n_layers, batch, q_len, n_q_heads, kv->n_kv_heads, kv->head_dim);
    if (workspace_bytes < L.total)
        return fail(HIPPO_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu bytes", who, workspace_bytes, L.total);
    if ((uintptr_t)workspace & 255) return fail(HIPPO_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", who);
    if (attn_tc_layers_supported(p, kv->dtype) && !attn_small_supported(p, kv->dtype))
        return launch_attn_tc_layers(p, n_layers, q_layers, kv_layers, out_layers, lse_layers, max_ctas, workspace, (cudaStream_t)stream);
    // shapes outside the multi-layer kernel: one single-layer call per layer, same results
    for (int l = 0; l < n_layers; ++l) {
        int32_t rc = attention_entry(who, false, batch, q_len, n_q_heads, q_layers[l], &kv_layers[l], kv_len, kv_len_host, max_kv_len,
                                     softmax_scale, 0, out_layers[l], lse_layers ? lse_layers[l] : nullptr, workspace,
                                     workspace_bytes, stream);
        if (rc != HIPPO_OK) return rc;
    }
    return HIPPO_OK;
}

}  // extern "C"
