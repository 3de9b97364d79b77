// Shared host/device helpers of the hippo CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <atomic>
#include <stdint.h>
#include <stdio.h>

#include "hippo.h"

namespace hippo {

constexpr int kPageSize = HIPPO_PAGE_SIZE;
constexpr int kMaxPackedRows = HIPPO_MAX_PACKED_ROWS;
constexpr int kNumSMs = 148;                 // B200
constexpr size_t kWsHeaderBytes = 256;       // status word + padding
constexpr int kExtraSlots = 4 * kNumSMs;     // partial-result slots beyond one per (sequence, kv head)

// First bytes of every workspace.
struct WsHeader {
    int32_t status;          // 0, or HIPPO_ERR_TIMEOUT once a bounded wait gave up
    int32_t where;           // code of the wait that gave up (debugging aid)
    long long wait_limit_ns; // 0: the built-in limit; else the limit of the bounded waits (hippo_workspace_set_wait_limit)
    int32_t pad[60];
};
static_assert(sizeof(WsHeader) == kWsHeaderBytes, "header size");

// Number of kernels this library has launched in this process (diagnostics; see hippo_launch_count()).
void count_launches(int n);
void set_error(const char *fmt, ...);
int32_t fail(int32_t status, const char *fmt, ...);
int32_t cuda_fail(cudaError_t e, const char *what);

#define HIPPO_CUDA_TRY(expr)                                   \
    do {                                                       \
        cudaError_t e_ = (expr);                               \
        if (e_ != cudaSuccess) return ::hippo::cuda_fail(e_, #expr); \
    } while (0)

// Function attributes and occupancy answers belong to a device: one flag per device ordinal, set after the first
// successful set-up there.  Two threads racing on a device's first call both do the set-up, which is harmless.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    std::atomic<bool> done[kMaxDevices];
    // true when the current device still needs its set-up; dev receives the ordinal (-1: unknown, always set up)
    bool needed(int &dev) {
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { dev = -1; return true; }
        return !done[dev].load(std::memory_order_acquire);
    }
    void mark(int dev) { if (dev >= 0) done[dev].store(true, std::memory_order_release); }
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// One partial-result slot: m[rows_padded] | l[rows_padded] | O[rows][head_dim] (fp32), rows_padded = rows rounded up
// to a multiple of 4 so that every part starts on a 16-byte boundary.
__host__ __device__ inline int slot_rows_padded(int rows) { return (rows + 3) & ~3; }
__host__ __device__ inline size_t slot_float_count(int rows, int head_dim) {
    return 2 * (size_t)slot_rows_padded(rows) + (size_t)rows * head_dim;
}

// Layout of an attention workspace: header | per-unit slot table | partial slots.
struct AttnWsLayout {
    size_t counters_off, counters_bytes, partials_off, slot_floats, n_slots, total;
};
inline AttnWsLayout attn_ws_layout(int batch, int q_len, int n_q_heads, int n_kv_heads, int head_dim) {
    AttnWsLayout L;
    int rows = q_len * (n_q_heads / n_kv_heads);
    L.counters_off = kWsHeaderBytes;
    L.counters_bytes = align_up((size_t)batch * n_kv_heads * 2 * sizeof(int32_t), 256);   // per unit: first slot, contributors
    L.partials_off = L.counters_off + L.counters_bytes;
    L.slot_floats = slot_float_count(rows, head_dim);
    L.n_slots = (size_t)batch * n_kv_heads + kExtraSlots;
    L.total = L.partials_off + align_up(L.n_slots * L.slot_floats * sizeof(float), 256);
    return L;
}

// Arguments shared by the attention kernels.
struct AttnParams {
    const void *q;
    void *out;
    float *lse;
    const void *k_pages;
    const void *v_pages;
    const int32_t *page_table;   // may be null: identity
    const int32_t *kv_len;
    const int32_t *kv_len_host;  // may be null: host copy of kv_len, used only to plan the launch
    WsHeader *header;
    int32_t *counters;
    float *partials;             // n_slots x slot_float_count(rows, D) floats
    int batch, q_len, n_q_heads, n_kv_heads, head_dim, group, rows;
    int n_pages, max_pages_per_seq, max_kv_len;
    int num_splits;
    int kv_resident;             // the cache is small and read again call after call (draft): ask L2 to keep it; else it streams
    float scale;
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_from_float(float *p, float x) { *p = x; }
__device__ __forceinline__ void store_from_float(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ int page_of(const int32_t *page_table, int max_pages_per_seq, int b, int logical_page) {
    return page_table ? page_table[(size_t)b * max_pages_per_seq + logical_page] : b * max_pages_per_seq + logical_page;
}

// entry points implemented per translation unit
int32_t launch_attn_generic(const AttnParams &p, int dtype, cudaStream_t stream);
int32_t launch_attn_combine(const AttnParams &p, int dtype, int n_splits, cudaStream_t stream);
int32_t launch_attn_tc(const AttnParams &p, cudaStream_t stream);
bool attn_tc_supported(const AttnParams &p, int dtype);
// several layers in one launch: header | per-unit slot table | done[layers][units], merged[layers] | slot sets
struct AttnLayersWsLayout {
    size_t counters_off, done_off, done_bytes, partials_off, slot_floats, slots_per_set, total;
};
AttnLayersWsLayout attn_layers_ws_layout(int n_layers, int batch, int q_len, int n_q_heads, int n_kv_heads, int head_dim);
bool attn_tc_layers_supported(const AttnParams &p, int dtype);
int32_t launch_attn_tc_layers(const AttnParams &p, int n_layers, const void *const *q, const hippo_kv_cache_t *kv,
                              void *const *out, float *const *lse, int max_ctas, void *workspace, cudaStream_t stream);
int32_t launch_attn_small(const AttnParams &p, cudaStream_t stream);
bool attn_small_supported(const AttnParams &p, int dtype);

}  // namespace hippo
