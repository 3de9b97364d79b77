// Status strings, per-thread error text and workspace header helpers.
#include <stdarg.h>
#include <stddef.h>
#include <string.h>

#include <atomic>

#include "common.cuh"

namespace hippo {

static thread_local char g_err[512] = {0};
static std::atomic<unsigned long long> g_launches{0};

void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
unsigned long long launches() { return g_launches.load(std::memory_order_relaxed); }

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

int32_t fail(int32_t status, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return status;
}

int32_t cuda_fail(cudaError_t e, const char *what) {
    snprintf(g_err, sizeof(g_err), "%s: %s (%s)", what, cudaGetErrorString(e), cudaGetErrorName(e));
    return HIPPO_ERR_CUDA;
}

}  // namespace hippo

extern "C" {

int32_t hippo_version(void) { return HIPPO_VERSION; }

const char *hippo_status_string(int32_t status) {
    switch (status) {
        case HIPPO_OK: return "ok";
        case HIPPO_ERR_INVALID_ARG: return "invalid argument";
        case HIPPO_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case HIPPO_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case HIPPO_ERR_CUDA: return "CUDA error";
        case HIPPO_ERR_TIMEOUT: return "device-side wait timed out";
        case HIPPO_ERR_UNIMPLEMENTED: return "not implemented";
        default: return "unknown status";
    }
}

const char *hippo_last_error(void) { return hippo::g_err; }

uint64_t hippo_launch_count(void) { return (uint64_t)hippo::launches(); }

int32_t hippo_workspace_status(const void *workspace, void *stream) {
    if (!workspace) return hippo::fail(HIPPO_ERR_INVALID_ARG, "hippo_workspace_status: null workspace");
    cudaStream_t s = (cudaStream_t)stream;
    hippo::WsHeader h;
    HIPPO_CUDA_TRY(cudaMemcpyAsync(&h, workspace, sizeof(int32_t) * 2, cudaMemcpyDeviceToHost, s));
    HIPPO_CUDA_TRY(cudaStreamSynchronize(s));
    if (h.status != 0) return hippo::fail(h.status, "device-side wait gave up (site %d)", h.where);
    return HIPPO_OK;
}

int32_t hippo_workspace_set_wait_limit(void *workspace, int64_t limit_ns, void *stream) {
    if (!workspace) return hippo::fail(HIPPO_ERR_INVALID_ARG, "hippo_workspace_set_wait_limit: null workspace");
    if (limit_ns < 0) return hippo::fail(HIPPO_ERR_INVALID_ARG, "hippo_workspace_set_wait_limit: negative limit");
    cudaStream_t s = (cudaStream_t)stream;
    long long v = (long long)limit_ns;
    HIPPO_CUDA_TRY(cudaMemcpyAsync((char *)workspace + offsetof(hippo::WsHeader, wait_limit_ns), &v, sizeof(v),
                                   cudaMemcpyHostToDevice, s));
    HIPPO_CUDA_TRY(cudaStreamSynchronize(s));   // `v` lives on this stack frame
    return HIPPO_OK;
}

int32_t hippo_workspace_reset(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace) return hippo::fail(HIPPO_ERR_INVALID_ARG, "hippo_workspace_reset: null workspace");
    if (workspace_bytes < hippo::kWsHeaderBytes)
        return hippo::fail(HIPPO_ERR_WORKSPACE_TOO_SMALL, "hippo_workspace_reset: %zu bytes < header", workspace_bytes);
    // header plus the arrival counters that follow it (bounded by 64 KiB; counters never extend further)
    size_t n = workspace_bytes < 65536 ? workspace_bytes : 65536;
    HIPPO_CUDA_TRY(cudaMemsetAsync(workspace, 0, n, (cudaStream_t)stream));
    return HIPPO_OK;
}

}  // extern "C"
