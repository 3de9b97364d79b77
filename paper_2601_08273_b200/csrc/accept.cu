// hippo_accept: lossless speculative acceptance (Section 3.2, Eq. 1 and the resampling rule that follows it).
//
//   P_j, Q_j = softmax(target row j), softmax(draft row j)            (temperature 1)
//   accept x_{j+1} iff u_accept[j] * Q_j[x] < P_j[x]                   (probability min(1, P/Q), Eq. 1)
//   first rejection at n < gamma: draw from norm(max(0, P_n - Q_n));   none: draw the bonus token from P_gamma
//   draw = inverse CDF in ascending token id: smallest t with cumsum_t > u_resample * total
//
// All probabilities, normalisers and CDFs are fp64 so that the decisions agree with an fp64 reference unless a
// uniform lands within ~1e-15 of a boundary.  Four small kernels over the vocabulary:
//   stats   per (sequence, logit row, 4096-token chunk): max and sum of exponentials
//   decide  per sequence: merge the chunk stats, run the accept tests, store n and the two normalisers of row n
//   wsum    per (sequence, chunk): total residual (or bonus) weight of the chunk, by the same in-order scan as `pick`
//   pick    per sequence: locate the chunk, then the token, where the CDF crosses u * total
#include <math.h>

#include <mutex>

#include "common.cuh"

namespace hippo {

constexpr int kAccThreads = 256;
constexpr int kAccPerThread = 16;
constexpr int kAccChunk = kAccThreads * kAccPerThread;  // 4096 vocabulary entries per chunk

struct RowInfo {
    double Mp, Zp, Mq, Zq;  // max logit and sum of exponentials of target row n / draft row n
    int32_t n;              // accepted count
    int32_t bonus;          // 1: n == gamma, draw from P_gamma
    int32_t pad[2];
};

struct AcceptParams {
    const float *tl, *dl, *ua, *ur;
    const int32_t *x;
    int32_t *n_acc, *out;
    double2 *stats;  // [B][2*gamma+1][n_chunks]: (max, sum exp)
    double *wsum;    // [B][n_chunks]
    RowInfo *info;   // [B]
    int B, gamma, V, n_chunks;
};

__device__ __forceinline__ const float *logit_row(const AcceptParams &p, int b, int r) {
    // r in [0, gamma]: target row r; r in (gamma, 2*gamma]: draft row r - gamma - 1
    return r <= p.gamma ? p.tl + ((size_t)b * (p.gamma + 1) + r) * p.V : p.dl + ((size_t)b * p.gamma + (r - p.gamma - 1)) * p.V;
}

// In-order inclusive scan over the block's threads (thread i holds element i).  Deterministic.
__device__ double block_scan_inclusive(double v, double *warp_tot /* [8] shared */, double *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
        double t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    __syncthreads();  // protect warp_tot from a previous use
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    double pre = 0.0, tot = 0.0;
    for (int w = 0; w < kAccThreads / 32; ++w) {
        if (w < warp) pre += warp_tot[w];
        tot += warp_tot[w];
    }
    *total = tot;
    return v + pre;
}

__global__ void __launch_bounds__(kAccThreads) accept_stats_kernel(const AcceptParams p) {
    __shared__ float smax[kAccThreads / 32];
    __shared__ double ssum[kAccThreads / 32];
    const int c = blockIdx.x, r = blockIdx.y, b = blockIdx.z, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *row = logit_row(p, b, r);
    float v[kAccPerThread];
    float m = -INFINITY;
#pragma unroll
    for (int e = 0; e < kAccPerThread; ++e) {
        int t = c * kAccChunk + e * kAccThreads + tid;
        v[e] = t < p.V ? row[t] : -INFINITY;
        m = fmaxf(m, v[e]);
    }
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) smax[warp] = m;
    __syncthreads();
    m = smax[0];
    for (int w = 1; w < kAccThreads / 32; ++w) m = fmaxf(m, smax[w]);
    double s = 0.0;
#pragma unroll
    for (int e = 0; e < kAccPerThread; ++e)
        if (v[e] != -INFINITY) s += exp((double)v[e] - (double)m);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) ssum[warp] = s;
    __syncthreads();
    if (tid == 0) {
        double tot = 0.0;
        for (int w = 0; w < kAccThreads / 32; ++w) tot += ssum[w];
        p.stats[((size_t)b * (2 * p.gamma + 1) + r) * p.n_chunks + c] = make_double2((double)m, tot);
    }
}

__global__ void __launch_bounds__(kAccThreads) accept_decide_kernel(const AcceptParams p) {
    extern __shared__ double rowstat[];  // [2*gamma+1][2]: M, Z
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_rows = 2 * p.gamma + 1;
    for (int r = warp; r < n_rows; r += kAccThreads / 32) {
        const double2 *st = p.stats + ((size_t)b * n_rows + r) * p.n_chunks;
        double M = -INFINITY;
        for (int c = lane; c < p.n_chunks; c += 32) M = fmax(M, st[c].x);
        for (int o = 16; o; o >>= 1) M = fmax(M, __shfl_xor_sync(0xffffffffu, M, o));
        double Z = 0.0;
        for (int c = lane; c < p.n_chunks; c += 32)
            if (st[c].x != -INFINITY) Z += st[c].y * exp(st[c].x - M);
        for (int o = 16; o; o >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, o);
        if (lane == 0) { rowstat[2 * r] = M; rowstat[2 * r + 1] = Z; }
    }
    __syncthreads();
    if (tid == 0) {
        const int32_t *x = p.x + (size_t)b * p.gamma;
        int32_t *out = p.out + (size_t)b * (p.gamma + 1);
        int n = 0;
        for (; n < p.gamma; ++n) {
            const int rq = p.gamma + 1 + n;
            const double P = exp((double)logit_row(p, b, n)[x[n]] - rowstat[2 * n]) / rowstat[2 * n + 1];
            const double Q = exp((double)logit_row(p, b, rq)[x[n]] - rowstat[2 * rq]) / rowstat[2 * rq + 1];
            const double u = (double)p.ua[(size_t)b * p.gamma + n];
            if (!(u * Q < P)) break;
            out[n] = x[n];
        }
        for (int j = n; j <= p.gamma; ++j) out[j] = -1;  // out[n] is filled by the pick kernel
        p.n_acc[b] = n;
        RowInfo ri;
        ri.n = n;
        ri.bonus = (n == p.gamma);
        ri.Mp = rowstat[2 * n]; ri.Zp = rowstat[2 * n + 1];
        if (n < p.gamma) { ri.Mq = rowstat[2 * (p.gamma + 1 + n)]; ri.Zq = rowstat[2 * (p.gamma + 1 + n) + 1]; }
        else { ri.Mq = 0.0; ri.Zq = 1.0; }
        ri.pad[0] = ri.pad[1] = 0;
        p.info[b] = ri;
    }
}

// Weight of token t in the distribution the emitted token is drawn from.  use_target_only: bonus row, or the
// degenerate rejection with P_n == Q_n everywhere.
__device__ __forceinline__ double draw_weight(const float *trow, const float *drow, int t, const RowInfo &ri, bool use_target_only) {
    const double P = exp((double)trow[t] - ri.Mp) / ri.Zp;
    if (use_target_only) return P;
    const double Q = exp((double)drow[t] - ri.Mq) / ri.Zq;
    const double w = P - Q;
    return w > 0.0 ? w : 0.0;
}

// Thread-local weights of one chunk (16 consecutive tokens per thread) and their in-order sum.
__device__ __forceinline__ double chunk_local(const float *trow, const float *drow, int c, int V, const RowInfo &ri,
                                              bool target_only, double *w) {
    double s = 0.0;
    const int t0 = c * kAccChunk + threadIdx.x * kAccPerThread;
#pragma unroll
    for (int e = 0; e < kAccPerThread; ++e) {
        const int t = t0 + e;
        w[e] = t < V ? draw_weight(trow, drow, t, ri, target_only) : 0.0;
        s += w[e];
    }
    return s;
}

__global__ void __launch_bounds__(kAccThreads) accept_wsum_kernel(const AcceptParams p) {
    __shared__ double warp_tot[kAccThreads / 32];
    const int c = blockIdx.x, b = blockIdx.y;
    const RowInfo ri = p.info[b];
    const float *trow = logit_row(p, b, ri.n);
    const float *drow = ri.bonus ? nullptr : logit_row(p, b, p.gamma + 1 + ri.n);
    double w[kAccPerThread], total;
    double s = chunk_local(trow, drow, c, p.V, ri, ri.bonus != 0, w);
    block_scan_inclusive(s, warp_tot, &total);
    if (threadIdx.x == 0) p.wsum[(size_t)b * p.n_chunks + c] = total;
}

__global__ void __launch_bounds__(kAccThreads) accept_pick_kernel(const AcceptParams p) {
    __shared__ double warp_tot[kAccThreads / 32];
    __shared__ double s_prefix, s_target;
    __shared__ int s_chunk, s_tok, s_target_only;
    const int b = blockIdx.x, tid = threadIdx.x;
    const RowInfo ri = p.info[b];
    const float *trow = logit_row(p, b, ri.n);
    const float *drow = ri.bonus ? nullptr : logit_row(p, b, p.gamma + 1 + ri.n);
    double *wsum = p.wsum + (size_t)b * p.n_chunks;
    double w[kAccPerThread], total;

    if (tid == 0) {
        double Z = 0.0;
        for (int c = 0; c < p.n_chunks; ++c) Z += wsum[c];
        s_target_only = ri.bonus || !(Z > 0.0);
        s_prefix = Z;
    }
    __syncthreads();
    const bool target_only = s_target_only != 0;
    if (target_only && !ri.bonus) {
        // residual is identically zero (P_n == Q_n): fall back to P_n; recompute the chunk totals
        for (int c = 0; c < p.n_chunks; ++c) {
            double s = chunk_local(trow, drow, c, p.V, ri, true, w);
            block_scan_inclusive(s, warp_tot, &total);
            if (tid == 0) wsum[c] = total;
        }
        __syncthreads();
    }
    if (tid == 0) {
        double Z = 0.0;
        for (int c = 0; c < p.n_chunks; ++c) Z += wsum[c];
        const double target = (double)p.ur[b] * Z;
        double cum = 0.0;
        int chunk = -1;
        for (int c = 0; c < p.n_chunks; ++c) {
            if (cum + wsum[c] > target) { chunk = c; break; }
            cum += wsum[c];
        }
        s_chunk = chunk; s_prefix = cum; s_target = target; s_tok = 0x7fffffff;
    }
    __syncthreads();
    int tok = -1;
    if (s_chunk >= 0) {
        const int c = s_chunk;
        double s = chunk_local(trow, drow, c, p.V, ri, target_only, w);
        double incl = block_scan_inclusive(s, warp_tot, &total);
        double run = s_prefix + (incl - s);  // CDF just before this thread's first token
        int mine = 0x7fffffff;
#pragma unroll
        for (int e = 0; e < kAccPerThread; ++e) {
            run += w[e];
            if (mine == 0x7fffffff && run > s_target) mine = c * kAccChunk + tid * kAccPerThread + e;
        }
        if (mine != 0x7fffffff) atomicMin(&s_tok, mine);
        __syncthreads();
        if (s_tok != 0x7fffffff) tok = s_tok;
    }
    if (tok < 0 && tid == 0) {
        // the CDF never exceeded the target (possible only through rounding): last token with positive weight
        for (int t = p.V - 1; t >= 0; --t)
            if (draw_weight(trow, drow, t, ri, target_only) > 0.0) { tok = t; break; }
    }
    if (tid == 0) p.out[(size_t)b * (p.gamma + 1) + ri.n] = tok;
}

struct AcceptWs { size_t stats_off, wsum_off, info_off, total; int n_chunks; };
static AcceptWs accept_ws(int B, int gamma, int V) {
    AcceptWs w;
    w.n_chunks = ceil_div(V, kAccChunk);
    w.stats_off = kWsHeaderBytes;
    w.wsum_off = w.stats_off + align_up((size_t)B * (2 * gamma + 1) * w.n_chunks * sizeof(double2), 256);
    w.info_off = w.wsum_off + align_up((size_t)B * w.n_chunks * sizeof(double), 256);
    w.total = w.info_off + align_up((size_t)B * sizeof(RowInfo), 256);
    return w;
}

}  // namespace hippo

extern "C" {

size_t hippo_accept_workspace_bytes(int32_t batch, int32_t gamma, int32_t vocab) {
    if (batch <= 0 || gamma < 0 || vocab <= 0) return 0;
    return hippo::accept_ws(batch, gamma, vocab).total;
}

int32_t hippo_accept(int32_t batch, int32_t gamma, int32_t vocab, const float *target_logits,
                     const float *draft_logits, const int32_t *draft_tokens, const float *u_accept,
                     const float *u_resample, int32_t mode, int32_t *n_accepted, int32_t *out_tokens,
                     void *workspace, size_t workspace_bytes, void *stream) {
    using namespace hippo;
    if (batch <= 0 || gamma < 0 || vocab <= 0) return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept: bad sizes");
    if (mode != HIPPO_ACCEPT_SAMPLE) return fail(HIPPO_ERR_UNIMPLEMENTED, "hippo_accept: mode %d", mode);
    if (!target_logits || !u_resample || !n_accepted || !out_tokens || !workspace)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept: null pointer");
    if (gamma > 0 && (!draft_logits || !draft_tokens || !u_accept))
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept: null draft arrays with gamma > 0");
    if (gamma > 64) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_accept: gamma > 64");
    if ((uintptr_t)workspace & 255) return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept: workspace must be 256-byte aligned");
    AcceptWs w = accept_ws(batch, gamma, vocab);
    if (workspace_bytes < w.total)
        return fail(HIPPO_ERR_WORKSPACE_TOO_SMALL, "hippo_accept: workspace %zu < %zu bytes", workspace_bytes, w.total);
    if (batch > 65535 || 2 * gamma + 1 > 65535) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_accept: batch too large");
    AcceptParams p;
    p.tl = target_logits; p.dl = draft_logits; p.ua = u_accept; p.ur = u_resample; p.x = draft_tokens;
    p.n_acc = n_accepted; p.out = out_tokens;
    p.stats = (double2 *)((char *)workspace + w.stats_off);
    p.wsum = (double *)((char *)workspace + w.wsum_off);
    p.info = (RowInfo *)((char *)workspace + w.info_off);
    p.B = batch; p.gamma = gamma; p.V = vocab; p.n_chunks = w.n_chunks;
    cudaStream_t s = (cudaStream_t)stream;
    accept_stats_kernel<<<dim3(w.n_chunks, 2 * gamma + 1, batch), kAccThreads, 0, s>>>(p);
    accept_decide_kernel<<<batch, kAccThreads, (2 * gamma + 1) * 2 * sizeof(double), s>>>(p);
    accept_wsum_kernel<<<dim3(w.n_chunks, batch), kAccThreads, 0, s>>>(p);
    accept_pick_kernel<<<batch, kAccThreads, 0, s>>>(p);
    count_launches(4);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}

}  // extern "C"

// ---- hippo_accept_noalloc: the same acceptance step for callers that cannot provide a workspace -----------------
//
// Some callers have no way to obtain scratch memory at the moment they need to accept a draft: a decode loop whose
// device memory was handed in full to a serving engine's pool at start-up, a plug-in whose host forbids cudaMalloc
// (it synchronises the whole device and would stall the draft and verify streams), or glue code that only sees the
// logits and has no allocator handle at all.  For them the scratch lives in the library image itself: one
// file-scope device array per GPU that loads libhippo.so, held until the process exits.
namespace hippo {

constexpr size_t kNoAllocScratchBytes = HIPPO_ACCEPT_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_accept_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
static void *g_scratch_addr[kMaxDevices] = {nullptr};   // device address of g_accept_scratch, per device ordinal
static std::mutex g_scratch_mutex;

// In host code `g_accept_scratch` is only a handle for the runtime, not an address a kernel could use.  The real
// device address differs per GPU and is looked up once per device, with that device current.
static int32_t noalloc_scratch(void **out) {
    int dev = -1;
    HIPPO_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_accept_noalloc: device ordinal %d >= %d", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        HIPPO_CUDA_TRY(cudaGetSymbolAddress((void **)&ptr, g_accept_scratch));
        if (!ptr || ((uintptr_t)ptr & 255)) return fail(HIPPO_ERR_CUDA, "hippo_accept_noalloc: bad scratch address %p", ptr);
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return HIPPO_OK;
}

}  // namespace hippo

extern "C" int32_t hippo_accept_noalloc(int32_t batch, int32_t gamma, int32_t vocab, const float *target_logits,
                                        const float *draft_logits, const int32_t *draft_tokens, const float *u_accept,
                                        const float *u_resample, int32_t mode, int32_t *n_accepted, int32_t *out_tokens,
                                        void *stream) {
    using namespace hippo;
    if (batch <= 0 || gamma < 0 || vocab <= 0) return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept_noalloc: bad sizes");
    if (mode != HIPPO_ACCEPT_SAMPLE) return fail(HIPPO_ERR_UNIMPLEMENTED, "hippo_accept_noalloc: mode %d", mode);
    if (!target_logits || !u_resample || !n_accepted || !out_tokens)
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept_noalloc: null pointer");
    if (gamma > 0 && (!draft_logits || !draft_tokens || !u_accept))
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept_noalloc: null draft arrays with gamma > 0");
    if (gamma > 64 || batch > 65535) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "hippo_accept_noalloc: gamma > 64 or batch > 65535");
    const AcceptWs w = accept_ws(batch, gamma, vocab);
    if (w.total > kNoAllocScratchBytes)
        return fail(HIPPO_ERR_WORKSPACE_TOO_SMALL,
                    "hippo_accept_noalloc: batch %d x gamma %d x vocab %d needs %zu bytes of scratch, the built-in array "
                    "holds %zu; use hippo_accept with a caller-owned workspace",
                    batch, gamma, vocab, w.total, kNoAllocScratchBytes);
    void *scratch = nullptr;
    const int32_t rc = noalloc_scratch(&scratch);
    if (rc != HIPPO_OK) return rc;
    // Every word the kernels read from the scratch is written earlier in the same call (chunk statistics, chunk
    // weights, the per-sequence record), so nothing has to be cleared although the array keeps the previous
    // call's contents.
    AcceptParams p;
    p.tl = target_logits; p.dl = draft_logits; p.ua = u_accept; p.ur = u_resample; p.x = draft_tokens;
    p.n_acc = n_accepted; p.out = out_tokens;
    p.stats = (double2 *)((char *)scratch + w.stats_off);
    p.wsum = (double *)((char *)scratch + w.wsum_off);
    p.info = (RowInfo *)((char *)scratch + w.info_off);
    p.B = batch; p.gamma = gamma; p.V = vocab; p.n_chunks = w.n_chunks;
    cudaStream_t s = (cudaStream_t)stream;
    accept_stats_kernel<<<dim3(w.n_chunks, 2 * gamma + 1, batch), kAccThreads, 0, s>>>(p);
    accept_decide_kernel<<<batch, kAccThreads, (2 * gamma + 1) * 2 * sizeof(double), s>>>(p);
    accept_wsum_kernel<<<dim3(w.n_chunks, batch), kAccThreads, 0, s>>>(p);
    accept_pick_kernel<<<batch, kAccThreads, 0, s>>>(p);
    count_launches(4);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}
