// hippo_accept: lossless speculative acceptance (Section 3.2, Eq. 1 and the resampling rule that follows it).
//
//   P_j, Q_j = softmax(target row j), softmax(draft row j)            (temperature 1)
//   accept x_{j+1} iff u_accept[j] * Q_j[x] < P_j[x]                   (probability min(1, P/Q), Eq. 1)
//   first rejection at n < gamma: draw from norm(max(0, P_n - Q_n));   none: draw the bonus token from P_gamma
//   draw = inverse CDF in ascending token id: smallest t with cumsum_t > u_resample * total
//
// All probabilities, normalisers and CDFs are fp64 so that the decisions agree with an fp64 reference unless a
// uniform lands within ~1e-15 of a boundary.  Three kernels over the vocabulary, chained with programmatic
// dependent launches (each waits for its predecessor before it reads anything):
//   stats   per (sequence, logit row, 4096-token chunk): max and sum of exponentials
//   weigh   per (sequence, chunk): every CTA merges the chunk stats of its sequence and runs the accept tests
//           itself (a few hundred values; cheaper than a launch of its own), then scans the residual (or bonus)
//           weights of its chunk in token order and stores the running sum after each thread's 16 tokens
//   pick    per sequence: locate the chunk, then the 16-token group, then the token where the CDF crosses
//           u * total; only that one group's weights are evaluated again
#include <math.h>

#include <atomic>
#include <mutex>

#include "common.cuh"

namespace hippo {

constexpr int kAccThreads = 256;
constexpr int kAccPerThread = 16;
constexpr int kAccChunk = kAccThreads * kAccPerThread;  // 4096 vocabulary entries per chunk
constexpr int kAccMaxRows = 2 * 64 + 1;
constexpr bool kAcceptFusedByDefault = false;

struct RowInfo {
    double Mp, Zp, Mq, Zq;  // max logit and 1 / (sum of exponentials) of target row n / draft row n
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
    double *tscan;   // [B][n_chunks][kAccThreads]: in-chunk running sum after each thread's tokens
    RowInfo *info;   // [B]
    int B, gamma, V, n_chunks;
};

__device__ __forceinline__ const float *logit_row(const AcceptParams &p, int b, int r) {
    // r in [0, gamma]: target row r; r in (gamma, 2*gamma]: draft row r - gamma - 1
    return r <= p.gamma ? p.tl + ((size_t)b * (p.gamma + 1) + r) * p.V : p.dl + ((size_t)b * p.gamma + (r - p.gamma - 1)) * p.V;
}

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

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

// Max and sum of exponentials of one 4096-token chunk of one logit row.
__device__ void stats_item(const AcceptParams &p, int b, int r, int c) {
    __shared__ float smax[kAccThreads / 32];
    __shared__ double ssum[kAccThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __syncthreads();   // the shared arrays may still be read by the previous item
    const float *row = logit_row(p, b, r);
    float v[kAccPerThread];
    float m = -INFINITY;
    if ((c + 1) * kAccChunk <= p.V && (((uintptr_t)row) & 15) == 0 && (p.V & 3) == 0) {
        // full chunk, 16-byte aligned: four float4 loads per thread
#pragma unroll
        for (int e4 = 0; e4 < kAccPerThread / 4; ++e4) {
            const float4 t = __ldg(reinterpret_cast<const float4 *>(row + c * kAccChunk) + e4 * kAccThreads + tid);
            v[4 * e4] = t.x; v[4 * e4 + 1] = t.y; v[4 * e4 + 2] = t.z; v[4 * e4 + 3] = t.w;
        }
    } else {
#pragma unroll
        for (int e = 0; e < kAccPerThread; ++e) {
            const int t = c * kAccChunk + e * kAccThreads + tid;
            v[e] = t < p.V ? row[t] : -INFINITY;
        }
    }
#pragma unroll
    for (int e = 0; e < kAccPerThread; ++e) m = fmaxf(m, v[e]);
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

__global__ void __launch_bounds__(kAccThreads) accept_stats_kernel(const AcceptParams p) {
    pdl_wait();
    pdl_trigger();
    stats_item(p, blockIdx.z, blockIdx.y, blockIdx.x);
}

// Weight of token t in the distribution the emitted token is drawn from.  use_target_only: bonus row, or the
// degenerate rejection with P_n == Q_n everywhere.
__device__ __forceinline__ double weight_of(float tl, float dl, const RowInfo &ri, bool use_target_only) {
    const double P = exp((double)tl - ri.Mp) * ri.Zp;
    if (use_target_only) return P;
    const double Q = exp((double)dl - ri.Mq) * ri.Zq;
    const double w = P - Q;
    return w > 0.0 ? w : 0.0;
}
__device__ __forceinline__ double draw_weight(const float *trow, const float *drow, int t, const RowInfo &ri, bool use_target_only) {
    return weight_of(trow[t], use_target_only ? 0.f : drow[t], ri, use_target_only);
}

// Thread-local weights of one chunk (16 consecutive tokens per thread) and their in-order sum.
__device__ __forceinline__ double chunk_local(const float *trow, const float *drow, int c, int V, const RowInfo &ri,
                                              bool target_only, double *w) {
    double s = 0.0;
    const int t0 = c * kAccChunk + threadIdx.x * kAccPerThread;
    float tv[kAccPerThread], dv[kAccPerThread];
    const bool vec = t0 + kAccPerThread <= V && (((uintptr_t)(trow + t0) | (target_only ? 0 : (uintptr_t)(drow + t0))) & 15) == 0;
    if (vec) {
#pragma unroll
        for (int e4 = 0; e4 < kAccPerThread / 4; ++e4) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(trow + t0) + e4);
            tv[4 * e4] = a.x; tv[4 * e4 + 1] = a.y; tv[4 * e4 + 2] = a.z; tv[4 * e4 + 3] = a.w;
            float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
            if (!target_only) d = __ldg(reinterpret_cast<const float4 *>(drow + t0) + e4);
            dv[4 * e4] = d.x; dv[4 * e4 + 1] = d.y; dv[4 * e4 + 2] = d.z; dv[4 * e4 + 3] = d.w;
        }
    } else {
#pragma unroll
        for (int e = 0; e < kAccPerThread; ++e) {
            const int t = t0 + e;
            tv[e] = t < V ? trow[t] : 0.f;
            dv[e] = (t < V && !target_only) ? drow[t] : 0.f;
        }
    }
#pragma unroll
    for (int e = 0; e < kAccPerThread; ++e) {
        w[e] = t0 + e < V ? weight_of(tv[e], dv[e], ri, target_only) : 0.0;
        s += w[e];
    }
    return s;
}

// Merge of the chunk statistics of every logit row of sequence b and the sequential accept tests.  Run by all
// threads of a block; the result is identical in every block of the sequence (same data, same order).
__device__ RowInfo decide_rows(const AcceptParams &p, int b, double *rowstat /* shared [2*gamma+1][2] */, int *s_n) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    if (warp == 0) {
        // lane j tests draft token j (all loads independent), then the first failing lane is n
        const int32_t *x = p.x + (size_t)b * p.gamma;
        int n = p.gamma;
        for (int j0 = 0; j0 < p.gamma; j0 += 32) {
            const int j = j0 + lane;
            bool accept = true;
            if (j < p.gamma) {
                const int rq = p.gamma + 1 + j, tok = x[j];
                // a token id outside the vocabulary (a fault upstream) is never looked up: it counts as rejected
                accept = false;
                if ((unsigned)tok < (unsigned)p.V) {
                    const double P = exp((double)logit_row(p, b, j)[tok] - rowstat[2 * j]) / rowstat[2 * j + 1];
                    const double Q = exp((double)logit_row(p, b, rq)[tok] - rowstat[2 * rq]) / rowstat[2 * rq + 1];
                    const double u = (double)p.ua[(size_t)b * p.gamma + j];
                    accept = u * Q < P;
                }
            }
            const unsigned rejected = __ballot_sync(0xffffffffu, !accept);
            if (rejected) { n = j0 + __ffs(rejected) - 1; break; }
        }
        if (lane == 0) *s_n = n;
    }
    __syncthreads();
    RowInfo ri;
    ri.n = *s_n;
    ri.bonus = (ri.n == p.gamma);
    ri.Mp = rowstat[2 * ri.n]; ri.Zp = 1.0 / rowstat[2 * ri.n + 1];
    if (ri.n < p.gamma) { ri.Mq = rowstat[2 * (p.gamma + 1 + ri.n)]; ri.Zq = 1.0 / rowstat[2 * (p.gamma + 1 + ri.n) + 1]; }
    else { ri.Mq = 0.0; ri.Zq = 1.0; }
    ri.pad[0] = ri.pad[1] = 0;
    return ri;
}

// Residual (or bonus) weights of one chunk of sequence b, scanned in token order.  Every caller re-derives the row
// normalisers and the accept decisions of the sequence (same data, same order: identical everywhere).
__device__ void weigh_item(const AcceptParams &p, int b, int c) {
    __shared__ double rowstat[2 * kAccMaxRows];
    __shared__ double warp_tot[kAccThreads / 32];
    __shared__ int s_n;
    const int tid = threadIdx.x;
    __syncthreads();   // the shared arrays may still be read by the previous item
    const RowInfo ri = decide_rows(p, b, rowstat, &s_n);
    if (c == 0 && tid == 0) {
        const int32_t *x = p.x + (size_t)b * p.gamma;
        int32_t *out = p.out + (size_t)b * (p.gamma + 1);
        for (int j = 0; j < ri.n; ++j) out[j] = x[j];
        for (int j = ri.n; j <= p.gamma; ++j) out[j] = -1;  // out[n] is filled by the pick step
        p.n_acc[b] = ri.n;
        p.info[b] = ri;
    }
    const float *trow = logit_row(p, b, ri.n);
    const float *drow = ri.bonus ? nullptr : logit_row(p, b, p.gamma + 1 + ri.n);
    double w[kAccPerThread], total;
    double s = chunk_local(trow, drow, c, p.V, ri, ri.bonus != 0, w);
    const double incl = block_scan_inclusive(s, warp_tot, &total);
    p.tscan[((size_t)b * p.n_chunks + c) * kAccThreads + tid] = incl;
    if (tid == 0) p.wsum[(size_t)b * p.n_chunks + c] = total;
}

__global__ void __launch_bounds__(kAccThreads) accept_weigh_kernel(const AcceptParams p) {
    pdl_wait();
    pdl_trigger();
    weigh_item(p, blockIdx.y, blockIdx.x);
}

// The emitted token of sequence b: chunk, 16-token group and token where the CDF crosses u * total.  ws: n_chunks doubles of
// shared memory.
__device__ void pick_item(const AcceptParams &p, int b, double *ws) {
    __shared__ double warp_tot[kAccThreads / 32];
    __shared__ double s_prefix, s_target;
    __shared__ int s_chunk, s_tok, s_target_only;
    const int tid = threadIdx.x;
    __syncthreads();   // the shared arrays may still be read by the previous item
    const RowInfo ri = p.info[b];
    const float *trow = logit_row(p, b, ri.n);
    const float *drow = ri.bonus ? nullptr : logit_row(p, b, p.gamma + 1 + ri.n);
    double *wsum = p.wsum + (size_t)b * p.n_chunks;
    double w[kAccPerThread], total;
    for (int c = tid; c < p.n_chunks; c += kAccThreads) ws[c] = wsum[c];
    __syncthreads();
    if (tid == 0) {
        double Z = 0.0;
        for (int c = 0; c < p.n_chunks; ++c) Z += ws[c];
        s_target_only = ri.bonus || !(Z > 0.0);
    }
    __syncthreads();
    const bool target_only = s_target_only != 0;
    if (target_only && !ri.bonus) {
        // residual is identically zero (P_n == Q_n): fall back to P_n; recompute the chunk totals
        for (int c = 0; c < p.n_chunks; ++c) {
            double s = chunk_local(trow, drow, c, p.V, ri, true, w);
            block_scan_inclusive(s, warp_tot, &total);
            if (tid == 0) ws[c] = total;
        }
        __syncthreads();
    }
    if (tid == 0) {
        double Z = 0.0;
        for (int c = 0; c < p.n_chunks; ++c) Z += ws[c];
        const double target = (double)p.ur[b] * Z;
        double cum = 0.0;
        int chunk = -1;
        for (int c = 0; c < p.n_chunks; ++c) {
            if (cum + ws[c] > target) { chunk = c; break; }
            cum += ws[c];
        }
        s_chunk = chunk; s_prefix = cum; s_target = target; s_tok = 0x7fffffff;
    }
    __syncthreads();
    int tok = -1;
    if (s_chunk >= 0 && !(target_only && !ri.bonus)) {
        // the 16-token group: first thread of the chunk whose stored running sum exceeds the target
        const int c = s_chunk;
        const double incl = p.tscan[((size_t)b * p.n_chunks + c) * kAccThreads + tid];
        const bool over = s_prefix + incl > s_target;
        const unsigned bal = __ballot_sync(0xffffffffu, over);
        __shared__ int s_first[kAccThreads / 32];
        if ((tid & 31) == 0) s_first[tid >> 5] = bal ? (tid & ~31) + __ffs(bal) - 1 : 0x7fffffff;
        __syncthreads();
        int first = 0x7fffffff;
        for (int w8 = 0; w8 < kAccThreads / 32; ++w8) first = min(first, s_first[w8]);
        if (first != 0x7fffffff && tid == first) {
            // this thread's tokens alone, in order, from the running sum before them
            const int t0 = c * kAccChunk + tid * kAccPerThread;
            double run = s_prefix + incl, back = 0.0;
            double wt[kAccPerThread];
#pragma unroll
            for (int e = 0; e < kAccPerThread; ++e) {
                wt[e] = t0 + e < p.V ? draw_weight(trow, drow, t0 + e, ri, target_only) : 0.0;
                back += wt[e];
            }
            run -= back;
            int mine = -1;
#pragma unroll
            for (int e = 0; e < kAccPerThread; ++e) {
                run += wt[e];
                if (mine < 0 && run > s_target) mine = t0 + e;
            }
            // rounding may leave the crossing just past the group's end: then its last positive weight
            if (mine < 0) {
#pragma unroll
                for (int e = 0; e < kAccPerThread; ++e) if (wt[e] > 0.0) mine = t0 + e;
            }
            s_tok = mine < 0 ? 0x7fffffff : mine;
        }
        __syncthreads();
        if (s_tok != 0x7fffffff) tok = s_tok;
    } else if (s_chunk >= 0) {
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

__global__ void __launch_bounds__(kAccThreads) accept_pick_kernel(const AcceptParams p) {
    extern __shared__ double ws[];   // [n_chunks] chunk weights
    pdl_wait();
    pdl_trigger();
    pick_item(p, blockIdx.x, ws);
}

// ---- the same three steps in one launch ----------------------------------------------------------------------------
// A grid of at most one wave of CTAs walks the items of each step; between the steps all CTAs meet at a counter in the
// workspace header (zeroed before the launch).  The wait at the counter is bounded: after 2 s a CTA records
// HIPPO_ERR_TIMEOUT in the header and leaves, and so does every CTA that sees the status word set.
constexpr unsigned long long kAccWaitLimitNs = 2000000000ull;

__device__ bool accept_grid_barrier(WsHeader *hdr, int which) {
    __shared__ int s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        int *counter = &hdr->pad[which];
        __threadfence();
        atomicAdd(counter, 1);
        bool ok = true;
        unsigned long long t0 = 0;
        for (;;) {
            int seen;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= (int)gridDim.x) break;
            if (*reinterpret_cast<volatile int *>(&hdr->status) != 0) { ok = false; break; }
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            if (now - t0 > kAccWaitLimitNs) {
                if (atomicCAS(&hdr->status, 0, (int)HIPPO_ERR_TIMEOUT) == 0) hdr->where = 200 + which;
                ok = false;
                break;
            }
            __nanosleep(64);
        }
        s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    return s_ok != 0;
}

__global__ void __launch_bounds__(kAccThreads) accept_fused_kernel(const AcceptParams p, WsHeader *hdr) {
    extern __shared__ double ws[];   // [n_chunks] chunk weights
    pdl_wait();
    pdl_trigger();
    const int rows = 2 * p.gamma + 1;
    for (int i = blockIdx.x; i < p.B * rows * p.n_chunks; i += gridDim.x)
        stats_item(p, i / (rows * p.n_chunks), (i / p.n_chunks) % rows, i % p.n_chunks);
    if (!accept_grid_barrier(hdr, 0)) return;
    for (int i = blockIdx.x; i < p.B * p.n_chunks; i += gridDim.x) weigh_item(p, i / p.n_chunks, i % p.n_chunks);
    if (!accept_grid_barrier(hdr, 1)) return;
    for (int b = blockIdx.x; b < p.B; b += gridDim.x) pick_item(p, b, ws);
}

struct AcceptWs { size_t stats_off, wsum_off, info_off, tscan_off, total; int n_chunks; };
static AcceptWs accept_ws(int B, int gamma, int V) {
    AcceptWs w;
    w.n_chunks = ceil_div(V, kAccChunk);
    w.stats_off = kWsHeaderBytes;
    w.wsum_off = w.stats_off + align_up((size_t)B * (2 * gamma + 1) * w.n_chunks * sizeof(double2), 256);
    w.info_off = w.wsum_off + align_up((size_t)B * w.n_chunks * sizeof(double), 256);
    w.tscan_off = w.info_off + align_up((size_t)B * sizeof(RowInfo), 256);
    w.total = w.tscan_off + align_up((size_t)B * w.n_chunks * kAccThreads * sizeof(double), 256);
    return w;
}

// ---- greedy verification (the decoding mode of the paper's experiments): keep draft tokens while they equal the
// arg-max of the target row, then emit the target's arg-max (lowest token id on ties).
//   argmax  per (sequence, target row, chunk): maximum and its first position -> stats[b][row][chunk] = (max, index)
//   greedy  per sequence: merge the chunks of every row, compare with the draft tokens, write the outputs
__global__ void __launch_bounds__(kAccThreads) accept_argmax_kernel(const AcceptParams p) {
    __shared__ float smax[kAccThreads / 32];
    __shared__ int sidx[kAccThreads / 32];
    pdl_wait();
    pdl_trigger();
    const int c = blockIdx.x, r = blockIdx.y, b = blockIdx.z, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *row = logit_row(p, b, r);
    float m = -INFINITY;
    int mi = 0x7fffffff;
#pragma unroll
    for (int e = 0; e < kAccPerThread; ++e) {
        const int t = c * kAccChunk + e * kAccThreads + tid;     // ascending in e: a strict '>' keeps the first maximum
        const float v = t < p.V ? row[t] : -INFINITY;
        if (v > m || (v == m && t < mi && t < p.V)) { m = v; mi = t; }
    }
    for (int o = 16; o; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, o);
        const int oi = __shfl_xor_sync(0xffffffffu, mi, o);
        if (om > m || (om == m && oi < mi)) { m = om; mi = oi; }
    }
    if (lane == 0) { smax[warp] = m; sidx[warp] = mi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < kAccThreads / 32; ++w)
            if (smax[w] > m || (smax[w] == m && sidx[w] < mi)) { m = smax[w]; mi = sidx[w]; }
        p.stats[((size_t)b * (2 * p.gamma + 1) + r) * p.n_chunks + c] = make_double2((double)m, (double)mi);
    }
}

__global__ void __launch_bounds__(kAccThreads) accept_greedy_kernel(const AcceptParams p) {
    __shared__ int best[kAccMaxRows];
    pdl_wait();
    pdl_trigger();
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_rows = 2 * p.gamma + 1;
    for (int r = warp; r <= p.gamma; r += kAccThreads / 32) {
        const double2 *st = p.stats + ((size_t)b * n_rows + r) * p.n_chunks;
        double m = -INFINITY, mi = 2147483647.0;
        for (int c = lane; c < p.n_chunks; c += 32)
            if (st[c].x > m || (st[c].x == m && st[c].y < mi)) { m = st[c].x; mi = st[c].y; }
        for (int o = 16; o; o >>= 1) {
            const double om = __shfl_xor_sync(0xffffffffu, m, o), oi = __shfl_xor_sync(0xffffffffu, mi, o);
            if (om > m || (om == m && oi < mi)) { m = om; mi = oi; }
        }
        if (lane == 0) best[r] = (int)mi;
    }
    __syncthreads();
    if (tid == 0) {
        const int32_t *x = p.x + (size_t)b * p.gamma;
        int32_t *out = p.out + (size_t)b * (p.gamma + 1);
        int n = 0;
        while (n < p.gamma && x[n] == best[n]) { out[n] = x[n]; ++n; }
        out[n] = best[n];
        for (int j = n + 1; j <= p.gamma; ++j) out[j] = -1;
        p.n_acc[b] = n;
    }
}

static int32_t launch_accept_greedy(const AcceptParams &p, cudaStream_t s) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kAccThreads);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)p.n_chunks, (unsigned)(p.gamma + 1), (unsigned)p.B);
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_argmax_kernel, p));
    cfg.gridDim = dim3((unsigned)p.B);
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_greedy_kernel, p));
    count_launches(2);
    return HIPPO_OK;
}

// The three kernels, launched with programmatic stream serialization (each one waits before it reads).
static int32_t launch_accept_chain(const AcceptParams &p, cudaStream_t s) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kAccThreads);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)p.n_chunks, (unsigned)(2 * p.gamma + 1), (unsigned)p.B);
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_stats_kernel, p));
    cfg.gridDim = dim3((unsigned)p.n_chunks, (unsigned)p.B);
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_weigh_kernel, p));
    cfg.gridDim = dim3((unsigned)p.B);
    cfg.dynamicSmemBytes = (size_t)p.n_chunks * sizeof(double);
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_pick_kernel, p));
    count_launches(3);
    return HIPPO_OK;
}

// One launch: the grid is at most what the device keeps resident at once (the CTAs wait for one another between the
// steps), and never more than the first step has items.
static int32_t launch_accept_fused(const AcceptParams &p, WsHeader *hdr, cudaStream_t s) {
    const size_t smem = (size_t)p.n_chunks * sizeof(double);
    if (smem > 40 * 1024) return launch_accept_chain(p, s);
    static std::atomic<int> resident[kMaxDevices];
    int dev = -1;
    HIPPO_CUDA_TRY(cudaGetDevice(&dev));
    int cap = (dev >= 0 && dev < kMaxDevices) ? resident[dev].load(std::memory_order_relaxed) : 0;
    if (cap == 0) {
        int per_sm = 0, sms = 0;
        HIPPO_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, accept_fused_kernel, kAccThreads, 40 * 1024));
        HIPPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        cap = per_sm * sms;
        if (cap < 1) return launch_accept_chain(p, s);
        if (dev >= 0 && dev < kMaxDevices) resident[dev].store(cap, std::memory_order_relaxed);
    }
    long long grid = (long long)p.B * (2 * p.gamma + 1) * p.n_chunks;
    if (grid > cap) grid = cap;
    HIPPO_CUDA_TRY(cudaMemsetAsync(hdr, 0, sizeof(WsHeader), s));    // status word and the two arrival counters
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kAccThreads);
    cfg.gridDim = dim3((unsigned)grid);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_fused_kernel, p, hdr));
    count_launches(1);
    return HIPPO_OK;
}

// variant: 0 the faster of the two for the shape, else HIPPO_ACCEPT_ONE_LAUNCH / HIPPO_ACCEPT_THREE_LAUNCHES
static int32_t launch_accept(const AcceptParams &p, WsHeader *hdr, int variant, cudaStream_t s) {
    const bool fused = variant == HIPPO_ACCEPT_ONE_LAUNCH || (variant == 0 && kAcceptFusedByDefault);
    return fused ? launch_accept_fused(p, hdr, s) : launch_accept_chain(p, s);
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
    const int variant = mode & (HIPPO_ACCEPT_ONE_LAUNCH | HIPPO_ACCEPT_THREE_LAUNCHES);
    mode &= ~(HIPPO_ACCEPT_ONE_LAUNCH | HIPPO_ACCEPT_THREE_LAUNCHES);
    if ((mode != HIPPO_ACCEPT_SAMPLE && mode != HIPPO_ACCEPT_GREEDY) || variant == (HIPPO_ACCEPT_ONE_LAUNCH | HIPPO_ACCEPT_THREE_LAUNCHES))
        return fail(HIPPO_ERR_UNIMPLEMENTED, "hippo_accept: mode %d", mode | variant);
    const bool greedy = mode == HIPPO_ACCEPT_GREEDY;
    if (!target_logits || !n_accepted || !out_tokens || !workspace || (!greedy && !u_resample))
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept: null pointer");
    if (gamma > 0 && (!draft_tokens || (!greedy && (!draft_logits || !u_accept))))
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
    p.tscan = (double *)((char *)workspace + w.tscan_off);
    p.B = batch; p.gamma = gamma; p.V = vocab; p.n_chunks = w.n_chunks;
    cudaStream_t s = (cudaStream_t)stream;
    return greedy ? launch_accept_greedy(p, s) : launch_accept(p, (WsHeader *)workspace, variant, s);
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
    const int variant = mode & (HIPPO_ACCEPT_ONE_LAUNCH | HIPPO_ACCEPT_THREE_LAUNCHES);
    mode &= ~(HIPPO_ACCEPT_ONE_LAUNCH | HIPPO_ACCEPT_THREE_LAUNCHES);
    if ((mode != HIPPO_ACCEPT_SAMPLE && mode != HIPPO_ACCEPT_GREEDY) || variant == (HIPPO_ACCEPT_ONE_LAUNCH | HIPPO_ACCEPT_THREE_LAUNCHES))
        return fail(HIPPO_ERR_UNIMPLEMENTED, "hippo_accept_noalloc: mode %d", mode | variant);
    const bool greedy = mode == HIPPO_ACCEPT_GREEDY;
    if (!target_logits || !n_accepted || !out_tokens || (!greedy && !u_resample))
        return fail(HIPPO_ERR_INVALID_ARG, "hippo_accept_noalloc: null pointer");
    if (gamma > 0 && (!draft_tokens || (!greedy && (!draft_logits || !u_accept))))
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
    p.tscan = (double *)((char *)scratch + w.tscan_off);
    p.B = batch; p.gamma = gamma; p.V = vocab; p.n_chunks = w.n_chunks;
    cudaStream_t s = (cudaStream_t)stream;
    return greedy ? launch_accept_greedy(p, s) : launch_accept(p, (WsHeader *)scratch, variant, s);
}
