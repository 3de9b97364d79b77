// Low-latency split-KV attention for few packed rows over a short cache: the draft model's decode step over the
// pruned KV (Section 3.2, drafting phase: one query token, R = G <= 16 packed rows, a few hundred to a few thousand
// keys).  Such a call moves well under a megabyte, so its cost is the length of the dependency chain, not bandwidth:
// this kernel has no tensor-memory or TMA pipeline to fill and needs one launch.
//
// One thread-block cluster per (sequence, kv head) unit.  The CTAs of a cluster split the unit's 64-key pages evenly.
// Per page, in a CTA of 128 threads:
//   scores   two threads per key, each holding half of the key's row in registers, dot it with the R query rows
//            (fp32, query pre-scaled by scale*log2e and kept in shared memory)
//   softmax  exact online update per page: row maxima by warp reduction, p = 2^(s - m) to shared memory
//   output   thread (key group, 8-column group) accumulates R x 8 outputs over its keys of the page
// The next page's K and V registers are loaded while the current page is computed.  At the end the key groups are
// summed (warp shuffles, then one pass through shared memory).  Row r of the unit is merged by CTA r mod cluster
// size: every CTA pushes its (m, l, O[r]) into that CTA's shared memory with remote stores, and after one cluster
// barrier the owners merge what they received and write the output.
#include <math.h>

#include "common.cuh"

namespace hippo {

constexpr int kSmThreads = 128;
constexpr int kSmPage = kPageSize;     // keys per step
constexpr float kSmLog2e = 1.4426950408889634f;
constexpr float kSmLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint32_t sm_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void sm_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t sm_cluster_map(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void sm_st_cluster(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void sm_st_cluster_v4(uint32_t addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ float sm_warp_max(float x) {
    float y;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float sm_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void unpack8(const uint4 &u, float *f) {
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}

template <int D, int RMAX>
struct SmallShared {
    static constexpr int kHalf = D / 2;
    static constexpr int kQHalfStride = RMAX * kHalf + 4;      // +4 floats: the two halves fall in different banks
    static constexpr int kJG = kSmThreads / (D / 8);           // key groups of the output phase
    float q[2 * kQHalfStride];                                 // [half][row][D/2], scaled by scale*log2e
    float p[kSmPage][RMAX];                                    // probabilities of the current page
    float wmax[4][RMAX];
    float m[2][RMAX];                                          // running maxima, double buffered by page parity
    float wsum[4][RMAX];
    int limit[RMAX];
    float red[4][RMAX][D];                                     // per-warp output partials
    // partials pushed by the cluster peers for the rows this CTA merges: entry = slot * cluster size + peer,
    // slot = r / cluster size; (slots x cluster size) <= max(RMAX, 16)
    float recv_ml[16][2];
    float recv_o[16][D];
};

template <int D, int RMAX>
__global__ void __launch_bounds__(kSmThreads) attn_small_kernel(const AttnParams p, const int cluster_size) {
    using S = SmallShared<D, RMAX>;
    constexpr int kHalf = D / 2, kKV4 = kHalf / 8;       // uint4 loads of a half row
    constexpr int kDG = D / 8, kJG = S::kJG, kKPT = kSmPage / kJG;   // keys per thread in the output phase
    __shared__ __align__(16) S sh;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = p.rows, G = p.group, Hkv = p.n_kv_heads;
    const int unit = blockIdx.x / cluster_size, rank = blockIdx.x % cluster_size;
    const int b = unit / Hkv, hk = unit % Hkv;
    const int kvl = p.kv_len ? p.kv_len[b] : p.max_kv_len;   // no length array: every sequence has max_kv_len keys
    const bool skipped = kvl < p.q_len;
    const int n_pages = skipped ? 0 : (kvl + kSmPage - 1) / kSmPage;
    const int pg_begin = (int)((long long)n_pages * rank / cluster_size), pg_end = (int)((long long)n_pages * (rank + 1) / cluster_size);
    const float sl2 = p.scale * kSmLog2e;

    // ---- query rows (scaled) and per-row visibility limits
    for (int x = tid; x < RMAX * (D / 8); x += kSmThreads) {
        const int r = x / (D / 8), c8 = x % (D / 8);
        float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (r < R) {
            const int t = r / G, g = r % G;
            unpack8(__ldg(reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)p.q + (((size_t)b * p.q_len + t) * p.n_q_heads + hk * G + g) * D) + c8), v);
        }
        float *dstq = sh.q + ((c8 * 8) / kHalf) * S::kQHalfStride + r * kHalf + (c8 * 8) % kHalf;
        *reinterpret_cast<float4 *>(dstq) = make_float4(v[0] * sl2, v[1] * sl2, v[2] * sl2, v[3] * sl2);
        *reinterpret_cast<float4 *>(dstq + 4) = make_float4(v[4] * sl2, v[5] * sl2, v[6] * sl2, v[7] * sl2);
    }
    if (tid < RMAX) {
        sh.limit[tid] = tid < R ? kvl - p.q_len + tid / G : 0x7fffffff;
        sh.m[0][tid] = -INFINITY;
        sh.m[1][tid] = -INFINITY;
    }
    __syncthreads();

    const int key_j = tid >> 1, half = tid & 1;          // score phase: key of the page, half of the row
    const int jg = tid / kDG, dg = tid % kDG;            // output phase: key group, 8-column group
    const __nv_bfloat16 *kp = (const __nv_bfloat16 *)p.k_pages, *vp = (const __nv_bfloat16 *)p.v_pages;

    float acc[RMAX][8], lpart[RMAX];
#pragma unroll
    for (int r = 0; r < RMAX; ++r) {
        lpart[r] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[r][e] = 0.f;
    }
    uint4 kreg[kKV4], vreg[kKPT], knext[kKV4], vnext[kKPT];
    auto load_page = [&](int pg, uint4 *kr, uint4 *vr) {
        const int pid = page_of(p.page_table, p.max_pages_per_seq, b, pg);
        const size_t base = ((size_t)pid * Hkv + hk) * kSmPage * D;
        const int key0 = pg * kSmPage;
#pragma unroll
        for (int i = 0; i < kKV4; ++i)
            kr[i] = key0 + key_j < kvl ? __ldg(reinterpret_cast<const uint4 *>(kp + base + (size_t)key_j * D + half * kHalf) + i) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < kKPT; ++i) {
            const int j = jg * kKPT + i;
            vr[i] = key0 + j < kvl ? __ldg(reinterpret_cast<const uint4 *>(vp + base + (size_t)j * D + dg * 8)) : make_uint4(0, 0, 0, 0);
        }
    };
    if (pg_begin < pg_end) load_page(pg_begin, kreg, vreg);

    for (int pg = pg_begin; pg < pg_end; ++pg) {
        const int par = (pg - pg_begin) & 1;
        if (pg + 1 < pg_end) load_page(pg + 1, knext, vnext);
        // ---- scores of this thread's key against the R rows (half a row per thread, then the pair adds up)
        float s[RMAX];
#pragma unroll
        for (int r = 0; r < RMAX; ++r) s[r] = 0.f;
        const float *qh = sh.q + half * S::kQHalfStride;
#pragma unroll
        for (int i = 0; i < kKV4; ++i) {
            float kf[8];
            unpack8(kreg[i], kf);
#pragma unroll
            for (int r = 0; r < RMAX; ++r) {
                const float4 q0 = *reinterpret_cast<const float4 *>(qh + r * kHalf + i * 8);
                const float4 q1 = *reinterpret_cast<const float4 *>(qh + r * kHalf + i * 8 + 4);
                s[r] = fmaf(kf[0], q0.x, fmaf(kf[1], q0.y, fmaf(kf[2], q0.z, fmaf(kf[3], q0.w, s[r]))));
                s[r] = fmaf(kf[4], q1.x, fmaf(kf[5], q1.y, fmaf(kf[6], q1.z, fmaf(kf[7], q1.w, s[r]))));
            }
        }
        const int key = pg * kSmPage + key_j;
#pragma unroll
        for (int r = 0; r < RMAX; ++r) {
            s[r] += __shfl_xor_sync(0xffffffffu, s[r], 1);
            s[r] = key <= sh.limit[r] && key < kvl ? s[r] : -INFINITY;
            const float wm = sm_warp_max(s[r]);
            if (lane == r) sh.wmax[warp][r] = wm;
        }
        __syncthreads();
        // ---- new maxima, probabilities, rescale of what has been accumulated
#pragma unroll
        for (int r = 0; r < RMAX; ++r) {
            const float m_old = sh.m[par][r];
            const float m_new = fmaxf(fmaxf(m_old, fmaxf(sh.wmax[0][r], sh.wmax[1][r])), fmaxf(sh.wmax[2][r], sh.wmax[3][r]));
            const float f = (m_old == -INFINITY) ? 0.f : sm_ex2(m_old - m_new);     // m_new = -inf implies m_old = -inf
            const float pr = (s[r] == -INFINITY) ? 0.f : sm_ex2(s[r] - m_new);
            lpart[r] = lpart[r] * f + (half == 0 ? pr : 0.f);
            if (half == 0) sh.p[key_j][r] = pr;
            if (tid == r) sh.m[par ^ 1][r] = m_new;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[r][e] *= f;
        }
        __syncthreads();
        // ---- output: this thread's keys of the page, 8 columns, all rows
#pragma unroll
        for (int i = 0; i < kKPT; ++i) {
            const int j = jg * kKPT + i;
            float vf[8];
            unpack8(vreg[i], vf);
#pragma unroll
            for (int r4 = 0; r4 < RMAX; r4 += 4) {
                const float4 pr = *reinterpret_cast<const float4 *>(&sh.p[j][r4]);
                const float pw[4] = {pr.x, pr.y, pr.z, pr.w};
#pragma unroll
                for (int x = 0; x < 4; ++x)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[r4 + x][e] = fmaf(pw[x], vf[e], acc[r4 + x][e]);
            }
        }
        if (pg + 1 < pg_end) {
#pragma unroll
            for (int i = 0; i < kKV4; ++i) kreg[i] = knext[i];
#pragma unroll
            for (int i = 0; i < kKPT; ++i) vreg[i] = vnext[i];
        }
        // the next page's barrier after the scores separates these reads of p and wmax from their next writes
    }
    const int par_end = (pg_end - pg_begin) & 1;
    __syncthreads();
    // ---- the CTA's partial: sums over the threads (l) and over the key groups (O)
#pragma unroll
    for (int r = 0; r < RMAX; ++r) {
        float v = lpart[r];
#pragma unroll
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == r) sh.wsum[warp][r] = v;
    }
    // key groups inside a warp (lane = key group * kDG + column group), then the four warps through shared memory
#pragma unroll
    for (int r = 0; r < RMAX; ++r)
#pragma unroll
        for (int e = 0; e < 8; ++e)
#pragma unroll
            for (int o = kDG; o < 32; o <<= 1) acc[r][e] += __shfl_xor_sync(0xffffffffu, acc[r][e], o);
    if (lane < kDG) {
#pragma unroll
        for (int r = 0; r < RMAX; ++r) {
            *reinterpret_cast<float4 *>(&sh.red[warp][r][lane * 8]) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            *reinterpret_cast<float4 *>(&sh.red[warp][r][lane * 8 + 4]) = make_float4(acc[r][4], acc[r][5], acc[r][6], acc[r][7]);
        }
    }
    __syncthreads();
    // ---- push this CTA's partial of row r to the CTA that merges it
    {
        const uint32_t a_ml = sm_smem_u32(sh.recv_ml), a_o = sm_smem_u32(sh.recv_o);
        for (int x = tid; x < R * (D / 4); x += kSmThreads) {
            const int r = x / (D / 4), c4 = x % (D / 4);
            float4 v = *reinterpret_cast<const float4 *>(&sh.red[0][r][c4 * 4]);
#pragma unroll
            for (int w = 1; w < 4; ++w) {
                const float4 t = *reinterpret_cast<const float4 *>(&sh.red[w][r][c4 * 4]);
                v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
            }
            const int entry = (r / cluster_size) * cluster_size + rank;
            sm_st_cluster_v4(sm_cluster_map(a_o, (uint32_t)(r % cluster_size)) + 4 * (entry * D + c4 * 4), v);
        }
        if (tid < R) {
            const int r = tid, entry = (r / cluster_size) * cluster_size + rank;
            const uint32_t dst = sm_cluster_map(a_ml, (uint32_t)(r % cluster_size)) + 8 * entry;
            sm_st_cluster(dst, sh.m[par_end][r]);
            sm_st_cluster(dst + 4, (sh.wsum[0][r] + sh.wsum[1][r]) + (sh.wsum[2][r] + sh.wsum[3][r]));
        }
    }
    sm_cluster_sync();   // release / acquire: the pushed partials are visible to their owners
    // ---- merge the rows r = rank, rank + cluster_size, ...: one warp per row, lanes over the columns
    {
        constexpr int V = D / 32;
        for (int r = rank + cluster_size * warp; r < R; r += cluster_size * (kSmThreads / 32)) {
            const size_t ro = ((size_t)b * p.q_len + r / G) * p.n_q_heads + hk * G + r % G;
            __nv_bfloat16 *o = (__nv_bfloat16 *)p.out + ro * D + lane * V;
            const int e0 = (r / cluster_size) * cluster_size;
            float M = -INFINITY, L = 0.f, av[V];
#pragma unroll
            for (int x = 0; x < V; ++x) av[x] = 0.f;
            if (!skipped) {
                for (int c = 0; c < cluster_size; ++c) M = fmaxf(M, sh.recv_ml[e0 + c][0]);
                for (int c = 0; c < cluster_size; ++c) {
                    const float m = sh.recv_ml[e0 + c][0];
                    if (m == -INFINITY) continue;
                    const float f = sm_ex2(m - M);
                    L = fmaf(sh.recv_ml[e0 + c][1], f, L);
#pragma unroll
                    for (int x = 0; x < V; ++x) av[x] = fmaf(sh.recv_o[e0 + c][lane * V + x], f, av[x]);
                }
            }
            const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
            for (int x = 0; x < V; x += 2) {
                __nv_bfloat162 h2 = __floats2bfloat162_rn(av[x] * inv, av[x + 1] * inv);
                *reinterpret_cast<__nv_bfloat162 *>(o + x) = h2;
            }
            if (p.lse && lane == 0) p.lse[ro] = L > 0.f ? (M + log2f(L)) * kSmLn2 : -INFINITY;
        }
    }
}

// Pages of 64 keys a CTA may walk before the tensor-core kernel is the better choice (measured: beyond one page per
// CTA, i.e. 1,024 keys with the largest cluster, the tensor-core kernel's deeper pipeline wins).
constexpr int kSmMaxPagesPerCta = 1;
constexpr int kSmMaxCluster = 16;

bool attn_small_supported(const AttnParams &p, int dtype) {
    if (dtype != HIPPO_DTYPE_BF16 || (p.head_dim != 64 && p.head_dim != 128) || p.rows > 8) return false;
    const int pages = ceil_div(p.max_kv_len, kSmPage);
    return ceil_div(pages, kSmMaxCluster) <= kSmMaxPagesPerCta && (long long)p.batch * p.n_kv_heads * kSmMaxCluster <= 65535;
}

template <int D, int RMAX>
static int32_t launch_small(const AttnParams &p, cudaStream_t stream) {
    static PerDeviceOnce attr_set;
    int dev;
    if (attr_set.needed(dev)) {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_small_kernel<D, RMAX>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        attr_set.mark(dev);
    }
    const int pages = ceil_div(p.max_kv_len, kSmPage);
    int cs = pages < kSmMaxCluster ? pages : kSmMaxCluster;
    if (cs < 1) cs = 1;
    const int units = p.batch * p.n_kv_heads;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kSmThreads);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    for (;;) {
        attr[1].val.clusterDim.x = (unsigned)cs;
        cfg.gridDim = dim3((unsigned)(units * cs));
        const cudaError_t e = cudaLaunchKernelEx(&cfg, attn_small_kernel<D, RMAX>, p, cs);
        if (e == cudaSuccess) break;
        (void)cudaGetLastError();
        if (cs <= 8) return cuda_fail(e, "attention (small) launch");
        cs = 8;   // clusters beyond the portable size are not available here
        if (ceil_div(pages, cs) > 2 * kSmMaxPagesPerCta) return cuda_fail(e, "attention (small) launch");
    }
    count_launches(1);
    return HIPPO_OK;
}

int32_t launch_attn_small(const AttnParams &p, cudaStream_t stream) {
    if (p.head_dim == 64) return launch_small<64, 8>(p, stream);
    return launch_small<128, 8>(p, stream);
}

}  // namespace hippo
