// CUDA-core split-KV attention (fp32 arithmetic, fp32 or bf16 storage) and the split combine.
//
// Computes softmax(scale * q K^T) V with grouped-query attention and a bottom-right-aligned causal tail
// (Section 3.2: the drafting and verification forward passes attend over the KV cache).  This is the path for
// fp32 caches (the tiny configuration, 1e-5 tolerance) and for shapes the tensor-core kernel does not cover.
//
// Grid (split, kv_head, batch); 4 warps.  A CTA streams 32-key tiles of its split through shared memory; every
// warp owns the packed rows r = warp, warp+4, ... (row r = t*G + g: query token t, head g of the group), keeps
// their running max / sum / output in shared memory and updates them tile by tile (online softmax).
#include <math.h>

#include "common.cuh"

namespace hippo {

constexpr int kGenThreads = 128;
constexpr int kGenWarps = kGenThreads / 32;
constexpr int kGenTile = 32;

template <typename T>
__global__ void __launch_bounds__(kGenThreads) attn_generic_kernel(const AttnParams p) {
    extern __shared__ float smem[];
    const int D = p.head_dim, R = p.rows, G = p.group;
    float *Qs = smem;                       // [R][D]
    float *Os = Qs + (size_t)R * D;         // [R][D]
    float *Ks = Os + (size_t)R * D;         // [32][D+1]
    float *Vs = Ks + kGenTile * (D + 1);    // [32][D]
    float *ms = Vs + kGenTile * D;          // [R]
    float *ls = ms + R;                     // [R]

    const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kvl = p.kv_len ? p.kv_len[b] : p.max_kv_len;
    float *slot = p.partials + ((size_t)(b * p.n_kv_heads + hk) * p.num_splits + split) * slot_float_count(R, D);
    const int Rp = slot_rows_padded(R);
    if (kvl < p.q_len) return;  // combine writes zeros for such sequences

    const T *q = (const T *)p.q;
    for (int i = tid; i < R * D; i += kGenThreads) {
        int r = i / D, d = i % D, t = r / G, g = r % G;
        Qs[i] = to_float(q[(((size_t)b * p.q_len + t) * p.n_q_heads + hk * G + g) * D + d]);
        Os[i] = 0.f;
    }
    for (int r = tid; r < R; r += kGenThreads) { ms[r] = -INFINITY; ls[r] = 0.f; }

    const int n_tiles = (kvl + kGenTile - 1) / kGenTile;
    const int per = (n_tiles + p.num_splits - 1) / p.num_splits;
    const int t0 = split * per, t1 = min(n_tiles, t0 + per);
    const T *kp = (const T *)p.k_pages, *vp = (const T *)p.v_pages;

    for (int tile = t0; tile < t1; ++tile) {
        __syncthreads();
        const int tok0 = tile * kGenTile;
        const int pid = page_of(p.page_table, p.max_pages_per_seq, b, tok0 / kPageSize);
        const size_t base = (((size_t)pid * p.n_kv_heads + hk) * kPageSize + (tok0 % kPageSize)) * D;
        for (int i = tid; i < kGenTile * D; i += kGenThreads) {
            int j = i / D, d = i % D;
            bool ok = tok0 + j < kvl;
            Ks[j * (D + 1) + d] = ok ? to_float(kp[base + i]) : 0.f;
            Vs[j * D + d] = ok ? to_float(vp[base + i]) : 0.f;
        }
        __syncthreads();
        for (int r = warp; r < R; r += kGenWarps) {
            const int t = r / G;
            const int limit = kvl - p.q_len + t;  // last visible key of this row
            const int key = tok0 + lane;
            float s = -INFINITY;
            if (key <= limit) {
                float acc = 0.f;
                const float *qr = Qs + (size_t)r * D, *kr = Ks + lane * (D + 1);
                for (int d = 0; d < D; ++d) acc = fmaf(qr[d], kr[d], acc);
                s = acc * p.scale;
            }
            float tmax = s;
            for (int o = 16; o; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
            const float m_old = ms[r];
            const float m_new = fmaxf(m_old, tmax);
            if (m_new == -INFINITY) continue;  // nothing visible yet (uniform across the warp)
            const float pj = (s == -INFINITY) ? 0.f : expf(s - m_new);
            const float corr = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
            float psum = pj;
            for (int o = 16; o; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
            for (int d = lane; d < D; d += 32) {
                float acc = Os[(size_t)r * D + d] * corr;
                for (int j = 0; j < kGenTile; ++j) acc = fmaf(__shfl_sync(0xffffffffu, pj, j), Vs[j * D + d], acc);
                Os[(size_t)r * D + d] = acc;
            }
            __syncwarp();
            if (lane == 0) { ms[r] = m_new; ls[r] = ls[r] * corr + psum; }
            __syncwarp();
        }
    }
    __syncthreads();
    for (int r = tid; r < R; r += kGenThreads) { slot[r] = ms[r]; slot[Rp + r] = ls[r]; }
    for (int i = tid; i < R * D; i += kGenThreads) slot[2 * Rp + i] = Os[i];
}

// One warp per output row (b, t, h): merge the per-split (m, l, O) partials of its (b, kv head).
// Slots of one (b, kv head) are the n_splits consecutive slots starting at (b*H_kv + hk) * n_splits.
template <typename T>
__global__ void attn_combine_kernel(const AttnParams p, int n_splits) {
    const int D = p.head_dim, R = p.rows, G = p.group;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int total = p.batch * p.q_len * p.n_q_heads;
    if (row >= total) return;
    const int h = row % p.n_q_heads, t = (row / p.n_q_heads) % p.q_len, b = row / (p.n_q_heads * p.q_len);
    const int hk = h / G, r = t * G + (h % G);
    T *out = (T *)p.out + (size_t)row * D;
    if ((p.kv_len ? p.kv_len[b] : p.max_kv_len) < p.q_len) {
        for (int d = lane; d < D; d += 32) store_from_float(out + d, 0.f);
        if (p.lse && lane == 0) p.lse[row] = -INFINITY;
        return;
    }
    const size_t slot_floats = slot_float_count(R, D);
    const int Rp = slot_rows_padded(R);
    const float *base = p.partials + (size_t)(b * p.n_kv_heads + hk) * n_splits * slot_floats;
    float M = -INFINITY;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, base[s * slot_floats + r]);
    float L = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        float m = base[s * slot_floats + r];
        if (m != -INFINITY) L += base[s * slot_floats + Rp + r] * expf(m - M);
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    for (int d = lane; d < D; d += 32) {
        float acc = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            float m = base[s * slot_floats + r];
            if (m != -INFINITY) acc = fmaf(base[s * slot_floats + 2 * Rp + (size_t)r * D + d], expf(m - M), acc);
        }
        store_from_float(out + d, acc * inv);
    }
    if (p.lse && lane == 0) p.lse[row] = M + logf(L);
}

static size_t generic_smem_bytes(const AttnParams &p) {
    size_t f = 2 * (size_t)p.rows * p.head_dim + kGenTile * (p.head_dim + 1) + kGenTile * p.head_dim + 2 * (size_t)p.rows;
    return f * sizeof(float);
}

int32_t launch_attn_generic(const AttnParams &p, int dtype, cudaStream_t stream) {
    size_t smem = generic_smem_bytes(p);
    if (smem > 227 * 1024) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "attention: rows*head_dim too large for shared memory");
    dim3 grid(p.num_splits, p.n_kv_heads, p.batch);
    if (dtype == HIPPO_DTYPE_FP32) {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_generic_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attn_generic_kernel<float><<<grid, kGenThreads, smem, stream>>>(p);
    } else {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_generic_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attn_generic_kernel<__nv_bfloat16><<<grid, kGenThreads, smem, stream>>>(p);
    }
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return launch_attn_combine(p, dtype, p.num_splits, stream);
}

int32_t launch_attn_combine(const AttnParams &p, int dtype, int n_splits, cudaStream_t stream) {
    const int total = p.batch * p.q_len * p.n_q_heads;
    const int warps_per_block = 4;
    dim3 grid((total + warps_per_block - 1) / warps_per_block);
    if (dtype == HIPPO_DTYPE_FP32)
        attn_combine_kernel<float><<<grid, warps_per_block * 32, 0, stream>>>(p, n_splits);
    else
        attn_combine_kernel<__nv_bfloat16><<<grid, warps_per_block * 32, 0, stream>>>(p, n_splits);
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}

}  // namespace hippo
