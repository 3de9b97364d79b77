// hippo_select_tokens: semantic-aware visual-token preservation (Section 5.1).
//
//   Eq. 3-4  s_temp(j) = 1 - mean over the adjacent frames that contain j's grid cell of cos(v_j^f, v_j^f')
//   Eq. 5-6  s_spa(j)  = (1/M) sum_k (S_jk - mu_j)^2 over the M tokens of j's crop, S = cosine Gram matrix, S_jj = 1
//   Eq. 7    fused = z(attn) + z(spa) + z(temp), z = per-frame standardisation with the population sigma
//   top-k    k best over the sequence by (fused as fp32 descending, index ascending), emitted ascending
//
// The standardisation of s_spa divides by a sigma of ~1e-4 on near-orthogonal embeddings, which magnifies any
// rounding in the Gram entries by four orders of magnitude.  All dot products, crop statistics and frame
// statistics are therefore accumulated in fp64 (bf16 x bf16 products are exact in fp64), so the kept set only
// depends on the final rounding of the fused score to fp32.
//
// Kernels:  dots (norms + next-frame dot, one warp per token)  ->  spatial (one CTA per crop, fp64 tensor instructions)  ->
//           fuse (one CTA per frame: s_temp, three standardisations, sum)  ->  topk (one CTA per sequence,
//           bisection on order-preserving keys, ordered compaction).
//
// hippo_select_tokens_policy adds the selection rules the paper compares itself with, as rules only: a uniform budget
// per frame (the attention-guided uniform pruning of earlier video speculative decoding, related-work section), the k
// best by caller-supplied random keys and whole frames at a regular stride (exploration of pruning criteria,
// Section 6).  Uniform: budgets by one thread per sequence, then one CTA per frame ranks its tokens by counting.
#include <math.h>

#include <type_traits>

#include "common.cuh"

namespace hippo {

constexpr int kMaxCrop = 32;       // tokens per crop
constexpr int kSelMaxBatch = 64;   // sequences per call (kernel-parameter tables)

struct SelectParams {
    const void *embeds;
    const float *attn_mass;
    float *fused;
    int32_t *kept;
    double *norm2, *tdot, *s_spa;   // [total tokens]
    int batch, grid_h, grid_w, crop_h, crop_w, d, tpf, crops_y, crops_x;
    unsigned mask;
    int seq_off[kSelMaxBatch + 1];    // token offset of each sequence
    int frame_off[kSelMaxBatch + 1];  // frame offset of each sequence
    int k[kSelMaxBatch];
    int k_off[kSelMaxBatch + 1];
    int *frame_budget;               // per-frame policy: [frames] tokens kept / [frames] first output position
    int *frame_out;
};

__device__ __forceinline__ double ld_as_double(const float *p, size_t i) { return (double)p[i]; }
__device__ __forceinline__ double ld_as_double(const __nv_bfloat16 *p, size_t i) { return (double)__bfloat162float(p[i]); }

__device__ __forceinline__ double warp_sum(double v) {
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block, result valid in every thread.  Fixed reduction order.
__device__ double block_sum(double v, double *scratch /* [32] shared */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < nw; ++w) t += scratch[w];
    return t;
}

__device__ __forceinline__ int find_seq(const int *off, int n, int x) {  // largest b with off[b] <= x
    int b = 0;
    while (b + 1 < n && off[b + 1] <= x) ++b;
    return b;
}

// ---- norms and the dot product with the same cell of the next frame ------------------------------------------
template <typename T> __device__ __forceinline__ void load8(const T *p, double *v);
template <> __device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16 *p, double *v) {
    const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 f = __bfloat1622float2(h[i]); v[2 * i] = (double)f.x; v[2 * i + 1] = (double)f.y; }
}
template <> __device__ __forceinline__ void load8<float>(const float *p, double *v) {
    const float4 a = __ldg(reinterpret_cast<const float4 *>(p)), c = __ldg(reinterpret_cast<const float4 *>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = c.x; v[5] = c.y; v[6] = c.z; v[7] = c.w;
}

// One warp per token; a lane takes 8 consecutive elements per step (embed_dim is a multiple of 8).
template <typename T>
__global__ void __launch_bounds__(256) select_dots_kernel(const SelectParams p) {
    const int total = p.seq_off[p.batch];
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (j >= total) return;
    const int b = find_seq(p.seq_off, p.batch, j);
    const T *E = (const T *)p.embeds;
    const size_t a = (size_t)j * p.d;
    const bool has_next = j + p.tpf < p.seq_off[b + 1];
    const size_t c = a + (size_t)p.tpf * p.d;
    double n2 = 0.0, td = 0.0;
    for (int i = lane * 8; i < p.d; i += 256) {
        double x[8], y[8];
        load8(E + a + i, x);
        if (has_next) load8(E + c + i, y);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            n2 = fma(x[e], x[e], n2);
            if (has_next) td = fma(x[e], y[e], td);
        }
    }
    n2 = warp_sum(n2);
    td = warp_sum(td);
    if (lane == 0) { p.norm2[j] = n2; p.tdot[j] = td; }
}

// ---- spatial score on the fp64 tensor path: one CTA per crop ---------------------------------------------------------
// The Gram matrix of the crop's embeddings is a dense fp64 contraction over the embedding dimension: it runs on
// mma.sync.m8n8k4.f64 (exact fp64 products of the widened inputs, fp64 accumulation; measured on B200: one instruction per
// 16.1 clocks and SM quarter, i.e. 63.6 multiply-adds per clock and SM, whatever the operand values and also with the
// operands read from shared memory and widened on the way).  Tokens are taken in groups of eight; for the groups a <= c the
// 8 x 8 tile G[a][c] needs one fragment per group and step of four dimensions, and for a Gram matrix the A fragment of a
// group (row = lane / 4, dimension = lane % 4) is also its B fragment.  Warp w owns dimensions [16 w, 16 w + 16) of every
// 128-dimension chunk: it stages them itself, in the storage type, straight from global memory with cp.async into a ring
// of its own (rows back to back, so the eight rows of a fragment load are contiguous), and waits for nobody else's
// copies: there is no block-wide barrier inside the loop.  Since the order of a dot product's terms is free, lane l takes
// dimensions 4 (l % 4) .. + 3 of the warp's sixteen: one 8-byte (bf16) load per group and chunk, widened to fp64 in
// registers, feeds the four steps.  Every staged element is read exactly once.  The eight warps' tiles are added in shared
// memory at the end, in a fixed order; the diagonal of G holds the squared norms.
// The multiply sequence is instantiated per number of groups: with the group count a run-time value every instruction of
// it sat behind a branch of its own and the pipe was busy half of the time (32k tokens, whole selection: 472 us with the
// branches, 351 us without, 343 us with the warps' own rings).
// A crop of 8 n + 1 tokens (the paper's 5 x 5 = 25) would pay n + 1 tiles for its last token: that token's dot products
// come from plain multiply-adds on the fragments the lane holds anyway (see below).
constexpr int kMmaChunk = 128;                 // dimensions per chunk, over the eight warps
constexpr int kMmaWarpDims = 16;               // dimensions of a chunk that one warp stages and multiplies
constexpr int kMmaThreads = 256;
constexpr int kMmaWarps = kMmaThreads / 32;
constexpr int kMmaTiles = 10;                  // 4 groups: upper triangle incl. diagonal
static_assert(kMmaWarps * kMmaWarpDims == kMmaChunk, "the warps' slices make up a chunk");
template <typename T> struct MmaShape {
    static constexpr int kPiece = 16 / (int)sizeof(T);               // elements per 16-byte piece
    static constexpr int kPiecesPerRow = kMmaWarpDims / kPiece;
    static constexpr int kWarpRowBytes = kMmaWarpDims * (int)sizeof(T);   // rows back to back: the eight rows of a fragment load are contiguous
    static constexpr int kWarpStageBytes = kMaxCrop * kWarpRowBytes;
    static constexpr int kStages = 12 / (int)sizeof(T);              // 6 chunks in flight per warp (bf16), 3 (fp32): 6 KB per warp
    static constexpr size_t kWarpRingBytes = (size_t)kStages * kWarpStageBytes;
    static constexpr size_t kRingBytes = (size_t)kMmaWarps * kWarpRingBytes;
    static constexpr size_t kRedBytes = (size_t)kMmaWarps * kMmaTiles * 64 * sizeof(double);
    static constexpr size_t kSmemBytes = kRingBytes > kRedBytes ? kRingBytes : kRedBytes;
};

__device__ __forceinline__ void dmma_m8n8k4(double &c0, double &c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}
// 16 bytes global -> shared, asynchronously; n_bytes = 0 writes zeros and reads nothing
__device__ __forceinline__ void cp_async_16(void *dst, const void *src, int n_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src), "r"(n_bytes) : "memory");
}
__device__ __forceinline__ void load_frag4(const __nv_bfloat16 *p, double *v) {
    const uint2 u = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    v[0] = (double)a.x; v[1] = (double)a.y; v[2] = (double)b.x; v[3] = (double)b.y;
}
__device__ __forceinline__ void load_frag4(const float *p, double *v) {
    const float4 a = *reinterpret_cast<const float4 *>(p);
    v[0] = (double)a.x; v[1] = (double)a.y; v[2] = (double)a.z; v[3] = (double)a.w;
}

template <typename T>
__global__ void __launch_bounds__(kMmaThreads, 3) select_spatial_mma_kernel(const SelectParams p) {
    using Sh = MmaShape<T>;
    extern __shared__ __align__(16) uint8_t mma_smem[];   // ring of staged chunks; reused for the warps' partial tiles
    __shared__ int tok[kMaxCrop];
    __shared__ double S[kMaxCrop][kMaxCrop + 1];
    __shared__ double nrm2[kMaxCrop];
    __shared__ double tail_red[kMmaWarps][kMaxCrop + 1];
    __shared__ int s_M;
    const int crops_per_frame = p.crops_y * p.crops_x;
    const int gframe = blockIdx.x / crops_per_frame, cr = blockIdx.x % crops_per_frame;
    const int b = find_seq(p.frame_off, p.batch, gframe);
    const int f = gframe - p.frame_off[b];
    const int n_v = p.seq_off[b + 1] - p.seq_off[b];
    const int nf = min(p.tpf, n_v - f * p.tpf);
    const int y0 = (cr / p.crops_x) * p.crop_h, x0 = (cr % p.crops_x) * p.crop_w;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        int M = 0;
        for (int y = y0; y < y0 + p.crop_h && y < p.grid_h; ++y)
            for (int x = x0; x < x0 + p.crop_w && x < p.grid_w; ++x)
                if (y * p.grid_w + x < nf) tok[M++] = p.seq_off[b] + f * p.tpf + y * p.grid_w + x;
        s_M = M;
    }
    __syncthreads();
    const int M = s_M;
    if (M == 0) return;
    const T *E = (const T *)p.embeds;
    if (M > 1) {
        // A crop of 8n + 1 tokens (the full 5 x 5 crop: 25) would pay a whole extra group, n + 1 tiles, for its last
        // token.  Its n * 8 dot products and its norm come from plain multiply-adds instead: at every step a lane already
        // holds, as tile operands, token (8g + lane / 4) at the step's dimension for each group g, so all it needs besides
        // is the last token's value at that dimension (one broadcast load per four steps), and the four lanes of a row
        // are added at the end.
        const bool tail = (M & 7) == 1 && M > 8;
        const int n_groups = tail ? M / 8 : (M + 7) / 8;     // groups that go through the tiles
        const int rows = tail ? M : 8 * n_groups;            // staged rows; rows >= M are zero
        const int n_chunks = (p.d + kMmaChunk - 1) / kMmaChunk;
        // Each warp stages its own 16 dimensions of every chunk into a ring of its own and waits only for its own
        // copies: no block-wide barrier inside the loop, so the warps drift apart and keep the fp64 pipe fed while
        // others load and widen.
        uint8_t *ring = mma_smem + (size_t)warp * Sh::kWarpRingBytes;
        // a lane copies the same pieces (row, 16-byte column) of every chunk: source pointers and ring offsets are set up once
        constexpr int kLanePieces = (kMaxCrop * Sh::kPiecesPerRow + 31) / 32;
        const T *src[kLanePieces];
        int dst_off[kLanePieces], col[kLanePieces];
#pragma unroll
        for (int i = 0; i < kLanePieces; ++i) {
            const int it = lane + 32 * i;
            const int r = it / Sh::kPiecesPerRow, c = it % Sh::kPiecesPerRow;
            col[i] = warp * kMmaWarpDims + c * Sh::kPiece;
            src[i] = r < M ? E + (size_t)tok[r] * p.d + col[i] : nullptr;     // rows M .. rows - 1 are zero-filled
            dst_off[i] = it < rows * Sh::kPiecesPerRow ? r * Sh::kWarpRowBytes + c * 16 : -1;
        }
        auto stage_chunk = [&](int ch) {
            uint8_t *dst = ring + (size_t)(ch % Sh::kStages) * Sh::kWarpStageBytes;
#pragma unroll
            for (int i = 0; i < kLanePieces; ++i) {
                if (dst_off[i] < 0) continue;
                const bool live = src[i] != nullptr && ch * kMmaChunk + col[i] < p.d;   // embed_dim is a multiple of 8: a piece is all there or not at all
                cp_async_16(dst + dst_off[i], live ? (const void *)(src[i] + (size_t)ch * kMmaChunk) : (const void *)E, live ? 16 : 0);
            }
        };
        double acc[kMmaTiles][2];
#pragma unroll
        for (int t = 0; t < kMmaTiles; ++t) acc[t][0] = acc[t][1] = 0.0;
        double tacc[4] = {0.0, 0.0, 0.0, 0.0};               // last token x groups 0..2, and its squared norm
        // the loop over the chunks, instantiated per (groups, tail) so that the multiply sequence is straight-line code
        auto gram_loop = [&](auto ng_tag, auto tail_tag) {
            constexpr int NG = decltype(ng_tag)::value;
            constexpr bool TAIL = decltype(tail_tag)::value;
            for (int s = 0; s < Sh::kStages - 1; ++s) {
                if (s < n_chunks) stage_chunk(s);
                asm volatile("cp.async.commit_group;" ::: "memory");
            }
            for (int ch = 0; ch < n_chunks; ++ch) {
                // this lane's copies of chunk ch have landed; after the warp barrier so have the other lanes', and every
                // lane is done reading the slot that the next copies overwrite
                asm volatile("cp.async.wait_group %0;" ::"n"(Sh::kStages - 2) : "memory");
                __syncwarp();
                if (ch + Sh::kStages - 1 < n_chunks) stage_chunk(ch + Sh::kStages - 1);
                asm volatile("cp.async.commit_group;" ::: "memory");
                const T *st = reinterpret_cast<const T *>(ring + (size_t)(ch % Sh::kStages) * Sh::kWarpStageBytes);
                double frag[NG][4], tv[4] = {0.0, 0.0, 0.0, 0.0};   // [group][step]
#pragma unroll
                for (int g = 0; g < NG; ++g) load_frag4(st + (g * 8 + (lane >> 2)) * kMmaWarpDims + (lane & 3) * 4, frag[g]);
                if (TAIL) load_frag4(st + (M - 1) * kMmaWarpDims + (lane & 3) * 4, tv);
#pragma unroll
                for (int step = 0; step < 4; ++step) {
#pragma unroll
                    for (int ga = 0; ga < NG; ++ga)
#pragma unroll
                        for (int gc = ga; gc < NG; ++gc) {
                            const int t = ga * 4 - ga * (ga - 1) / 2 + (gc - ga);   // constant after unrolling
                            dmma_m8n8k4(acc[t][0], acc[t][1], frag[ga][step], frag[gc][step]);
                        }
                    if (TAIL) {
#pragma unroll
                        for (int g = 0; g < NG; ++g) tacc[g] = __fma_rn(frag[g][step], tv[step], tacc[g]);
                        tacc[3] = __fma_rn(tv[step], tv[step], tacc[3]);
                    }
                }
            }
        };
        using std::integral_constant;
        switch (n_groups * 2 + (tail ? 1 : 0)) {
            case 2: gram_loop(integral_constant<int, 1>{}, integral_constant<bool, false>{}); break;
            case 3: gram_loop(integral_constant<int, 1>{}, integral_constant<bool, true>{}); break;
            case 4: gram_loop(integral_constant<int, 2>{}, integral_constant<bool, false>{}); break;
            case 5: gram_loop(integral_constant<int, 2>{}, integral_constant<bool, true>{}); break;
            case 6: gram_loop(integral_constant<int, 3>{}, integral_constant<bool, false>{}); break;
            case 7: gram_loop(integral_constant<int, 3>{}, integral_constant<bool, true>{}); break;
            default: gram_loop(integral_constant<int, 4>{}, integral_constant<bool, false>{}); break;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncthreads();
        // the eight warps' partial tiles meet in shared memory (the ring is idle now)
        double *red = reinterpret_cast<double *>(mma_smem);
        {
            double *mine = red + (size_t)warp * (kMmaTiles * 64);
            int t = 0;
#pragma unroll
            for (int ga = 0; ga < 4; ++ga)
#pragma unroll
                for (int gc = ga; gc < 4; ++gc, ++t)
                    if (gc < n_groups) {
                        mine[t * 64 + (lane >> 2) * 8 + (lane & 3) * 2] = acc[t][0];
                        mine[t * 64 + (lane >> 2) * 8 + (lane & 3) * 2 + 1] = acc[t][1];
                    }
        }
        if (tail) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                tacc[g] += __shfl_xor_sync(0xffffffffu, tacc[g], 1);
                tacc[g] += __shfl_xor_sync(0xffffffffu, tacc[g], 2);
            }
            if ((lane & 3) == 0) {
#pragma unroll
                for (int g = 0; g < 3; ++g)
                    if (g < n_groups) tail_red[warp][g * 8 + (lane >> 2)] = tacc[g];
                if (lane == 0) tail_red[warp][M - 1] = tacc[3];
            }
        }
        __syncthreads();
        // G[a][c] for a <= c, summed over the warps in a fixed order; then the cosines
        for (int x = tid; x < M * M; x += kMmaThreads) {
            const int a = x / M, c = x % M;
            if (a > c) continue;
            if (tail && c == M - 1) {
                double g = 0.0;
                for (int w = 0; w < kMmaWarps; ++w) g += tail_red[w][a];
                S[a][c] = g;
                continue;
            }
            const int ga = a >> 3, gc = c >> 3;
            const int t = ga * 4 - ga * (ga - 1) / 2 + (gc - ga);       // index of tile (ga, gc) in the upper triangle of 4 x 4
            double g = 0.0;
            for (int w = 0; w < kMmaWarps; ++w) g += red[(size_t)w * (kMmaTiles * 64) + t * 64 + (a & 7) * 8 + (c & 7)];
            S[a][c] = g;
        }
        __syncthreads();
        if (tid < M) nrm2[tid] = S[tid][tid];
        __syncthreads();
        for (int x = tid; x < M * M; x += kMmaThreads) {
            const int a = x / M, c = x % M;
            if (a >= c) continue;
            const double na = nrm2[a], nc = nrm2[c];
            const double cs = (na > 0.0 && nc > 0.0) ? S[a][c] / (sqrt(na) * sqrt(nc)) : 0.0;
            S[a][c] = cs;
            S[c][a] = cs;
        }
        __syncthreads();
    }
    if (tid < M) S[tid][tid] = 1.0;
    __syncthreads();
    if (tid < M) {
        const int a = tid;
        double mu = 0.0;
        for (int c = 0; c < M; ++c) mu += S[a][c];
        mu /= M;
        double var = 0.0;
        for (int c = 0; c < M; ++c) var += (S[a][c] - mu) * (S[a][c] - mu);
        p.s_spa[tok[a]] = var / M;
    }
}

// ---- per-frame standardisation and fusion: one CTA per frame ---------------------------------------------------
__device__ double standardise(double x, bool valid, int n, double *scratch) {
    const double mu = block_sum(valid ? x : 0.0, scratch) / n;
    const double dv = valid ? x - mu : 0.0;
    const double var = block_sum(dv * dv, scratch) / n;
    const double floor_ = 1e-24 * fmax(1.0, mu * mu);
    if (var <= floor_) return 0.0;
    return dv / sqrt(var);
}

__global__ void __launch_bounds__(1024) select_fuse_kernel(const SelectParams p) {
    __shared__ double scratch[32];
    const int gframe = blockIdx.x;
    const int b = find_seq(p.frame_off, p.batch, gframe);
    const int f = gframe - p.frame_off[b];
    const int n_v = p.seq_off[b + 1] - p.seq_off[b];
    const int n_frames = (n_v + p.tpf - 1) / p.tpf;
    const int nf = min(p.tpf, n_v - f * p.tpf);
    // blockDim.x >= tokens per frame (checked on the host): thread c owns grid cell c
    const int c = threadIdx.x;
    const bool valid = c < nf;
    const int j = p.seq_off[b] + f * p.tpf + c;
    double fused = 0.0;
    if (p.mask & HIPPO_SCORE_ATTN) fused += standardise(valid ? (double)p.attn_mass[j] : 0.0, valid, nf, scratch);
    if (p.mask & HIPPO_SCORE_SPA) fused += standardise(valid ? p.s_spa[j] : 0.0, valid, nf, scratch);
    if (p.mask & HIPPO_SCORE_TEMP) {
        double st = 0.0;
        if (valid) {
            double sum = 0.0;
            int cnt = 0;
            const double nj = p.norm2[j];
            if (f > 0) {  // previous frame always holds every cell
                const double nk = p.norm2[j - p.tpf];
                sum += (nj > 0.0 && nk > 0.0) ? p.tdot[j - p.tpf] / (sqrt(nj) * sqrt(nk)) : 0.0;
                ++cnt;
            }
            if (f + 1 < n_frames && c < min(p.tpf, n_v - (f + 1) * p.tpf)) {
                const double nk = p.norm2[j + p.tpf];
                sum += (nj > 0.0 && nk > 0.0) ? p.tdot[j] / (sqrt(nj) * sqrt(nk)) : 0.0;
                ++cnt;
            }
            st = 1.0 - (cnt ? sum / cnt : 0.0);
        }
        fused += standardise(st, valid, nf, scratch);
    }
    if (valid) p.fused[j] = (float)fused;
}

// ---- top-k: one CTA per sequence --------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t order_key(float x) {  // larger float -> larger key
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// smem_keys: keys beyond the 32 per thread that live in registers are staged in this many words of dynamic shared memory
__global__ void __launch_bounds__(1024) select_topk_kernel(const SelectParams p, const int smem_keys) {
    extern __shared__ uint32_t skeys[];
    __shared__ int warp_cnt[32];
    __shared__ uint32_t s_prefix;
    __shared__ int s_remaining, s_base_eq, s_base_out;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.seq_off[b + 1] - p.seq_off[b];
    const int k = p.k[b];
    if (k <= 0) return;
    const float *score = p.fused + p.seq_off[b];
    int32_t *out = p.kept + p.k_off[b];
    // The key T of the k-th largest element, two bits at a time from the top: T is the largest value with at least k
    // keys >= T.  Each thread keeps its keys in registers (32 per thread), the next ones in shared memory, and only
    // what is left beyond both is read again from memory, so a step is a few compares and one block-wide sum of three
    // counters.
    constexpr int kKeysPerThread = 32;
    __shared__ int warp_cnt3[32][3];
    __shared__ int s_cnt3[3];
    uint32_t keys[kKeysPerThread];
    const int n_regs = kKeysPerThread * (int)blockDim.x;            // keys [0, n_regs) in registers
    const int n_staged = min(n, n_regs + smem_keys);                 // keys [n_regs, n_staged) in shared memory
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        const int i = e * blockDim.x + tid;
        keys[e] = i < n ? order_key(score[i]) : 0u;   // padding: key 0 is never counted (candidates are > 0)
    }
    for (int i = n_regs + tid; i < n_staged; i += blockDim.x) skeys[i - n_regs] = order_key(score[i]);
    __syncthreads();
    const int per_thread = min(kKeysPerThread, (n + (int)blockDim.x - 1) / (int)blockDim.x);
    // counts of keys >= c1, >= c2, >= c3 over the sequence (candidates are non-zero)
    auto count3 = [&](uint32_t c1, uint32_t c2, uint32_t c3) {
        int a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
        for (int e0 = 0; e0 < kKeysPerThread; e0 += 8) {
            if (e0 < per_thread) {      // uniform: only the groups of eight that hold keys
#pragma unroll
                for (int e = e0; e < e0 + 8; ++e) {
                    a1 += keys[e] >= c1 ? 1 : 0; a2 += keys[e] >= c2 ? 1 : 0; a3 += keys[e] >= c3 ? 1 : 0;
                }
            }
        }
        for (int i = n_regs + tid; i < n_staged; i += blockDim.x) {
            const uint32_t key = skeys[i - n_regs];
            a1 += key >= c1 ? 1 : 0; a2 += key >= c2 ? 1 : 0; a3 += key >= c3 ? 1 : 0;
        }
        for (int i = n_staged + tid; i < n; i += blockDim.x) {
            const uint32_t key = order_key(score[i]);
            a1 += key >= c1 ? 1 : 0; a2 += key >= c2 ? 1 : 0; a3 += key >= c3 ? 1 : 0;
        }
        a1 = __reduce_add_sync(0xffffffffu, a1);
        a2 = __reduce_add_sync(0xffffffffu, a2);
        a3 = __reduce_add_sync(0xffffffffu, a3);
        __syncthreads();                 // the counters of the previous step have been read
        if (lane == 0) { warp_cnt3[warp][0] = a1; warp_cnt3[warp][1] = a2; warp_cnt3[warp][2] = a3; }
        __syncthreads();
        if (warp == 0) {
            const bool has = lane < (int)(blockDim.x >> 5);
            int t1 = has ? warp_cnt3[lane][0] : 0, t2 = has ? warp_cnt3[lane][1] : 0, t3 = has ? warp_cnt3[lane][2] : 0;
            t1 = __reduce_add_sync(0xffffffffu, t1);
            t2 = __reduce_add_sync(0xffffffffu, t2);
            t3 = __reduce_add_sync(0xffffffffu, t3);
            if (lane == 0) { s_cnt3[0] = t1; s_cnt3[1] = t2; s_cnt3[2] = t3; }
        }
        __syncthreads();
    };
    uint32_t Tsel = 0;
    for (int bit = 30; bit >= 0; bit -= 2) {
        // candidates with the two bits set to 01, 10, 11 (ascending): keep the largest that still has k keys above it
        const uint32_t c1 = Tsel | (1u << bit), c2 = Tsel | (2u << bit), c3 = Tsel | (3u << bit);
        count3(c1, c2, c3);
        if (s_cnt3[2] >= k) Tsel = c3; else if (s_cnt3[1] >= k) Tsel = c2; else if (s_cnt3[0] >= k) Tsel = c1;
    }
    int n_gt = 0;
    if (Tsel != 0xffffffffu) { count3(Tsel + 1, Tsel + 1, Tsel + 1); n_gt = s_cnt3[0]; }
    __syncthreads();
    if (tid == 0) { s_prefix = Tsel; s_remaining = k - n_gt; }
    __syncthreads();
    const uint32_t T = s_prefix;
    const int need_eq = s_remaining;  // elements equal to T to keep: those with the smallest indices
    if (tid == 0) { s_base_eq = 0; s_base_out = 0; }
    __syncthreads();
    // Ordered compaction.  Element i = e * blockDim.x + tid of the first n_regs sits in this thread's register e, so the
    // output position of a kept element is (kept elements of rows e' < e) + (kept elements of row e in lower threads).
    // Three sweeps over the registers, ballots only, and two scans of the 32 x 32 table of per-(row, warp) counts in
    // between: first the ranks of the elements equal to the threshold (only the need_eq lowest indices among them are
    // kept), then the output positions.
    __shared__ int cnt[32][33];
    __shared__ int row_tot[32];
    const int nw = blockDim.x >> 5;
    const int rows_used = min(kKeysPerThread, (n + (int)blockDim.x - 1) / (int)blockDim.x);
    // exclusive scan of cnt[e][w] in (e, w) order, in place; returns the grand total through row_tot[31]
    auto scan_counts = [&]() {
        __syncthreads();
        if (warp < rows_used) {
            const int c = lane < nw ? cnt[warp][lane] : 0;
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += v; }
            cnt[warp][lane] = inc - c;
            if (lane == 31) row_tot[warp] = inc;
        } else if (lane == 31) {
            row_tot[warp] = 0;
        }
        __syncthreads();
        if (warp == 0) {
            const int c = row_tot[lane];
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += v; }
            row_tot[lane] = inc - c;
            if (lane == 31) s_base_eq = inc;      // scratch: the grand total
        }
        __syncthreads();
    };
    const unsigned lt_mask = (1u << lane) - 1;
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        if (e < rows_used) {   // uniform
            const unsigned bal = __ballot_sync(0xffffffffu, e * (int)blockDim.x + tid < n && keys[e] == T);
            if (lane == 0) cnt[e][warp] = __popc(bal);
        }
    }
    scan_counts();
    const int eq_in_regs = s_base_eq;
    __syncthreads();
    __shared__ int eq_off[32][33];
    __shared__ int eq_row[32];
    for (int x = tid; x < 32 * 32; x += blockDim.x) eq_off[x >> 5][x & 31] = cnt[x >> 5][x & 31];
    if (tid < 32) eq_row[tid] = row_tot[tid];
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        if (e < rows_used) {
            const bool in = e * (int)blockDim.x + tid < n;
            const bool eq = in && keys[e] == T, gt = in && keys[e] > T;
            const unsigned bal_eq = __ballot_sync(0xffffffffu, eq);
            const int rank = eq_row[e] + eq_off[e][warp] + __popc(bal_eq & lt_mask);
            const unsigned bal = __ballot_sync(0xffffffffu, gt || (eq && rank < need_eq));
            if (lane == 0) cnt[e][warp] = __popc(bal);
        }
    }
    scan_counts();
    const int out_in_regs = s_base_eq;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) {
        if (e < rows_used) {
            const int i = e * (int)blockDim.x + tid;
            const bool in = i < n;
            const bool eq = in && keys[e] == T, gt = in && keys[e] > T;
            const unsigned bal_eq = __ballot_sync(0xffffffffu, eq);
            const int rank = eq_row[e] + eq_off[e][warp] + __popc(bal_eq & lt_mask);
            const bool sel = gt || (eq && rank < need_eq);
            const unsigned bal = __ballot_sync(0xffffffffu, sel);
            const int pos = row_tot[e] + cnt[e][warp] + __popc(bal & lt_mask);
            if (sel && pos < k) out[pos] = i;
        }
    }
    __syncthreads();
    if (tid == 0) { s_base_eq = eq_in_regs; s_base_out = out_in_regs; }
    __syncthreads();
    // what lies beyond the registers (more than 32 keys per thread): blockDim.x elements at a time, ranks from ballots,
    // warp offsets from a scan by warp 0
    __shared__ int tail_eq_off[33], sel_off[33];
    for (int start = n_regs; start < n; start += blockDim.x) {
        const int i = start + tid;
        const uint32_t key = i < n ? order_key(score[i]) : 0u;
        const bool gt = i < n && key > T, eq = i < n && key == T;
        const unsigned bal_eq = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) warp_cnt[warp] = __popc(bal_eq);
        __syncthreads();
        if (warp == 0) {
            const int c = lane < nw ? warp_cnt[lane] : 0;
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += v; }
            tail_eq_off[lane] = inc - c;
            if (lane == 31) tail_eq_off[32] = inc;
        }
        __syncthreads();
        const int eq_rank2 = s_base_eq + tail_eq_off[warp] + __popc(bal_eq & lt_mask);
        const bool sel = gt || (eq && eq_rank2 < need_eq);
        const unsigned bal = __ballot_sync(0xffffffffu, sel);
        if (lane == 0) warp_cnt[warp] = __popc(bal);
        __syncthreads();
        if (warp == 0) {
            const int c = lane < nw ? warp_cnt[lane] : 0;
            int inc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += v; }
            sel_off[lane] = inc - c;
            if (lane == 31) sel_off[32] = inc;
        }
        __syncthreads();
        const int pos = s_base_out + sel_off[warp] + __popc(bal & lt_mask);
        if (sel && pos < k) out[pos] = i;
        __syncthreads();
        if (tid == 0) { s_base_eq += tail_eq_off[32]; s_base_out += sel_off[32]; }
        __syncthreads();
    }
}

// ---- uniform budget per frame ------------------------------------------------------------------------------------
// Budgets of one sequence, by one thread: floor(k / F) per frame, the first k mod F frames one more; a frame with fewer
// tokens than its budget keeps them all and the shortfall goes, one token at a time in frame order, to the frames that
// still have room.  Also the first output position of every frame.
__global__ void select_budget_kernel(const SelectParams p) {
    const int b = blockIdx.x;
    if (threadIdx.x != 0) return;
    const int n = p.seq_off[b + 1] - p.seq_off[b], k = p.k[b];
    const int F = (n + p.tpf - 1) / p.tpf;
    int *budget = p.frame_budget + p.frame_off[b], *first = p.frame_out + p.frame_off[b];
    int given = 0;
    for (int f = 0; f < F; ++f) {
        const int want = k / F + (f < k % F ? 1 : 0), have = min(p.tpf, n - f * p.tpf);
        budget[f] = min(want, have);
        given += budget[f];
    }
    while (given < k)
        for (int f = 0; f < F && given < k; ++f)
            if (budget[f] < min(p.tpf, n - f * p.tpf)) { ++budget[f]; ++given; }
    int acc = 0;
    for (int f = 0; f < F; ++f) { first[f] = acc; acc += budget[f]; }
}

// One CTA per frame, thread c owns grid cell c: its rank among the frame's tokens by (score as fp32 descending, index
// ascending) is a count over the frame's keys in shared memory; the kept ones are written in index order.
__global__ void __launch_bounds__(1024) select_frame_topk_kernel(const SelectParams p) {
    __shared__ uint32_t keys[1024];
    __shared__ int warp_cnt[32];
    const int gframe = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = find_seq(p.frame_off, p.batch, gframe);
    const int f = gframe - p.frame_off[b];
    const int n_v = p.seq_off[b + 1] - p.seq_off[b];
    const int nf = min(p.tpf, n_v - f * p.tpf);
    const int kf = p.frame_budget[gframe];
    const bool valid = tid < nf;
    const uint32_t key = valid ? order_key(p.fused[p.seq_off[b] + f * p.tpf + tid]) : 0u;
    keys[tid] = key;
    __syncthreads();
    int rank = 0;
    for (int c = 0; c < nf; ++c) {
        const uint32_t other = keys[c];
        rank += (other > key || (other == key && c < tid)) ? 1 : 0;
    }
    const bool sel = valid && rank < kf;
    const unsigned bal = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) warp_cnt[warp] = __popc(bal);
    __syncthreads();
    int before = __popc(bal & ((1u << lane) - 1));
    for (int w = 0; w < warp; ++w) before += warp_cnt[w];
    if (sel) p.kept[p.k_off[b] + p.frame_out[gframe] + before] = f * p.tpf + tid;
}

// ---- whole frames at a regular stride --------------------------------------------------------------------------------
// Output position i of sequence b: with m = ceil(k / T) frames kept out of the Fc complete ones, frame floor(q * Fc / m)
// for q = i / T, cell i mod T (the last kept frame is cut short when k is not a multiple of T); when k reaches Fc * T, or
// there is no complete frame, the first k tokens.
__global__ void select_frames_kernel(const SelectParams p) {
    const int b = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int k = p.k[b];
    if (i >= k) return;
    const int n = p.seq_off[b + 1] - p.seq_off[b], T = p.tpf, Fc = n / T;
    int idx = i;
    if (Fc > 0 && (long long)k < (long long)Fc * T) {
        const int m = (k + T - 1) / T;
        idx = (int)((long long)(i / T) * Fc / m) * T + i % T;
    }
    p.kept[p.k_off[b] + i] = idx;
}

__global__ void select_copy_keys_kernel(const float *keys, float *fused, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) fused[i] = keys[i];
}

struct SelectWs { size_t norm2_off, tdot_off, spa_off, budget_off, total; };
static SelectWs select_ws(long long total_tokens, long long total_frames) {
    SelectWs w;
    const size_t a = align_up((size_t)total_tokens * sizeof(double), 256);
    w.norm2_off = kWsHeaderBytes;
    w.tdot_off = w.norm2_off + a;
    w.spa_off = w.tdot_off + a;
    w.budget_off = w.spa_off + a;       // per-frame policy: budget and first output position of every frame
    w.total = w.budget_off + align_up((size_t)total_frames * 2 * sizeof(int), 256);
    return w;
}

}  // namespace hippo

extern "C" {

size_t hippo_select_workspace_bytes(int32_t batch, const int32_t *n_visual, int32_t grid_h, int32_t grid_w,
                                    int32_t crop_h, int32_t crop_w) {
    (void)crop_h; (void)crop_w;
    if (batch <= 0 || !n_visual || grid_h <= 0 || grid_w <= 0) return 0;
    long long t = 0, f = 0;
    const long long tpf = (long long)grid_h * grid_w;
    for (int b = 0; b < batch; ++b) { if (n_visual[b] <= 0) return 0; t += n_visual[b]; f += (n_visual[b] + tpf - 1) / tpf; }
    return hippo::select_ws(t, f).total;
}

int32_t hippo_select_tokens(int32_t batch, const int32_t *n_visual, int32_t grid_h, int32_t grid_w, int32_t crop_h,
                            int32_t crop_w, int32_t embed_dim, int32_t dtype, const void *embeds,
                            const float *attn_mass, const int32_t *k, const int32_t *kept_offsets,
                            uint32_t score_mask, int32_t *kept_idx, float *fused_score, void *workspace,
                            size_t workspace_bytes, void *stream) {
    return hippo_select_tokens_policy(batch, n_visual, grid_h, grid_w, crop_h, crop_w, embed_dim, dtype, embeds, attn_mass, k,
                                      kept_offsets, score_mask, HIPPO_SELECT_HOLISTIC, nullptr, kept_idx, fused_score,
                                      workspace, workspace_bytes, stream);
}

int32_t hippo_select_tokens_policy(int32_t batch, const int32_t *n_visual, int32_t grid_h, int32_t grid_w, int32_t crop_h,
                                   int32_t crop_w, int32_t embed_dim, int32_t dtype, const void *embeds,
                                   const float *attn_mass, const int32_t *k, const int32_t *kept_offsets,
                                   uint32_t score_mask, int32_t policy, const float *random_keys, int32_t *kept_idx,
                                   float *fused_score, void *workspace, size_t workspace_bytes, void *stream) {
    using namespace hippo;
    const char *who = "hippo_select_tokens";
    if (batch <= 0 || !n_visual || !k) return fail(HIPPO_ERR_INVALID_ARG, "%s: bad batch / null host arrays", who);
    if (policy < HIPPO_SELECT_HOLISTIC || policy > HIPPO_SELECT_FRAMES) return fail(HIPPO_ERR_INVALID_ARG, "%s: unknown policy %d", who, policy);
    const bool scored = policy == HIPPO_SELECT_HOLISTIC || policy == HIPPO_SELECT_UNIFORM_PER_FRAME;
    if (policy == HIPPO_SELECT_RANDOM && !random_keys) return fail(HIPPO_ERR_INVALID_ARG, "%s: the random policy needs random_keys", who);
    if (batch > kSelMaxBatch) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: batch > %d", who, kSelMaxBatch);
    if (grid_h <= 0 || grid_w <= 0 || crop_h <= 0 || crop_w <= 0 || embed_dim <= 0)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: non-positive geometry", who);
    if (dtype != HIPPO_DTYPE_FP32 && dtype != HIPPO_DTYPE_BF16) return fail(HIPPO_ERR_INVALID_ARG, "%s: unknown dtype", who);
    if (crop_h * crop_w > kMaxCrop) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: crop larger than %d tokens", who, kMaxCrop);
    if ((long long)grid_h * grid_w > 1024) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: more than 1024 tokens per frame", who);
    if (embed_dim % 8) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: embed_dim must be a multiple of 8", who);
    if (!workspace || (scored && (!embeds || !attn_mass)) || (policy != HIPPO_SELECT_FRAMES && !fused_score))
        return fail(HIPPO_ERR_INVALID_ARG, "%s: null pointer", who);
    if ((score_mask & ~HIPPO_SCORE_ALL) != 0) return fail(HIPPO_ERR_INVALID_ARG, "%s: unknown score_mask bits", who);
    if ((uintptr_t)workspace & 255) return fail(HIPPO_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", who);
    if (scored && ((uintptr_t)embeds & 15)) return fail(HIPPO_ERR_INVALID_ARG, "%s: embeds must be 16-byte aligned", who);

    SelectParams p;
    p.tpf = grid_h * grid_w;
    long long tok = 0, frames = 0, ksum = 0;
    for (int b = 0; b < batch; ++b) {
        if (n_visual[b] <= 0) return fail(HIPPO_ERR_INVALID_ARG, "%s: n_visual[%d] <= 0", who, b);
        if (k[b] < 0 || k[b] > n_visual[b]) return fail(HIPPO_ERR_INVALID_ARG, "%s: k[%d] outside [0, n_visual]", who, b);
        p.seq_off[b] = (int)tok; p.frame_off[b] = (int)frames; p.k[b] = k[b];
        if (kept_offsets && kept_offsets[b] < 0) return fail(HIPPO_ERR_INVALID_ARG, "%s: kept_offsets[%d] < 0", who, b);
        p.k_off[b] = kept_offsets ? kept_offsets[b] : (int)ksum;
        tok += n_visual[b]; frames += (n_visual[b] + p.tpf - 1) / p.tpf; ksum += k[b];
        if (tok > 0x7fffffffLL / 2) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: too many tokens", who);
    }
    p.seq_off[batch] = (int)tok; p.frame_off[batch] = (int)frames; p.k_off[batch] = (int)ksum;
    if (ksum > 0 && !kept_idx) return fail(HIPPO_ERR_INVALID_ARG, "%s: null kept_idx", who);
    SelectWs w = select_ws(tok, frames);
    if (workspace_bytes < w.total) return fail(HIPPO_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu bytes", who, workspace_bytes, w.total);
    p.embeds = embeds; p.attn_mass = attn_mass; p.fused = fused_score; p.kept = kept_idx;
    p.norm2 = (double *)((char *)workspace + w.norm2_off);
    p.tdot = (double *)((char *)workspace + w.tdot_off);
    p.s_spa = (double *)((char *)workspace + w.spa_off);
    p.frame_budget = (int *)((char *)workspace + w.budget_off);
    p.frame_out = p.frame_budget + frames;
    p.batch = batch; p.grid_h = grid_h; p.grid_w = grid_w; p.crop_h = crop_h; p.crop_w = crop_w; p.d = embed_dim;
    p.crops_y = ceil_div(grid_h, crop_h); p.crops_x = ceil_div(grid_w, crop_w);
    p.mask = score_mask;
    cudaStream_t s = (cudaStream_t)stream;
    if (policy == HIPPO_SELECT_FRAMES) {
        // an index rule: no scores are formed, fused_score is not written
        int kmax = 0;
        for (int b = 0; b < batch; ++b) kmax = k[b] > kmax ? k[b] : kmax;
        if (kmax > 0) {
            select_frames_kernel<<<dim3((unsigned)ceil_div(kmax, 256), (unsigned)batch), 256, 0, s>>>(p);
            count_launches(1);
        }
        HIPPO_CUDA_TRY(cudaGetLastError());
        return HIPPO_OK;
    }
    if (policy == HIPPO_SELECT_RANDOM) {
        // the caller's keys take the place of the fused score (and are returned as such)
        select_copy_keys_kernel<<<(unsigned)((tok + 255) / 256), 256, 0, s>>>(random_keys, fused_score, (int)tok);
        count_launches(1);
    }
    const bool need_emb = scored && (score_mask & (HIPPO_SCORE_TEMP | HIPPO_SCORE_SPA)) != 0;
    if (need_emb) {
        const int warps = 8;
        dim3 g1((unsigned)((tok + warps - 1) / warps));
        if (dtype == HIPPO_DTYPE_FP32) select_dots_kernel<float><<<g1, warps * 32, 0, s>>>(p);
        else select_dots_kernel<__nv_bfloat16><<<g1, warps * 32, 0, s>>>(p);
        count_launches(1);
    }
    if (scored && (score_mask & HIPPO_SCORE_SPA)) {
        dim3 g2((unsigned)(frames * p.crops_y * p.crops_x));
        static PerDeviceOnce spa_attr;
        int dev;
        if (spa_attr.needed(dev)) {
            HIPPO_CUDA_TRY(cudaFuncSetAttribute(select_spatial_mma_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MmaShape<float>::kSmemBytes));
            HIPPO_CUDA_TRY(cudaFuncSetAttribute(select_spatial_mma_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MmaShape<__nv_bfloat16>::kSmemBytes));
            spa_attr.mark(dev);
        }
        if (dtype == HIPPO_DTYPE_FP32) select_spatial_mma_kernel<float><<<g2, kMmaThreads, MmaShape<float>::kSmemBytes, s>>>(p);
        else select_spatial_mma_kernel<__nv_bfloat16><<<g2, kMmaThreads, MmaShape<__nv_bfloat16>::kSmemBytes, s>>>(p);
        count_launches(1);
    }
    const int fuse_threads = ((p.tpf + 31) / 32) * 32;
    if (scored) {
        select_fuse_kernel<<<(unsigned)frames, fuse_threads, 0, s>>>(p);
        count_launches(1);
    }
    if (ksum > 0 && policy == HIPPO_SELECT_UNIFORM_PER_FRAME) {
        select_budget_kernel<<<batch, 32, 0, s>>>(p);
        select_frame_topk_kernel<<<(unsigned)frames, fuse_threads, 0, s>>>(p);
        count_launches(2);
    } else if (ksum > 0) {
        // shared-memory staging for the keys beyond 32 per thread, up to 48K of them
        int longest = 0;
        for (int b = 0; b < batch; ++b) longest = n_visual[b] > longest ? n_visual[b] : longest;
        int smem_keys = longest - 32 * 1024;
        smem_keys = smem_keys < 0 ? 0 : (smem_keys > 48 * 1024 ? 48 * 1024 : smem_keys);
        static PerDeviceOnce topk_attr;
        int dev;
        if (topk_attr.needed(dev)) {
            HIPPO_CUDA_TRY(cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 48 * 1024 * 4));
            topk_attr.mark(dev);
        }
        select_topk_kernel<<<batch, 1024, (size_t)smem_keys * 4, s>>>(p, smem_keys);
        count_launches(1);
    }
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}

}  // extern "C"
