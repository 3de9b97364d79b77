// Tensor-core split-KV attention for sm_100a: bf16 K/V pages streamed by TMA, QK^T and PV on tcgen05 with the
// accumulators in tensor memory.  Used for the verification pass (gamma+1 query tokens against the full video KV
// cache) and for the draft decode pass over the pruned cache (Section 3.2).
//
// Packing.  All query rows that read one KV head - the q_len tokens times the G = H_q/H_kv heads of its group - are
// packed as rows r = t*G + g of one M = 128 operand, so every K/V tile is fetched from HBM once per sequence and
// feeds up to 128 rows of tensor-core work.
//
// Work split.  The 64-key tiles of all (sequence, kv head) units form one flat list that is cut into gridDim.x equal
// contiguous ranges (persistent CTAs, one per SM).  A CTA walks its range unit by unit ("segments"); for each
// segment it produces either the final output (it owns the whole unit) or a partial (m, l, O) in slot unit+cta of
// the workspace, which the combine kernel merges.
//
// CTA = 6 warps:  warp 0 TMA producer (ring of kStages K+V tiles, full/empty mbarriers)
//                 warp 1 tcgen05.mma issuer and TMEM owner:  S[j] = Q K_i^T  (double buffered),  O += P_i V_i
//                 warps 2-5: one thread per packed row: S -> registers, online softmax in base 2 with lazy
//                 rescaling of O, P -> shared memory (bf16, 128B swizzle), epilogue.
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA records HIPPO_ERR_TIMEOUT in the
// workspace header, drains its own copies, frees its tensor memory and exits.
#include <cuda.h>
#include <math.h>

#include "common.cuh"

namespace hippo {

constexpr int kTcThreads = 192;
constexpr int kBlockN = 64;            // keys per tile = one KV page
constexpr int kBlockM = 128;           // packed rows (padded)
constexpr int kTcMaxBatch = 256;       // per-sequence tile prefix lives in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;              // lazy rescale: only when the running max grows by > 2^8
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

template <int D> struct TcCfg {
    static constexpr int kChunks = D / 64;                       // 64-column (128-byte) swizzle chunks per row
    static constexpr int kQBytes = kBlockM * D * 2;
    static constexpr int kPBytes = kBlockM * kBlockN * 2;         // one P buffer
    static constexpr int kTileBytes = kBlockN * D * 2;            // one K or V tile
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = D == 128 ? 5 : 8;
    static constexpr int kDataBytes = kQBytes + 2 * kPBytes + kStages * kStageBytes;
    static constexpr int kTmemCols = 256;                         // S0 | S1 | O
    static constexpr int kColS = 0, kColO = 128;
};

// ---- PTX wrappers -------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
    uint32_t *r = reinterpret_cast<uint32_t *>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                   "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
                   "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                   "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float *v) {
    const uint32_t *r = reinterpret_cast<const uint32_t *>(v);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
                   "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
                   "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
                   "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, Blackwell version field.  Offsets in bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBlockM >> 4) << 24);
}

// ---- work partition (shared by the main and the combine kernel) ---------------------------------------------------
struct Partition {
    long long total;   // tiles over all units
    int grid;          // CTAs
    __device__ __forceinline__ long long start_of(int c) const { return (long long)c * total / grid; }
    __device__ __forceinline__ int cta_of(long long t) const { return (int)(((t + 1) * grid - 1) / total); }
};

__device__ __forceinline__ int seq_tiles(int kvl, int q_len) { return kvl < q_len ? 0 : (kvl + kBlockN - 1) / kBlockN; }

// ---- shared control block -------------------------------------------------------------------------------------------
struct TcShared {
    unsigned long long full[8], empty[8], s_full[2], s_free[2], p_full[2], pv_done[2], q_full, q_free, drain;
    uint32_t tmem_base;
    volatile int abort;
    int tile_prefix[kTcMaxBatch + 1];  // only [0, batch] used
};

struct Waiter {
    TcShared *sh;
    WsHeader *hdr;
    __device__ __forceinline__ bool wait(unsigned long long *bar, uint32_t parity, int site) const {
        const uint32_t b = smem_u32(bar);
        if (mbar_try_wait(b, parity)) return true;
        const unsigned long long t0 = global_ns();
        for (uint32_t i = 1;; ++i) {
            if (mbar_try_wait(b, parity)) return true;
            if ((i & 31) == 0) {
                if (sh->abort) return false;
                if (global_ns() - t0 > kWaitLimitNs) {
                    sh->abort = 1;
                    atomicExch(&hdr->status, (int)HIPPO_ERR_TIMEOUT);
                    hdr->where = site;
                    return false;
                }
            }
        }
    }
};

template <int D> constexpr int tc_smem_bytes() { return TcCfg<D>::kDataBytes + 1024 /* alignment */ + (int)sizeof(TcShared); }
static_assert(tc_smem_bytes<128>() <= 227 * 1024, "shared memory budget");

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map) {
    using C = TcCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *q_s = base;                                    // [kChunks][128 rows][128 B]
    uint8_t *p_s = q_s + C::kQBytes;                        // [2][128 rows][128 B]
    uint8_t *kv_s = p_s + 2 * C::kPBytes;                   // [kStages][K: kChunks x 8 KB | V: kChunks x 8 KB]
    TcShared *sh = (TcShared *)(kv_s + C::kStages * C::kStageBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = p.rows, G = p.group, Hkv = p.n_kv_heads, B = p.batch;
    const Waiter W{sh, p.header};

    // ---- set-up: barriers, tile prefix, tensor memory
    if (tid == 0) {
        for (int s = 0; s < C::kStages; ++s) { mbar_init(smem_u32(&sh->full[s]), 1); mbar_init(smem_u32(&sh->empty[s]), 1); }
        for (int j = 0; j < 2; ++j) {
            mbar_init(smem_u32(&sh->s_full[j]), 1);
            mbar_init(smem_u32(&sh->s_free[j]), 128);
            mbar_init(smem_u32(&sh->p_full[j]), 128);
            mbar_init(smem_u32(&sh->pv_done[j]), 1);
        }
        mbar_init(smem_u32(&sh->q_full), 128);
        mbar_init(smem_u32(&sh->q_free), 1);
        mbar_init(smem_u32(&sh->drain), 1);
        sh->abort = 0;
        int acc = 0;
        for (int b = 0; b < B; ++b) { sh->tile_prefix[b] = acc; acc += seq_tiles(p.kv_len[b], p.q_len); }
        sh->tile_prefix[B] = acc;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;

    Partition part;
    part.total = (long long)sh->tile_prefix[B] * Hkv;
    part.grid = gridDim.x;
    const long long t_begin = part.total > 0 ? part.start_of(blockIdx.x) : 0;
    const long long t_end = part.total > 0 ? part.start_of(blockIdx.x + 1) : 0;

    // Segment iteration state shared by all roles: each role walks the same list of segments.
    // A segment = (b, hk, first tile, tile count, final?) derived from the flat range [t_begin, t_end).
    auto locate = [&](long long t, int &b, int &hk, int &tile) {
        // unit-major order: all tiles of (b, hk=0), then (b, hk=1), ...
        int lo = 0, hi = B;  // largest b with Hkv * prefix[b] <= t
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if ((long long)sh->tile_prefix[mid] * Hkv <= t) lo = mid; else hi = mid;
        }
        // skip sequences with zero tiles that share the same prefix
        b = lo;
        while (b + 1 < B && (long long)sh->tile_prefix[b + 1] * Hkv <= t) ++b;
        const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
        const long long off = t - (long long)sh->tile_prefix[b] * Hkv;
        hk = (int)(off / nt);
        tile = (int)(off % nt);
    };

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t it = 0;
            long long t = t_begin;
            bool ok = true;
            while (ok && t < t_end) {
                int b, hk, tile;
                locate(t, b, hk, tile);
                const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                const int n = (int)min((long long)(nt - tile), t_end - t);
                for (int i = 0; i < n && ok; ++i, ++it) {
                    const int s = it % C::kStages;
                    ok = W.wait(&sh->empty[s], ((it / C::kStages) & 1) ^ 1, 1);
                    if (!ok) break;
                    const int pid = page_of(p.page_table, p.max_pages_per_seq, b, tile + i);
                    const int row = (pid * Hkv + hk) * kPageSize;
                    const uint32_t bar = smem_u32(&sh->full[s]);
                    mbar_expect_tx(bar, C::kStageBytes);
                    const uint32_t dst = smem_u32(kv_s + s * C::kStageBytes);
#pragma unroll
                    for (int c = 0; c < C::kChunks; ++c) tma_load_2d(dst + c * 8192, &k_map, c * 64, row, bar);
#pragma unroll
                    for (int c = 0; c < C::kChunks; ++c) tma_load_2d(dst + C::kTileBytes + c * 8192, &v_map, c * 64, row, bar);
                }
                t += n;
            }
            // drain: every load that was issued must have landed before the CTA may exit
            const uint32_t issued = it;
            for (uint32_t k = (issued > (uint32_t)C::kStages ? issued - C::kStages : 0); k < issued; ++k)
                W.wait(&sh->full[k % C::kStages], (k / C::kStages) & 1, 2);
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(kBlockN, false);
            constexpr uint32_t idesc_pv = instr_desc(D, true);
            uint32_t it = 0, seg = 0;
            long long t = t_begin;
            bool ok = true;
            // issues O += P_i V_i for global tile counter `k` (stage and buffers derive from k)
            auto issue_pv = [&](uint32_t k, bool first_of_segment) -> bool {
                const int j = k & 1, s = k % C::kStages;
                if (!W.wait(&sh->p_full[j], (k >> 1) & 1, 3)) return false;
                tc_fence_after();
                const uint32_t pa = smem_u32(p_s + j * C::kPBytes);
                const uint32_t va = smem_u32(kv_s + s * C::kStageBytes + C::kTileBytes);
#pragma unroll
                for (int ks = 0; ks < kBlockN / 16; ++ks)
                    tc_mma(tmem + C::kColO, smem_desc(pa + ks * 32, 16, 1024), smem_desc(va + ks * 2048, 8192, 1024), idesc_pv,
                           (first_of_segment && ks == 0) ? 0u : 1u);
                tc_commit(smem_u32(&sh->pv_done[j]));
                tc_commit(smem_u32(&sh->empty[s]));
                return true;
            };
            while (ok && t < t_end) {
                int b, hk, tile;
                locate(t, b, hk, tile);
                const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                const int n = (int)min((long long)(nt - tile), t_end - t);
                ok = W.wait(&sh->q_full, seg & 1, 4);  // Q of this segment is in shared memory
                const uint32_t it0 = it;
                for (int i = 0; i < n && ok; ++i, ++it) {
                    const int j = it & 1, s = it % C::kStages;
                    ok = W.wait(&sh->full[s], (it / C::kStages) & 1, 5);
                    if (!ok) break;
                    // S buffer j was last read by the softmax of tile it-2
                    if (it >= 2) { ok = W.wait(&sh->s_free[j], ((it - 2) >> 1) & 1, 14); if (!ok) break; }
                    tc_fence_after();
                    const uint32_t qa = smem_u32(q_s), ka = smem_u32(kv_s + s * C::kStageBytes);
#pragma unroll
                    for (int c = 0; c < C::kChunks; ++c)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            tc_mma(tmem + C::kColS + j * kBlockN, smem_desc(qa + c * 16384 + ks * 32, 16, 1024),
                                   smem_desc(ka + c * 8192 + ks * 32, 16, 1024), idesc_qk, (c | ks) ? 1u : 0u);
                    tc_commit(smem_u32(&sh->s_full[j]));
                    if (i == n - 1) tc_commit(smem_u32(&sh->q_free));  // last QK of the segment: Q may be replaced
                    if (i >= 2) ok = issue_pv(it - 2, it - 2 == it0);    // PV trails QK by two tiles
                }
                for (uint32_t k = (n >= 2 ? it - 2 : it0); ok && k < it; ++k) ok = issue_pv(k, k == it0);
                t += n;
                ++seg;
            }
            // all tensor-core work of this CTA must be complete before tensor memory is released
            tc_commit(smem_u32(&sh->drain));
            W.wait(&sh->drain, 0, 6);
        }
    } else {
        // ================= softmax / epilogue: one thread per packed row =================
        const int quarter = warp & 3;                 // TMEM lanes this warp may access: 32*quarter .. +31
        const int r = quarter * 32 + lane;            // packed row
        const bool warp_active = quarter * 32 < R;
        const bool row_active = r < R;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const float sl2 = p.scale * kLog2e;
        const int t_row = r / G, g_row = r % G;
        uint32_t it = 0, seg = 0;
        long long t = t_begin;
        bool ok = true;
        while (ok && t < t_end) {
            int b, hk, tile;
            locate(t, b, hk, tile);
            const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
            const int n = (int)min((long long)(nt - tile), t_end - t);
            const int kvl = p.kv_len[b];
            const bool whole_unit = (tile == 0 && n == nt);
            // ---- Q of this segment -> shared memory (swizzled K-major), after the previous segment's QK MMAs are done
            if (seg > 0) ok = W.wait(&sh->q_free, (seg - 1) & 1, 7);
            if (!ok) break;
            {
                const __nv_bfloat16 *qg = (const __nv_bfloat16 *)p.q + (((size_t)b * p.q_len + t_row) * p.n_q_heads + hk * G + g_row) * D;
#pragma unroll
                for (int c = 0; c < D / 8; ++c) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (row_active) v = __ldg(reinterpret_cast<const uint4 *>(qg) + c);
                    *reinterpret_cast<uint4 *>(q_s + (c >> 3) * 16384 + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
                }
                fence_proxy_async();
                mbar_arrive(smem_u32(&sh->q_full));
            }
            const int limit = kvl - p.q_len + t_row;   // last visible key of this row
            float m_ref = -INFINITY, l_sum = 0.f;
            const uint32_t it0 = it;
            for (int i = 0; i < n && ok; ++i, ++it) {
                const int j = it & 1, s = it % C::kStages;
                const int key0 = (tile + i) * kBlockN;
                const bool tail = key0 + kBlockN > kvl - p.q_len + 1;  // some row needs masking in this tile
                if (key0 + kBlockN > kvl) {
                    // rows of V past the end of the sequence may hold anything: zero them (0 * NaN would poison O)
                    ok = W.wait(&sh->full[s], (it / C::kStages) & 1, 8);
                    if (!ok) break;
                    uint8_t *vs = kv_s + s * C::kStageBytes + C::kTileBytes;
                    const int first_bad = kvl - key0;
                    for (int x = (tid - 64); x < (kBlockN - first_bad) * C::kChunks * 8; x += 128) {
                        const int row = first_bad + x / (C::kChunks * 8), rem = x % (C::kChunks * 8);
                        *reinterpret_cast<uint4 *>(vs + (rem >> 3) * 8192 + row * 128 + ((rem & 7) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                }
                ok = W.wait(&sh->s_full[j], (it >> 1) & 1, 9);
                if (!ok) break;
                tc_fence_after();
                float sv[kBlockN];
                if (warp_active) {
                    tmem_ld32(tmem + lane_addr + C::kColS + j * kBlockN, sv);
                    tmem_ld32(tmem + lane_addr + C::kColS + j * kBlockN + 32, sv + 32);
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh->s_free[j]));   // S buffer may be overwritten by QK of tile it+2
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < kBlockN; ++c) {
                        float x = sv[c] * sl2;
                        if (tail && key0 + c > limit) x = -INFINITY;
                        sv[c] = x;
                        mx4[c & 3] = fmaxf(mx4[c & 3], x);
                    }
                    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                    // lazy rescale of the running output: only when the maximum moved by more than the threshold
                    bool need = (m_ref == -INFINITY) ? false : (mx > m_ref + kRescaleThreshold);
                    if (m_ref == -INFINITY && mx != -INFINITY) m_ref = mx;   // first visible keys: adopt, O is still empty
                    if (__any_sync(0xffffffffu, need)) {
                        // O holds tiles it0..it-1: wait until PV of tile it-1 has been accumulated
                        if (it > it0) {
                            ok = W.wait(&sh->pv_done[(it - 1) & 1], ((it - 1) >> 1) & 1, 10);
                            if (!ok) break;
                            tc_fence_after();
                            const float f = need ? exp2f(m_ref - mx) : 1.f;
                            float ov[32];
#pragma unroll
                            for (int c = 0; c < D / 32; ++c) {
                                tmem_ld32(tmem + lane_addr + C::kColO + c * 32, ov);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 32; ++e) ov[e] *= f;
                                tmem_st32(tmem + lane_addr + C::kColO + c * 32, ov);
                            }
                            tmem_wait_st();
                            if (need) { l_sum *= f; m_ref = mx; }
                        } else if (need) {
                            l_sum *= exp2f(m_ref - mx);
                            m_ref = mx;
                        }
                    }
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    // P buffer j was last read by PV of tile it-2
                    if (it >= 2) { ok = W.wait(&sh->pv_done[j], ((it - 2) >> 1) & 1, 11); if (!ok) break; }
                    uint8_t *prow = p_s + j * C::kPBytes + r * 128;
                    float ls4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int c = 0; c < kBlockN / 8; ++c) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float a = ex2_approx(sv[c * 8 + 2 * e] - m_use), bb = ex2_approx(sv[c * 8 + 2 * e + 1] - m_use);
                            ls4[e] += a + bb;
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(a, bb);
                            w[e] = *reinterpret_cast<uint32_t *>(&h2);
                        }
                        *reinterpret_cast<uint4 *>(prow + ((c ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    l_sum += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
                } else {
                    mbar_arrive(smem_u32(&sh->s_free[j]));
                    if (it >= 2) { ok = W.wait(&sh->pv_done[j], ((it - 2) >> 1) & 1, 12); if (!ok) break; }
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(smem_u32(&sh->p_full[j]));
            }
            if (!ok) break;
            // ---- epilogue of the segment
            if (n > 0) {
                ok = W.wait(&sh->pv_done[(it - 1) & 1], ((it - 1) >> 1) & 1, 13);
                if (!ok) break;
                tc_fence_after();
            }
            if (warp_active) {
                const int unit = b * Hkv + hk;
                float *slot = p.partials + (size_t)(unit + blockIdx.x) * slot_float_count(R, D);
                const int Rp = slot_rows_padded(R);
                const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
                __nv_bfloat16 *og = (__nv_bfloat16 *)p.out + (((size_t)b * p.q_len + t_row) * p.n_q_heads + hk * G + g_row) * D;
                float ov[32];
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    tmem_ld32(tmem + lane_addr + C::kColO + c * 32, ov);
                    tmem_wait_ld();
                    if (row_active) {
                        if (whole_unit) {
#pragma unroll
                            for (int e = 0; e < 32; e += 8) {
                                uint32_t w[4];
#pragma unroll
                                for (int x = 0; x < 4; ++x) {
                                    __nv_bfloat162 h2 = __floats2bfloat162_rn(ov[e + 2 * x] * inv, ov[e + 2 * x + 1] * inv);
                                    w[x] = *reinterpret_cast<uint32_t *>(&h2);
                                }
                                *reinterpret_cast<uint4 *>(og + c * 32 + e) = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        } else {
                            float4 *dst = reinterpret_cast<float4 *>(slot + 2 * Rp + (size_t)r * D + c * 32);
#pragma unroll
                            for (int e = 0; e < 8; ++e) dst[e] = make_float4(ov[4 * e], ov[4 * e + 1], ov[4 * e + 2], ov[4 * e + 3]);
                        }
                    }
                }
                if (row_active) {
                    if (whole_unit) {
                        if (p.lse) p.lse[((size_t)b * p.q_len + t_row) * p.n_q_heads + hk * G + g_row] =
                            l_sum > 0.f ? m_ref * kLn2 + logf(l_sum) : -INFINITY;
                    } else {
                        slot[r] = (m_ref == -INFINITY) ? -INFINITY : m_ref * kLn2;   // natural-log domain for the combine
                        slot[Rp + r] = l_sum;
                    }
                }
            }
            tc_fence_before();
            t += n;
            ++seg;
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
    }
}

// Merge of the per-CTA partials of one output row (b, t, h); rows whose unit was owned by a single CTA were written
// by it and are skipped.  One CTA of D threads per row: warp 0 turns the contributors' (m, l) into normalised
// weights with lane-parallel loads, then thread d accumulates column d over the contributors with independent,
// coalesced loads.
template <int D>
__global__ void __launch_bounds__(D) attn_tc_combine_kernel(const AttnParams p, int grid_main) {
    __shared__ float w_s[kExtraSlots];
    __shared__ float s_lse;
    const int R = p.rows, G = p.group, Hkv = p.n_kv_heads;
    const int row = blockIdx.x, tid = threadIdx.x;
    const int h = row % p.n_q_heads, t = (row / p.n_q_heads) % p.q_len, b = row / (p.n_q_heads * p.q_len);
    const int hk = h / G, r = t * G + (h % G);
    __nv_bfloat16 *out = (__nv_bfloat16 *)p.out + (size_t)row * D;
    long long before = 0, total = 0;
    for (int i = 0; i < p.batch; ++i) {
        const int nt_i = seq_tiles(p.kv_len[i], p.q_len);
        if (i < b) before += nt_i;
        total += nt_i;
    }
    const int nt = seq_tiles(p.kv_len[b], p.q_len);
    if (nt == 0) {
        out[tid] = __float2bfloat16_rn(0.f);
        if (p.lse && tid == 0) p.lse[row] = -INFINITY;
        return;
    }
    Partition part;
    part.total = total * Hkv;
    part.grid = grid_main;
    const long long u0 = before * Hkv + (long long)hk * nt, u1 = u0 + nt;
    const int c0 = part.cta_of(u0), c1 = part.cta_of(u1 - 1);
    if (c0 == c1) return;
    const int n = c1 - c0 + 1;
    const size_t slot_floats = slot_float_count(R, D);
    const int Rp = slot_rows_padded(R);
    const float *base = p.partials + (size_t)(b * Hkv + hk + c0) * slot_floats;   // slot index = unit + cta
    if (tid < 32) {
        float M = -INFINITY;
        for (int c = tid; c < n; c += 32) M = fmaxf(M, base[(size_t)c * slot_floats + r]);
        for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float L = 0.f;
        for (int c = tid; c < n; c += 32) {
            const float m = base[(size_t)c * slot_floats + r];
            const float w = (m == -INFINITY) ? 0.f : expf(m - M);
            w_s[c] = w;
            L += base[(size_t)c * slot_floats + Rp + r] * w;
        }
        for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
        const float inv = L > 0.f ? 1.f / L : 0.f;
        for (int c = tid; c < n; c += 32) w_s[c] *= inv;
        if (tid == 0) s_lse = L > 0.f ? M + logf(L) : -INFINITY;
    }
    __syncthreads();
    const float *o = base + 2 * Rp + (size_t)r * D + tid;
    float acc = 0.f;
#pragma unroll 8
    for (int c = 0; c < n; ++c) acc = fmaf(o[(size_t)c * slot_floats], w_s[c], acc);
    out[tid] = __float2bfloat16_rn(acc);
    if (p.lse && tid == 0) p.lse[row] = s_lse;
}

// ---- host side -----------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

static int32_t make_map(CUtensorMap *m, const void *pool, long long rows, int D) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kBlockN};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return HIPPO_OK;
}

bool attn_tc_supported(const AttnParams &p, int dtype) {
    return dtype == HIPPO_DTYPE_BF16 && (p.head_dim == 64 || p.head_dim == 128) && p.batch <= kTcMaxBatch &&
           p.rows <= kBlockM;
}

template <int D>
static int32_t launch_tc(const AttnParams &p, int grid, cudaStream_t stream) {
    CUtensorMap km, vm;
    const long long rows = (long long)p.n_pages * p.n_kv_heads * kPageSize;
    int32_t rc = make_map(&km, p.k_pages, rows, D);
    if (rc != HIPPO_OK) return rc;
    rc = make_map(&vm, p.v_pages, rows, D);
    if (rc != HIPPO_OK) return rc;
    static bool attr_set = false;
    if (!attr_set) {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc_smem_bytes<D>()));
        attr_set = true;
    }
    attn_tc_kernel<D><<<grid, kTcThreads, tc_smem_bytes<D>(), stream>>>(p, km, vm);
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    const int total_rows = p.batch * p.q_len * p.n_q_heads;
    attn_tc_combine_kernel<D><<<total_rows, D, 0, stream>>>(p, grid);
    count_launches(1);
    HIPPO_CUDA_TRY(cudaGetLastError());
    return HIPPO_OK;
}

int32_t launch_attn_tc(const AttnParams &p, bool draft_policy, cudaStream_t stream) {
    (void)draft_policy;
    // Upper bound of the tile count from the host-side length bound; the kernel derives the exact partition from
    // kv_len on the device.  The grid never exceeds the bound, so no CTA is started without work to look for.
    const long long max_tiles = (long long)p.batch * p.n_kv_heads * ceil_div(p.max_kv_len, kBlockN);
    long long grid = p.num_splits > 0 ? (long long)p.num_splits * p.batch * p.n_kv_heads : kNumSMs;
    if (grid > max_tiles) grid = max_tiles;
    if (grid > kExtraSlots) grid = kExtraSlots;
    if (grid < 1) grid = 1;
    if (p.head_dim == 128) return launch_tc<128>(p, (int)grid, stream);
    return launch_tc<64>(p, (int)grid, stream);
}

}  // namespace hippo
