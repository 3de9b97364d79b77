// Tensor-core split-KV attention for sm_100a: bf16 K/V pages streamed by TMA, both contractions on tcgen05 with the
// accumulators in tensor memory.  Used for the verification pass (gamma+1 query tokens against the full video KV
// cache) and for the draft decode pass over the pruned cache (Section 3.2).
//
// Operand order.  The path is bound by reading K and V once; the query side is tiny: all query rows that read one
// KV head - the q_len tokens times the G = H_q/H_kv heads of its group, R = q_len*G <= 128 rows, padded to
// Rp = multiple of 16 - are packed as row r = t*G + g.  A tile is 128 keys (two pages).  The keys go on the M
// dimension of the MMA and the packed rows on N, so no tensor-core or softmax lane is spent on padding rows:
//     S^T [128 keys x Rp] = K_tile [128 x D] . Q^T        (A = K pages as TMA wrote them, B = Q in shared memory)
//     O^T [D x Rp]       += V_tile^T [D x 128] . P^T       (A = V pages as TMA wrote them, read M-major; B = P^T)
// One tcgen05.mma costs about 60 cycles whatever its size below N = 128, so the tile is shaped to need few of
// them: 8 + 8 per 64 KB of K/V.  A softmax thread owns one key and walks the Rp rows; its partial row sums
// accumulate in tensor memory next to S^T and are reduced over the keys once per segment.  The only cross-thread
// traffic of a tile is one OR-reduction: "did any score rise more than 2^8 above the row's reference maximum?".
// If not (the common case after the first tile) the stale reference is kept; otherwise the exact row maxima are
// recomputed and O^T and the partial sums are rescaled in tensor memory.
//
// Work split (persistent CTAs, one per SM).  Three modes, chosen on the host from the shape:
//  * cluster: one thread-block cluster (2, 4, 8 or 16 CTAs) per unit.  The CTAs of a cluster split the unit's
//    tiles evenly, leave their partial (m, l, O) in their own shared memory, and after a cluster barrier every CTA
//    merges a share of the rows by reading its peers' partials through distributed shared memory.  One launch, no
//    trip through global memory; used whenever clusters of that size keep enough SMs busy.
//  * unit-aligned split + combine kernel: with no more (sequence, kv head) units than CTAs, every unit gets a
//    whole number of CTAs in proportion to its tile count (at least one; largest-remainder rounding) and each CTA
//    streams one contiguous range of its unit's tiles: one "segment" per CTA, no pipeline drain in the middle.
//  * flat split + combine kernel: with more units than CTAs the tiles of all units form one flat list cut into
//    gridDim.x equal ranges, and a CTA walks its range segment by segment.
// Without clusters a segment yields either the final output (it covers the whole unit) or a partial
// (m, l, O) in a workspace slot; CTA 0 records per unit the first slot and the number of contributors, and the
// combine kernel merges them.
//
// CTA = 10 warps: warp 0 TMA producer: ring of 2-page slots, alternately K and V of a tile, full/empty mbarriers;
//                        a K slot is released as soon as QK^T has read it
//                 warp 1 tcgen05.mma issuer and TMEM owner; S^T double buffered, PV trails QK by one tile
//                 warps 2-9 softmax / rescale / epilogue: warps w and w+4 share a quarter of the tensor-memory
//                        lanes and split the packed rows in alternating groups of 16
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA records HIPPO_ERR_TIMEOUT in the
// workspace header, drains its own copies, frees its tensor memory and exits.
//
// Several layers in one launch (hippo_verify_attention_layers).  The same CTAs walk the layers one after the other:
// barriers, tensor memory and the partition are set up once, the producer runs ahead into the next layer's tiles while
// the softmax threads finish the current layer, and no kernel boundary or second kernel separates two layers.  A layer's
// partials go to one of kLayerRing slot sets in the workspace; an eleventh warp per CTA publishes them (fence + one
// atomic per unit) and merges its share of the layer's output rows as soon as the contributing CTAs have published
// theirs, which happens while everybody streams the next layer.  From layer to layer the CTAs trade ranges (CTA c takes
// the range of virtual CTA (c + layer * stride) mod grid), so that every CTA sees the average range length.
#include <cuda.h>
#include <math.h>
#include <stddef.h>
#include <string.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace hippo {

constexpr int kTcThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr int kBlockN = 128;           // keys per tile = two KV pages
constexpr int kMaxRows = 128;          // packed rows (padded)
constexpr int kMaxSlots = 12;
constexpr int kTcMaxBatch = 256;       // per-sequence tile prefix lives in shared memory
constexpr int kMaxAlignedUnits = 256;  // unit-aligned split: per-unit tables live in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;              // lazy rescale: only when a score exceeds the reference by > 2^8
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s
constexpr int kLayersPerLaunch = 64;   // tensor maps and pointers of the layers travel as kernel parameters
constexpr int kLayerRing = 6;          // slot sets for the partials of consecutive layers
constexpr int kMergeWarp = kTcThreads / 32;   // the extra warp of the multi-layer kernel

// Per-layer operands.  NL = 1: the single-layer calls.
template <int NL>
struct LayerSetT {
    CUtensorMap k[NL], v[NL];
    const void *q[NL];
    void *out[NL];
    float *lse[NL];
};
// Cross-CTA bookkeeping of the multi-layer kernel (device memory, zeroed before the launch).
struct MultiCtl {
    int *done;            // [layers][units]: partials published
    int *merged;          // [layers]: output rows finished by the merge warps
    int n_layers;         // layers of this launch
    int layer0;           // index of its first layer in done / merged
    int rot;              // range rotation per layer, coprime with the grid
    long long ring_floats;   // floats per slot set
};

// ---- named barriers of the 256 softmax threads ----------------------------------------------------------------------
__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool softmax_bar_or(bool pred) {
    uint32_t out;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(out) : "r"((uint32_t)pred) : "memory");
    return out != 0;
}

// ---- work partition (shared by the main and the combine kernel) ---------------------------------------------------
struct Partition {
    long long total;   // tiles over all units
    int grid;          // CTAs
    __device__ __forceinline__ long long start_of(int c) const { return (long long)c * total / grid; }
    __device__ __forceinline__ int cta_of(long long t) const { return (int)(((t + 1) * grid - 1) / total); }
};

// The work of a sequence is counted in 64-key pages: CTA ranges begin and end on page boundaries, and a CTA forms its
// 128-key tiles from consecutive pairs of its pages (the last tile of a range may hold a single page).
__device__ __forceinline__ int seq_tiles(int kvl, int q_len) { return kvl < q_len ? 0 : (kvl + kPageSize - 1) / kPageSize; }

// Unit-aligned split worked out by one warp (at most 32 units): every unit with tiles gets one CTA, the others go to
// the units in proportion to their tile counts (largest remainders first, lower unit first on ties), never more CTAs
// than tiles.  Lane u holds unit u: my_tiles = its tiles (0 beyond the last unit), total = tiles of all units.
// Returns (first CTA, CTAs) of the lane's unit; all_ctas = CTAs in use.  The main kernel and the combine kernel both
// call this, so they cannot disagree.
__device__ __forceinline__ int2 aligned_split_warp(int lane, int U, int grid, int my_tiles, long long total, int &all_ctas) {
    const bool live = my_tiles > 0;
    const int spare = grid - __popc(__ballot_sync(0xffffffffu, live));
    int base = 0;
    uint32_t r = 0;
    if (live) {
        const long long num = (long long)spare * my_tiles;
        base = (int)(num / total);
        r = (uint32_t)(num % total);
    }
    int sum_base = base;
#pragma unroll
    for (int o = 16; o; o >>= 1) sum_base += __shfl_xor_sync(0xffffffffu, sum_base, o);
    const int leftover = spare - sum_base;
    int rank = 0;
    for (int v = 0; v < U; ++v) {
        const uint32_t rv = __shfl_sync(0xffffffffu, r, v);
        const int lv = __shfl_sync(0xffffffffu, (int)live, v);
        rank += (lv && (rv > r || (rv == r && v < lane))) ? 1 : 0;
    }
    const int n = live ? min(my_tiles, 1 + base + (rank < leftover ? 1 : 0)) : 0;
    int cinc = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, cinc, o); if (lane >= o) cinc += v; }
    all_ctas = __shfl_sync(0xffffffffu, cinc, 31);
    return make_int2(cinc - n, n);
}

// ---- shared control block -------------------------------------------------------------------------------------------
struct TcShared {
    unsigned long long full[kMaxSlots], empty[kMaxSlots], s_full[2], s_free[2], p_full[2], pv_done[2], q_full, q_free, drain;
    long long wait_limit;       // the header's wait limit (0: the built-in one), read once
    uint32_t tmem_base;
    volatile int abort;
    int seg_done;               // multi-layer kernel: segments whose partial is in memory (softmax threads -> merge warp)
    int slots_free_upto;        // multi-layer kernel: partials of layers < this may be written (merge warp -> softmax threads)
    // the per-row tables are read four entries at a time
    alignas(16) float mneg[kMaxRows];       // minus the reference maximum of each packed row, log2 domain (+inf: nothing seen yet)
    alignas(16) float fscale[kMaxRows];     // rescale factors of a slow path; row sums in the epilogue
    alignas(16) float wpart[4][kMaxRows];   // per-warp tile maxima (slow path) / per-warp row sums (epilogue)
    alignas(16) int limit[kMaxRows];        // last visible key of each packed row
    alignas(16) int rowoff[kMaxRows];       // (b*q_len + t)*H_q + h of each packed row, -1 for padding rows
    int tile_prefix[kTcMaxBatch + 1];  // only [0, batch] used
    int kvlen[kTcMaxBatch];            // kv_len, read once
    // unit-aligned split
    int sum_base;
    uint32_t rem[kMaxAlignedUnits];
    int n_cta[kMaxAlignedUnits];
    int cta_base[kMaxAlignedUnits + 1];
};

// The polling part of a bounded wait, kept out of line: it is entered only when the barrier is not yet complete and
// would otherwise be replicated at some twenty call sites.  The limit is 2 s unless the workspace header carries another
// one (a debugging aid, read once per CTA into shared memory): then the waits poll without suspending and look at the
// clock after every poll, so that the limit is honoured to a fraction of a microsecond.  A drain wait (`draining`) keeps
// the 2 s limit whatever the header says and does not give up because somebody else did: it guards the exit of the CTA,
// not its progress.
__device__ __noinline__ bool wait_slow(TcShared *sh, WsHeader *hdr, uint32_t b, uint32_t parity, int site, bool draining) {
    const unsigned long long t0 = global_ns();
    const long long user = draining ? 0 : sh->wait_limit;
    const unsigned long long limit = user > 0 ? (unsigned long long)user : kWaitLimitNs;
    for (uint32_t i = 1;; ++i) {
        if (user > 0 ? mbar_test_wait(b, parity) : mbar_try_wait(b, parity)) return true;
        if (user > 0 || (i & 31) == 0) {
            if (!draining && sh->abort) return false;
            if (global_ns() - t0 > limit) {
                sh->abort = 1;
                if (atomicCAS(&hdr->status, 0, (int)HIPPO_ERR_TIMEOUT) == 0) hdr->where = site;
                return false;
            }
        }
    }
}

struct Waiter {
    TcShared *sh;
    WsHeader *hdr;
    bool user_limit;    // the header carries a wait limit: poll without suspending
    __device__ __forceinline__ bool wait(unsigned long long *bar, uint32_t parity, int site) const {
        const uint32_t b = smem_u32(bar);
        if (user_limit ? mbar_test_wait(b, parity) : mbar_try_wait(b, parity)) return true;
        return wait_slow(sh, hdr, b, parity, site, false);
    }
    __device__ __forceinline__ bool wait_drain(unsigned long long *bar, uint32_t parity, int site) const {
        const uint32_t b = smem_u32(bar);
        if (mbar_try_wait(b, parity)) return true;
        return wait_slow(sh, hdr, b, parity, site, true);
    }
    // Bounded wait until a flag in this CTA's shared memory, written by another warp, exceeds `than`.
    __device__ __forceinline__ bool wait_shared_gt(const int *flag, int than, int site) const {
        if (ld_acquire_cta_shared(flag) > than) return true;
        const unsigned long long t0 = global_ns();
        const long long user = sh->wait_limit;
        const unsigned long long limit = user > 0 ? (unsigned long long)user : kWaitLimitNs;
        for (;;) {
            __nanosleep(40);
            if (ld_acquire_cta_shared(flag) > than) return true;
            if (sh->abort) return false;
            if (global_ns() - t0 > limit) {
                sh->abort = 1;
                if (atomicCAS(&hdr->status, 0, (int)HIPPO_ERR_TIMEOUT) == 0) hdr->where = site;
                return false;
            }
        }
    }
    // Bounded wait until *counter (device memory, written by other CTAs) reaches `want`.  Gives up at once when any
    // CTA has reported a time-out, so that one failure does not cost every other CTA its own limit.
    __device__ __forceinline__ bool wait_counter(const int *counter, int want, int site) const {
        if (ld_acquire_gpu(counter) >= want) return true;
        const unsigned long long t0 = global_ns();
        const long long user = sh->wait_limit;
        const unsigned long long limit = user > 0 ? (unsigned long long)user : kWaitLimitNs;
        for (;;) {
            __nanosleep(100);
            if (ld_acquire_gpu(counter) >= want) return true;
            if (sh->abort || *reinterpret_cast<const volatile int *>(&hdr->status) != 0) { sh->abort = 1; return false; }
            if (global_ns() - t0 > limit) {
                sh->abort = 1;
                if (atomicCAS(&hdr->status, 0, (int)HIPPO_ERR_TIMEOUT) == 0) hdr->where = site;
                return false;
            }
        }
    }
};

static_assert(offsetof(TcShared, mneg) % 16 == 0 && offsetof(TcShared, limit) % 16 == 0 && offsetof(TcShared, rowoff) % 16 == 0 &&
              offsetof(TcShared, fscale) % 16 == 0, "row tables are read as 16-byte vectors");

struct TcSmemPlan { int q_bytes, p_bytes, fixed, slots, total; };
// Shared-memory carve-up: [ring of 2-page slots | Q | P^T x2 | control], ring depth = whatever fits.
static TcSmemPlan tc_smem_plan(int D, int Rp) {
    TcSmemPlan s;
    s.q_bytes = Rp * D * 2;
    s.p_bytes = Rp * kBlockN * 2;
    s.fixed = s.q_bytes + 2 * s.p_bytes + (int)((sizeof(TcShared) + 127) & ~(size_t)127);
    const int slot = kBlockN * D * 2;
    int n = (227 * 1024 - 1024 - s.fixed) / slot;
    s.slots = n > kMaxSlots ? kMaxSlots : n;
    s.total = 1024 + s.fixed + s.slots * slot;
    return s;
}

template <int D, int NL>
__global__ void __launch_bounds__(NL == 1 ? kTcThreads : kTcThreads + 32, 1)
attn_tc_kernel(const AttnParams p, const __grid_constant__ LayerSetT<NL> set, const MultiCtl mc,
               const int Rp, const int n_slots, const int tmem_cols, const int cluster_size, const int spare_cols) {
    constexpr bool kMulti = NL > 1;
    constexpr int kThreads = kMulti ? kTcThreads + 32 : kTcThreads;
    constexpr int kChunks = D / 64;                     // 64-column (128-byte) swizzle chunks per row
    constexpr int kPageBytes = kPageSize * D * 2;       // K or V of one page and head
    constexpr int kSlotBytes = 2 * kPageBytes;          // K or V of one tile
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *ring = base;                                   // [n_slots] K: [chunk][page][64 rows][128 B]; V: [page][chunk][64][128 B]
    uint8_t *q_s = ring + n_slots * kSlotBytes;             // [kChunks][Rp rows][128 B], 128B swizzle
    uint8_t *p_s = q_s + Rp * D * 2;                        // [2][Rp/8][128 keys][8 rows] bf16 (no swizzle, row-contiguous)
    TcShared *sh = (TcShared *)(p_s + 2 * Rp * kBlockN * 2);
    const int p_bytes = Rp * kBlockN * 2;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = p.rows, G = p.group, Hkv = p.n_kv_heads, B = p.batch;
    const int n_layers = kMulti ? mc.n_layers : 1;
    // Launched with programmatic stream serialization: the CTAs may be scheduled while the previous kernel of the
    // stream drains.  Barriers and tensor memory are set up meanwhile; global memory is not touched before that
    // kernel has completed (griddepcontrol.wait below).

    // ---- set-up: barriers, tile prefix, CTA split, tensor memory
    const int U = B * Hkv;
    const bool clustered = cluster_size > 1;                  // one cluster per unit, merge through shared memory
    const bool aligned = !clustered && U <= (int)gridDim.x && U <= kMaxAlignedUnits;
    const bool small_problem = U <= 32;                       // tile prefix and CTA split by warp 0 alone, no block barriers
    {
        // one barrier per thread of warps 1..: [0, n_slots) full, [n_slots, 2 n_slots) empty, then the fixed ones
        const int nb = 2 * n_slots, t = tid - 32;
        if (t < 0) {}
        else if (t < nb) mbar_init(smem_u32(t < n_slots ? &sh->full[t] : &sh->empty[t - n_slots]), 1);
        else if (t < nb + 2) mbar_init(smem_u32(&sh->s_full[t - nb]), 1);
        else if (t < nb + 4) mbar_init(smem_u32(&sh->s_free[t - nb - 2]), kSoftmaxThreads);
        else if (t < nb + 6) mbar_init(smem_u32(&sh->p_full[t - nb - 4]), kSoftmaxThreads);
        else if (t < nb + 8) mbar_init(smem_u32(&sh->pv_done[t - nb - 6]), 1);
        else if (t == nb + 8) mbar_init(smem_u32(&sh->q_full), kSoftmaxThreads);
        else if (t == nb + 9) mbar_init(smem_u32(&sh->q_free), 1);
        else if (t == nb + 10) mbar_init(smem_u32(&sh->drain), 1);
        else if (t == nb + 11) { sh->abort = 0; sh->sum_base = 0; sh->seg_done = 0; sh->slots_free_upto = kLayerRing; }
        if (tid == 32) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&set.k[0]) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&set.v[0]) : "memory");
        }
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (tid == kThreads - 1) sh->wait_limit = p.header->wait_limit_ns;
        if (!small_problem) {
            // tiles per sequence; the exclusive prefix follows the barrier
            for (int b = tid; b < B; b += kThreads) {
                const int kvl = p.kv_len ? p.kv_len[b] : p.max_kv_len;
                sh->kvlen[b] = kvl;
                sh->tile_prefix[b + 1] = seq_tiles(kvl, p.q_len);
            }
        } else if (warp == 0) {
            // lane b: sequence b; lane u: unit u.  Everything by shuffles.
            const int kvl = lane < B ? (p.kv_len ? p.kv_len[lane] : p.max_kv_len) : 0;
            const int nt = lane < B ? seq_tiles(kvl, p.q_len) : 0;
            int incl = nt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
            if (lane < B) { sh->kvlen[lane] = kvl; sh->tile_prefix[lane + 1] = incl; }
            if (lane == 0) sh->tile_prefix[0] = 0;
            if (aligned) {
                // CTAs per unit: one each, the others in proportion to the tile counts (largest remainders first)
                const long long total = (long long)__shfl_sync(0xffffffffu, incl, 31) * Hkv;
                const int t_src = __shfl_sync(0xffffffffu, nt, lane < U ? lane / Hkv : 0);
                const int my_tiles = lane < U ? t_src : 0;
                int all;
                const int2 mine = aligned_split_warp(lane, U, (int)gridDim.x, my_tiles, total, all);
                if (lane < U) { sh->n_cta[lane] = mine.y; sh->cta_base[lane] = mine.x; }
                if (lane == 0) sh->cta_base[U] = all;
            }
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    if (!small_problem) {
        if (tid == 0) {
            int acc = 0;
            for (int b = 0; b < B; ++b) { const int n = sh->tile_prefix[b + 1]; sh->tile_prefix[b] = acc; acc += n; }
            sh->tile_prefix[B] = acc;
        }
        __syncthreads();
    }
    tc_fence_after();
    const Waiter W{sh, p.header, sh->wait_limit > 0};
    const uint32_t tmem = sh->tmem_base;
    const uint32_t col_s = 0, col_o = 2 * Rp, col_l = 3 * Rp;   // S^T[0] | S^T[1] | O^T | partial row sums, Rp columns each

    Partition part;
    part.total = (long long)sh->tile_prefix[B] * Hkv;
    part.grid = gridDim.x;
    int2 *unit_info = reinterpret_cast<int2 *>(p.counters);   // per unit: first slot, number of contributing CTAs
    if (aligned && !small_problem) {
        // CTAs per unit: one each, the others in proportion to the tile counts (largest remainders first)
        const int my_tiles = tid < U ? sh->tile_prefix[tid / Hkv + 1] - sh->tile_prefix[tid / Hkv] : 0;
        const bool live = my_tiles > 0;
        const int n_live = __syncthreads_count(live);
        const int spare = (int)gridDim.x - n_live;
        int my_base = 0;
        if (tid < U) {
            uint32_t r = 0;
            if (live) {
                const long long num = (long long)spare * my_tiles;
                my_base = (int)(num / part.total);
                r = (uint32_t)(num % part.total);
                if (my_base) atomicAdd(&sh->sum_base, my_base);
            }
            sh->rem[tid] = r;
            sh->n_cta[tid] = live ? 1 : 0;
        }
        __syncthreads();
        if (tid < U && live) {
            const int leftover = spare - sh->sum_base;
            const uint32_t r = sh->rem[tid];
            int rank = 0;
            for (int v = 0; v < U; ++v) rank += (sh->n_cta[v] && (sh->rem[v] > r || (sh->rem[v] == r && v < tid))) ? 1 : 0;
            sh->n_cta[tid] = min(my_tiles, 1 + my_base + (rank < leftover ? 1 : 0));
        }
        __syncthreads();
        if (tid == 0) {
            int acc = 0;
            for (int u = 0; u < U; ++u) { sh->cta_base[u] = acc; acc += sh->n_cta[u]; }
            sh->cta_base[U] = acc;
        }
        __syncthreads();
    }
    // Range [t_begin, t_end) of the flat tile list that CTA number c streams.  In the single-layer kernel c is the CTA's
    // own index; the multi-layer kernel hands CTA x the range of c = (x + layer * rot) mod grid in layer `layer`.
    auto range_of = [&](int c, long long &t_begin, long long &t_end) {
        t_begin = t_end = 0;
        if (clustered) {
            const int u = c / cluster_size, i = c % cluster_size;
            const int b = u / Hkv, hk = u % Hkv;
            const long long T = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
            const long long unit_start = (long long)sh->tile_prefix[b] * Hkv + hk * T;
            t_begin = unit_start + T * i / cluster_size;
            t_end = unit_start + T * (i + 1) / cluster_size;
        } else if (aligned) {
            if (c < sh->cta_base[U]) {
                int lo = 0, hi = U;   // largest u with cta_base[u] <= c
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (sh->cta_base[mid] <= c) lo = mid; else hi = mid;
                }
                while (sh->n_cta[lo] == 0) ++lo;   // units without tiles share their neighbour's base
                const int b = lo / Hkv, hk = lo % Hkv;
                const long long T = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                const long long unit_start = (long long)sh->tile_prefix[b] * Hkv + hk * T;
                const int i = c - sh->cta_base[lo], nc = sh->n_cta[lo];
                t_begin = unit_start + T * i / nc;
                t_end = unit_start + T * (i + 1) / nc;
            }
        } else if (part.total > 0) {
            t_begin = part.start_of(c);
            t_end = part.start_of(c + 1);
        }
    };
    // (first slot, number of contributing CTAs) of a unit, as the combine kernel and the merge warp need it
    auto unit_slots = [&](int u) -> int2 {
        if (aligned) return make_int2(sh->cta_base[u], sh->n_cta[u]);
        const int b = u / Hkv, hk = u % Hkv;
        const long long T = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
        if (T <= 0) return make_int2(0, 0);
        const long long u0 = (long long)sh->tile_prefix[b] * Hkv + hk * T;
        const int c0 = part.cta_of(u0), c1 = part.cta_of(u0 + T - 1);
        return make_int2(u + c0, c1 - c0 + 1);     // slot index = unit + cta
    };
    if (!kMulti && !clustered && blockIdx.x == 0)
        for (int u = tid; u < U; u += kThreads) unit_info[u] = unit_slots(u);
    const int slot_bias = aligned ? 0 : 1;   // slot = CTA number (+ unit in the flat split)
    auto cta_of_layer = [&](int layer) -> int {
        return kMulti ? (int)(((long long)blockIdx.x + (long long)layer * mc.rot) % (long long)gridDim.x) : (int)blockIdx.x;
    };
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel's CTAs may be scheduled

    // Every role walks the same list of segments.  A segment = (b, hk, first tile, tile count) taken from the flat
    // range [t_begin, t_end); order is unit-major: all tiles of (b, hk=0), then (b, hk=1), ...
    auto locate = [&](long long t, int &b, int &hk, int &tile) {
        int lo = 0, hi = B;  // largest b with Hkv * prefix[b] <= t
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if ((long long)sh->tile_prefix[mid] * Hkv <= t) lo = mid; else hi = mid;
        }
        b = lo;
        while (b + 1 < B && (long long)sh->tile_prefix[b + 1] * Hkv <= t) ++b;   // skip sequences without tiles
        const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
        const long long off = t - (long long)sh->tile_prefix[b] * Hkv;
        hk = (int)(off / nt);
        tile = (int)(off % nt);
    };

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            RingPos rp{0, 0};
            uint32_t issued = 0;
            bool ok = true;
            // verification reads K and V once per call: stream them through L2; the draft's pruned cache is read again by every call
            const uint64_t stream_pol = p.kv_resident ? l2_policy_evict_last() : l2_policy_evict_first();
            for (int layer = 0; layer < n_layers && ok; ++layer) {
                const CUtensorMap *k_map = &set.k[layer], *v_map = &set.v[layer];
                if (kMulti && layer + 1 < n_layers) {
                    asm volatile("prefetch.tensormap [%0];" ::"l"(&set.k[layer + 1]) : "memory");
                    asm volatile("prefetch.tensormap [%0];" ::"l"(&set.v[layer + 1]) : "memory");
                }
                long long t, t_end;
                range_of(cta_of_layer(layer), t, t_end);
                while (ok && t < t_end) {
                    int b, hk, tile;
                    locate(t, b, hk, tile);
                    const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                    const int n = (int)min((long long)(nt - tile), t_end - t);
                    if (kMulti) {
                        // This thread runs a few tiles ahead of the softmax threads, which fetch a segment's Q rows only when
                        // they get there: ask for the rows now, so that they are an L2 hit by then (per query position the
                        // G heads of a KV head are contiguous).
                        const char *qb = (const char *)set.q[layer];
                        for (int tq = 0; tq < p.q_len; ++tq) {
                            const char *rows = qb + ((size_t)(b * p.q_len + tq) * p.n_q_heads + (size_t)hk * G) * (D * 2);
                            for (int off = 0; off < G * D * 2; off += 128)
                                asm volatile("prefetch.global.L2 [%0];" ::"l"(rows + off) : "memory");
                        }
                    }
                    for (int i = 0; i < n && ok; i += 2) {
                        const int pg0 = tile + i;
                        const int np = min(2, n - i);                    // the last tile of a range may hold one page
                        int row[2];
                        for (int q = 0; q < np; ++q)
                            row[q] = (page_of(p.page_table, p.max_pages_per_seq, b, pg0 + q) * Hkv + hk) * kPageSize;
                        // K of the tile, then V of the tile
                        for (int kv = 0; kv < 2 && ok; ++kv, rp.advance(n_slots), ++issued) {
                            ok = W.wait(&sh->empty[rp.slot], rp.phase ^ 1, 1);
                            if (!ok) break;
                            const uint32_t bar = smem_u32(&sh->full[rp.slot]);
                            mbar_expect_tx(bar, np * kPageBytes);
                            const uint32_t dst = smem_u32(ring + rp.slot * kSlotBytes);
                            for (int q = 0; q < np; ++q) {
#pragma unroll
                                for (int c = 0; c < kChunks; ++c) {
                                    if (kv == 0) tma_load_2d_hint(dst + c * (2 * 8192) + q * 8192, k_map, c * 64, row[q], bar, stream_pol);
                                    else tma_load_2d_hint(dst + q * kPageBytes + c * 8192, v_map, c * 64, row[q], bar, stream_pol);
                                }
                            }
                        }
                    }
                    t += n;
                }
            }
            // drain: every load that was issued must have landed before the CTA may exit
            const int back = issued < (uint32_t)n_slots ? (int)issued : n_slots;
            for (int k = 0; k < back; ++k) {
                // step the ring position back by one
                if (rp.slot == 0) { rp.slot = n_slots - 1; rp.phase ^= 1; } else --rp.slot;
                W.wait_drain(&sh->full[rp.slot], rp.phase, 2);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            const uint32_t idesc_qk = instr_desc(kBlockN, Rp, false, false);   // S^T: A = K (K-major), B = Q (K-major)
            const uint32_t idesc_pv = instr_desc(D, Rp, true, true);           // O^T: A = V (M-major), B = P^T (N-major)
            // descriptors of the operands at offset 0; an operand at byte offset x adds x >> 4 to the address field
            const uint64_t kdesc0 = smem_desc(smem_u32(ring), 16, 1024, 2);
            const uint64_t vdesc0 = smem_desc(smem_u32(ring), 8192, 1024, 2);
            const uint64_t qdesc0 = smem_desc(smem_u32(q_s), 16, 1024, 2);
            const uint64_t pdesc0 = smem_desc(smem_u32(p_s), 128, kBlockN * 16, 0);
            const uint32_t q_chunk16 = (uint32_t)(Rp * 128) >> 4;
            RingPos rk{0, 0};            // slot of the next tile's K
            RingPos rv{1 % n_slots, (uint32_t)(n_slots == 1)};   // slot of the next PV's V (K and V alternate in the ring)
            uint32_t it = 0, seg = 0;
            bool ok = true;
            // O^T += V_k^T P_k^T for the CTA's tile number k
            auto issue_pv = [&](uint32_t k, bool first_of_segment) -> bool {
                const int j = k & 1;
                if (!W.wait(&sh->full[rv.slot], rv.phase, 15)) return false;
                if (!W.wait(&sh->p_full[j], (k >> 1) & 1, 3)) return false;
                tc_fence_after();
                const uint64_t pd = pdesc0 + (uint64_t)((uint32_t)(j * p_bytes) >> 4);
                const uint64_t vd = vdesc0 + (uint64_t)((uint32_t)(rv.slot * kSlotBytes) >> 4);
#pragma unroll
                for (int ks = 0; ks < kBlockN / 16; ++ks)
                    tc_mma(tmem + col_o, vd + (uint64_t)(((ks >> 2) * kPageBytes + (ks & 3) * 2048) >> 4), pd + (uint64_t)((ks * 256) >> 4),
                           idesc_pv, (first_of_segment && ks == 0) ? 0u : 1u);
                tc_commit(smem_u32(&sh->pv_done[j]));
                tc_commit(smem_u32(&sh->empty[rv.slot]));
                rv.advance(n_slots); rv.advance(n_slots);
                return true;
            };
            for (int layer = 0; layer < n_layers && ok; ++layer) {
                long long t, t_end;
                range_of(cta_of_layer(layer), t, t_end);
                while (ok && t < t_end) {
                    int b, hk, tile;
                    locate(t, b, hk, tile);
                    const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                    const int n = (int)min((long long)(nt - tile), t_end - t);
                    ok = W.wait(&sh->q_full, seg & 1, 4);  // Q of this segment is in shared memory
                    const uint32_t it0 = it;
                    for (int i = 0; i < n && ok; i += 2, ++it) {
                        const int j = it & 1;
                        ok = W.wait(&sh->full[rk.slot], rk.phase, 5);
                        if (!ok) break;
                        // S^T buffer j was last read by the softmax of tile it-2
                        if (it >= 2) { ok = W.wait(&sh->s_free[j], ((it - 2) >> 1) & 1, 14); if (!ok) break; }
                        tc_fence_after();
                        const uint64_t kd = kdesc0 + (uint64_t)((uint32_t)(rk.slot * kSlotBytes) >> 4);
#pragma unroll
                        for (int c = 0; c < kChunks; ++c)
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                tc_mma(tmem + col_s + j * Rp, kd + (uint64_t)((c * (2 * 8192) + ks * 32) >> 4),
                                       qdesc0 + (uint64_t)(c * q_chunk16 + ks * 2), idesc_qk, (c | ks) ? 1u : 0u);
                        tc_commit(smem_u32(&sh->s_full[j]));
                        tc_commit(smem_u32(&sh->empty[rk.slot]));            // K is not needed again
                        if (i + 2 >= n) tc_commit(smem_u32(&sh->q_free));    // last QK of the segment: Q may be replaced
                        rk.advance(n_slots); rk.advance(n_slots);
                        if (i >= 2) ok = issue_pv(it - 1, it - 1 == it0);    // PV trails QK by one tile
                    }
                    if (ok && n >= 1) ok = issue_pv(it - 1, it - 1 == it0);
                    t += n;
                    ++seg;
                }
            }
            // all tensor-core work of this CTA must be complete before tensor memory is released
            tc_commit(smem_u32(&sh->drain));
            W.wait_drain(&sh->drain, 0, 6);
        }
    } else if (kMulti && warp == kMergeWarp) {
        // ================= merge warp (multi-layer kernel) =================
        // Per layer: publish this CTA's partials as the softmax threads finish them, release the slot set of the next
        // layer, wait until every CTA has published the layer, merge rows blockIdx.x, blockIdx.x + gridDim.x, ...
        constexpr int V = D / 32;   // output columns per lane
        constexpr int kMergeBatch = 24;   // partials whose loads are in flight together
        const int total_rows = B * p.q_len * p.n_q_heads;
        const size_t slot_floats = slot_float_count(R, D);
        const int Rpad = slot_rows_padded(R);
        int published = 0;
        bool ok = true;
        for (int layer = 0; layer < n_layers && ok; ++layer) {
            const int gl = mc.layer0 + layer;
            int *done = mc.done + (size_t)gl * U;
            long long t, t_end;
            range_of(cta_of_layer(layer), t, t_end);
            while (ok && t < t_end) {
                int b, hk, tile;
                locate(t, b, hk, tile);
                const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                const int n = (int)min((long long)(nt - tile), t_end - t);
                if (!(tile == 0 && n == nt)) {   // a segment that covers its whole unit writes the output itself
                    ok = W.wait_shared_gt(&sh->seg_done, published, 20);
                    ++published;
                    if (ok && lane == 0) { __threadfence(); red_release_gpu_add(&done[b * Hkv + hk], 1); }
                }
                t += n;
            }
            if (ok && layer + 1 < n_layers && layer + 1 >= kLayerRing) {
                // layer + 1 reuses the slot set of layer + 1 - kLayerRing: all rows of that layer must have been merged
                ok = W.wait_counter(mc.merged + (gl + 1 - kLayerRing), total_rows, 21);
                __syncwarp();
                if (ok && lane == 0) st_release_cta_shared(&sh->slots_free_upto, layer + 2);
            }
            for (int u = lane; u < U && ok; u += 32) {
                const int n = unit_slots(u).y;
                if (n > 1) ok = W.wait_counter(&done[u], n, 22);
            }
            ok = __all_sync(0xffffffffu, ok);
            __syncwarp();   // every lane's acquire is ordered before every lane's loads of the partials
            if (!ok) break;
            const float *slots = p.partials + (long long)(layer % kLayerRing) * mc.ring_floats;
            __nv_bfloat16 *og = (__nv_bfloat16 *)set.out[layer];
            float *lse_g = set.lse[layer];
            int handled = 0;
            for (int row = blockIdx.x; row < total_rows; row += gridDim.x, ++handled) {
                const int h = row % p.n_q_heads, tq = (row / p.n_q_heads) % p.q_len, b = row / (p.n_q_heads * p.q_len);
                const int hk = h / G, r = tq * G + (h % G);
                const int2 info = unit_slots(b * Hkv + hk);
                const int n = info.y;
                __nv_bfloat16 *o = og + (size_t)row * D + lane * V;
                if (n == 1) continue;
                // All loads of a batch of kMergeBatch partials are issued before anything is used: lane j fetches the
                // (m, l) of partial j, every lane its V output columns of all of them.  Under a saturated memory system a
                // round trip to L2 takes microseconds, and this warp has to keep pace with the layers.
                float M = -INFINITY, L = 0.f, acc[V];   // L: this lane's share of the weighted sums (added up below)
#pragma unroll
                for (int x = 0; x < V; ++x) acc[x] = 0.f;
                const float *base = slots + (size_t)info.x * slot_floats;
                for (int c0 = 0; c0 < n; c0 += kMergeBatch) {
                    float mj = -INFINITY, lj = 0.f;
                    if (lane < kMergeBatch && c0 + lane < n) {
                        const float *sl = base + (size_t)(c0 + lane) * slot_floats;
                        mj = __ldcg(sl + r);
                        lj = __ldcg(sl + Rpad + r);
                    }
                    float v[kMergeBatch][V];
#pragma unroll
                    for (int j = 0; j < kMergeBatch; ++j) {
                        const float *sl = base + (size_t)min(c0 + j, n - 1) * slot_floats;   // clamped; repeats get weight 0
                        if (V == 4) {
                            const float4 t4 = __ldcg(reinterpret_cast<const float4 *>(sl + 2 * Rpad + (size_t)r * D + lane * V));
                            v[j][0] = t4.x; v[j][1] = t4.y; v[j][V - 2] = t4.z; v[j][V - 1] = t4.w;
                        } else {
                            const float2 t2 = __ldcg(reinterpret_cast<const float2 *>(sl + 2 * Rpad + (size_t)r * D + lane * V));
                            v[j][0] = t2.x; v[j][1] = t2.y;
                        }
                    }
                    const float m_new = fmaxf(M, warp_max(mj));
                    if (m_new == -INFINITY) continue;                       // nothing visible so far (uniform over the warp)
                    const float f_old = (M == -INFINITY) ? 0.f : expf(M - m_new);
                    const float w = (mj == -INFINITY) ? 0.f : expf(mj - m_new);   // 0 for lanes without a partial
                    L = L * f_old + lj * w;
#pragma unroll
                    for (int x = 0; x < V; ++x) acc[x] *= f_old;
#pragma unroll
                    for (int j = 0; j < kMergeBatch; ++j) {
                        const float wj = __shfl_sync(0xffffffffu, w, j);
#pragma unroll
                        for (int x = 0; x < V; ++x) acc[x] = fmaf(v[j][x], wj, acc[x]);
                    }
                    M = m_new;
                }
#pragma unroll
                for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
                // n == 0 (a sequence shorter than q_len is skipped) leaves L = 0: its outputs are defined as zero
                const float inv = L > 0.f ? 1.f / L : 0.f;
                if (V == 4) {
                    __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv), h1 = __floats2bfloat162_rn(acc[V - 2] * inv, acc[V - 1] * inv);
                    *reinterpret_cast<uint2 *>(o) = make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
                } else {
                    __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
                    *reinterpret_cast<uint32_t *>(o) = *reinterpret_cast<uint32_t *>(&h0);
                }
                if (lse_g && lane == 0) lse_g[row] = L > 0.f ? M + logf(L) : -INFINITY;
            }
            __syncwarp();
            if (lane == 0) { __threadfence(); red_release_gpu_add(mc.merged + gl, handled); }
        }
    } else {
        // ================= softmax / rescale / epilogue =================
        // Tensor memory: a warp reaches lanes 32*(warp%4)..+31.  S^T and the partial row sums keep key 32*q + l of
        // the tile on lane 32*q + l; O^T keeps output dimension d on lane d (D = 128) or on lane 32*(d/16) + d%16
        // (D = 64, an M = 64 accumulator).  Control flow below is uniform over the 256 threads between named
        // barriers: a failed wait is remembered in `ok` and acted upon only right after the per-tile reduction.
        const int st = tid - 64;                      // 0..255
        const int quarter = warp & 3;
        const int c_first = ((warp - 2) >> 2) * 16;   // this warp's row groups: c_first, c_first + 32, ...
        const uint32_t flip_groups = (Rp >> 4) & 1;
        const bool spare_l = spare_cols != 0;         // a second column set for the partial row sums
        int l_sel = 0;                                // which set holds the current sums
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int kk = quarter * 32 + lane;           // key inside the tile
        const bool d_active = (D == 128) || lane < 16;
        const int d = (D == 128) ? quarter * 32 + lane : quarter * 16 + lane;
        const float sl2 = p.scale * kLog2e;
        RingPos rv{1 % n_slots, (uint32_t)(n_slots == 1)};   // slot of the current tile's V
        uint32_t it = 0, seg = 0;
        bool ok = true, aborted = false;
        int n_partials = 0;   // multi-layer kernel: partials this CTA has written
        const uint64_t keep_pol = l2_policy_evict_last();
        for (int layer = 0; layer < n_layers && !aborted; ++layer) {
            const int my_cta = cta_of_layer(layer);
            long long t, t_end;
            range_of(my_cta, t, t_end);
            const __nv_bfloat16 *q_g = (const __nv_bfloat16 *)set.q[layer];
            __nv_bfloat16 *og = (__nv_bfloat16 *)set.out[layer];
            float *lse_g = set.lse[layer];
            float *slot_set = p.partials + (kMulti ? (long long)(layer % kLayerRing) * mc.ring_floats : 0ll);
            while (t < t_end) {
                int b, hk, tile;
                locate(t, b, hk, tile);
                const int nt = sh->tile_prefix[b + 1] - sh->tile_prefix[b];
                const int n = (int)min((long long)(nt - tile), t_end - t);
                const int kvl = sh->kvlen[b];
                const bool whole_unit = (tile == 0 && n == nt);
                // ---- per-segment tables and Q -> shared memory (after the previous segment's QK MMAs are done)
                if (seg > 0) ok = W.wait(&sh->q_free, (seg - 1) & 1, 7) && ok;
                if (st < Rp) {
                    if (st < R) {
                        const int tq = st / G, g = st % G;
                        sh->limit[st] = kvl - p.q_len + tq;
                        sh->rowoff[st] = (b * p.q_len + tq) * p.n_q_heads + hk * G + g;
                    } else {
                        sh->limit[st] = 0x7ffffffe;
                        sh->rowoff[st] = -1;
                    }
                    sh->mneg[st] = INFINITY;
                }
                softmax_bar_sync();
                for (int x = st; x < Rp * (D / 8); x += kSoftmaxThreads) {
                    const int r = x / (D / 8), c = x % (D / 8);
                    uint4 v = make_uint4(0, 0, 0, 0);
                    const int ro = sh->rowoff[r];
                    if (ro >= 0) v = __ldg(reinterpret_cast<const uint4 *>(q_g + (size_t)ro * D) + c);
                    *reinterpret_cast<uint4 *>(q_s + (c >> 3) * (Rp * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
                }
                fence_proxy_async();
                mbar_arrive(smem_u32(&sh->q_full));

                const uint32_t it0 = it;
                for (int i = 0; i < n; i += 2, ++it, rv.advance(n_slots), rv.advance(n_slots)) {
                    const int j = it & 1;
                    // with an odd number of 16-row groups the two warps of a quarter swap shares from tile to tile
                    const int c_tile = c_first ^ ((int)(it & flip_groups) << 4);
                    const int key0 = (tile + i) * kPageSize;
                    const int key_end = min(kvl, key0 + min(2, n - i) * kPageSize);   // first key of the tile that is not there
                    // a key that is not there compares greater than every row's limit
                    const int key = key0 + kk < key_end ? key0 + kk : 0x7fffffff;
                    const bool tail = key0 + kBlockN > kvl - p.q_len + 1 || key0 + kBlockN > key_end;  // some masking in this tile
                    const uint32_t s_addr = tmem + lane_addr + col_s + j * Rp;
                    if (key0 + kBlockN > key_end) {
                        // rows of V past the end of the sequence or of this CTA's range may hold anything (also a whole
                        // missing second page): zero them, 0 * NaN would poison O
                        ok = W.wait(&sh->full[rv.slot], rv.phase, 8) && ok;
                        uint8_t *vs = ring + rv.slot * kSlotBytes;
                        const int first_bad = key_end - key0;
                        for (int x = st; x < (kBlockN - first_bad) * kChunks * 8; x += kSoftmaxThreads) {
                            const int row = first_bad + x / (kChunks * 8), rem = x % (kChunks * 8);
                            *reinterpret_cast<uint4 *>(vs + (row >> 6) * kPageBytes + (rem >> 3) * 8192 + (row & 63) * 128 + ((rem & 7) << 4)) =
                                make_uint4(0, 0, 0, 0);
                        }
                        fence_proxy_async();
                    }
                    ok = W.wait(&sh->s_full[j], (it >> 1) & 1, 9) && ok;
                    // P^T buffer j was last read by PV of tile it-2
                    if (it >= 2) ok = W.wait(&sh->pv_done[j], ((it - 2) >> 1) & 1, 11) && ok;
                    tc_fence_after();
                    uint8_t *pk = p_s + j * p_bytes + kk * 16;
                    const bool first_tile = it == it0;
                    // P^T = 2^(s*scale*log2e - reference) as bf16, row-contiguous per key, and the partial row sums
                    // (read from column set l_src unless this is the segment's first tile, written to l_dst).  Returns the
                    // largest exponent seen among the visible scores.  Branch-free inside; the masked variant runs only
                    // for the last tiles of a sequence.
                    auto write_p = [&](uint32_t l_src, uint32_t l_dst) -> float {
                        float xmax = -INFINITY;
                        for (int c = c_tile; c < Rp; c += 32) {
                            float sv[16], lv[16];
                            tmem_ld16(s_addr + c, sv);
                            if (!first_tile) tmem_ld16(tmem + lane_addr + l_src + c, lv);
                            tmem_wait_ld();
                            uint32_t w[8];
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 mn = *reinterpret_cast<const float4 *>(&sh->mneg[c + 4 * e4]);
                                float x0 = fmaf(sv[4 * e4], sl2, mn.x), x1 = fmaf(sv[4 * e4 + 1], sl2, mn.y);
                                float x2 = fmaf(sv[4 * e4 + 2], sl2, mn.z), x3 = fmaf(sv[4 * e4 + 3], sl2, mn.w);
                                if (tail) {   // uniform over the CTA
                                    const int4 lm = *reinterpret_cast<const int4 *>(&sh->limit[c + 4 * e4]);
                                    x0 = key <= lm.x ? x0 : -INFINITY; x1 = key <= lm.y ? x1 : -INFINITY;
                                    x2 = key <= lm.z ? x2 : -INFINITY; x3 = key <= lm.w ? x3 : -INFINITY;
                                }
                                xmax = fmaxf(xmax, fmaxf(fmaxf(x0, x1), fmaxf(x2, x3)));
                                const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
                                __nv_bfloat162 h0 = __floats2bfloat162_rn(p0, p1), h1 = __floats2bfloat162_rn(p2, p3);
                                w[2 * e4] = *reinterpret_cast<uint32_t *>(&h0);
                                w[2 * e4 + 1] = *reinterpret_cast<uint32_t *>(&h1);
                                if (first_tile) { lv[4 * e4] = p0; lv[4 * e4 + 1] = p1; lv[4 * e4 + 2] = p2; lv[4 * e4 + 3] = p3; }
                                else { lv[4 * e4] += p0; lv[4 * e4 + 1] += p1; lv[4 * e4 + 2] += p2; lv[4 * e4 + 3] += p3; }
                            }
                            tmem_st16(tmem + lane_addr + l_dst + c, lv);
                            *reinterpret_cast<uint4 *>(pk + (c >> 3) * (kBlockN * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
                            *reinterpret_cast<uint4 *>(pk + ((c >> 3) + 1) * (kBlockN * 16)) = make_uint4(w[4], w[5], w[6], w[7]);
                        }
                        return xmax;
                    };
                    // ---- does any visible score exceed its row's reference by more than the threshold?
                    // With a spare column set for the row sums the answer comes out of the P^T pass itself, run on the
                    // stale references: if nothing grew (the common case) the tile is done after one sweep over S^T;
                    // otherwise the sweep is repeated below with the new references.  Without the spare set a cheaper
                    // sweep (maxima only) runs first.  The first tile of a segment always takes the slow path.
                    const uint32_t l_cur = col_l + l_sel * Rp, l_alt = spare_l ? col_l + (l_sel ^ 1) * Rp : l_cur;
                    float excess = NAN;
                    if (spare_l) {
                        if (!first_tile) {
                            excess = write_p(l_cur, l_alt);
                            tmem_wait_st();
                        }
                    } else if (!tail) {
                        excess = -INFINITY;
                        for (int c = c_tile; c < Rp; c += 32) {
                            float sv[16];
                            tmem_ld16(s_addr + c, sv);
                            tmem_wait_ld();
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 mn = *reinterpret_cast<const float4 *>(&sh->mneg[c + 4 * e4]);
                                excess = fmaxf(excess, fmaxf(fmaxf(fmaf(sv[4 * e4], sl2, mn.x), fmaf(sv[4 * e4 + 1], sl2, mn.y)),
                                                             fmaxf(fmaf(sv[4 * e4 + 2], sl2, mn.z), fmaf(sv[4 * e4 + 3], sl2, mn.w))));
                            }
                        }
                    } else {
                        excess = -INFINITY;
                        for (int c = c_tile; c < Rp; c += 32) {
                            float sv[16];
                            tmem_ld16(s_addr + c, sv);
                            tmem_wait_ld();
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 mn = *reinterpret_cast<const float4 *>(&sh->mneg[c + 4 * e4]);
                                const int4 lm = *reinterpret_cast<const int4 *>(&sh->limit[c + 4 * e4]);
                                const float x0 = fmaf(sv[4 * e4], sl2, mn.x), x1 = fmaf(sv[4 * e4 + 1], sl2, mn.y);
                                const float x2 = fmaf(sv[4 * e4 + 2], sl2, mn.z), x3 = fmaf(sv[4 * e4 + 3], sl2, mn.w);
                                excess = fmaxf(excess, fmaxf(fmaxf(key <= lm.x ? x0 : -INFINITY, key <= lm.y ? x1 : -INFINITY),
                                                             fmaxf(key <= lm.z ? x2 : -INFINITY, key <= lm.w ? x3 : -INFINITY)));
                            }
                        }
                    }
                    // a NaN excess (inf - inf on a row that has seen nothing; the first tile) must count as growth
                    const bool grow = !(excess <= kRescaleThreshold);
                    tc_fence_before();
                    const bool any_grow = softmax_bar_or(grow || !ok);
                    tc_fence_after();   // the partial sums of this tile's columns may be the other warp's stores
                    // A failed wait ends the CTA's work.  The decision comes out of a second reduction, taken only on this
                    // already slow path, so that all 256 threads leave together; the abort flag itself may be raised
                    // by another warp at any moment and cannot steer control flow between barriers.
                    if (any_grow && softmax_bar_or(!ok)) { aborted = true; break; }
                    if (any_grow) {
                        // ---- exact tile maxima per row, new references, rescale of what has been accumulated
                        for (int c = c_tile; c < Rp; c += 32) {
                            float sv[16];
                            tmem_ld16(s_addr + c, sv);
                            tmem_wait_ld();
                            float mine = -INFINITY;
                            if (tail) {   // uniform over the CTA
#pragma unroll
                                for (int e4 = 0; e4 < 4; ++e4) {
                                    const int4 lm = *reinterpret_cast<const int4 *>(&sh->limit[c + 4 * e4]);
                                    sv[4 * e4] = key <= lm.x ? sv[4 * e4] : -INFINITY;
                                    sv[4 * e4 + 1] = key <= lm.y ? sv[4 * e4 + 1] : -INFINITY;
                                    sv[4 * e4 + 2] = key <= lm.z ? sv[4 * e4 + 2] : -INFINITY;
                                    sv[4 * e4 + 3] = key <= lm.w ? sv[4 * e4 + 3] : -INFINITY;
                                }
                            }
#pragma unroll
                            for (int e = 0; e < 16; ++e) {
                                const float y = warp_max(sv[e] * sl2);
                                mine = (lane == e) ? y : mine;
                            }
                            if (lane < 16) sh->wpart[quarter][c + lane] = mine;
                        }
                        softmax_bar_sync();
                        if (st < Rp) {
                            const float m_old = -sh->mneg[st];
                            const float tm = fmaxf(fmaxf(sh->wpart[0][st], sh->wpart[1][st]), fmaxf(sh->wpart[2][st], sh->wpart[3][st]));
                            const float m_new = fmaxf(m_old, tm);
                            float f = 1.f;
                            if (m_new != -INFINITY) {
                                f = (m_old == -INFINITY) ? 0.f : exp2f(m_old - m_new);
                                sh->mneg[st] = -m_new;
                            }
                            sh->fscale[st] = f;
                        }
                        softmax_bar_sync();
                        if (it > it0) {
                            // O^T and the partial sums hold tiles it0..it-1: wait until PV of tile it-1 has been accumulated
                            ok = W.wait(&sh->pv_done[(it - 1) & 1], ((it - 1) >> 1) & 1, 10) && ok;
                            tc_fence_after();
                            for (int c = c_tile; c < Rp; c += 32) {
                                float ov[16], lv[16];
                                tmem_ld16(tmem + lane_addr + col_o + c, ov);
                                tmem_ld16(tmem + lane_addr + l_cur + c, lv);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 16; ++e) { const float f = sh->fscale[c + e]; ov[e] *= f; lv[e] *= f; }
                                tmem_st16(tmem + lane_addr + col_o + c, ov);
                                tmem_st16(tmem + lane_addr + l_cur + c, lv);
                            }
                            tmem_wait_st();
                        }
                    }
                    // ---- P^T and the row sums with the references that now hold
                    if (!spare_l || any_grow) (void)write_p(l_cur, l_alt);
                    l_sel ^= spare_l ? 1 : 0;
                    if (spare_l && any_grow && flip_groups) {
                        // the next tile's sweep reads these sums from the other warp of the quarter before any barrier
                        tmem_wait_st();
                        tc_fence_before();
                        softmax_bar_sync();
                        tc_fence_after();
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh->s_free[j]));   // S^T buffer may be overwritten by QK of tile it+2
                    fence_proxy_async();
                    mbar_arrive(smem_u32(&sh->p_full[j]));
                }
                if (aborted) break;
                // ---- epilogue of the segment: row sums over the keys, then O^T / l
                // (each warp sums the columns it stored itself in the segment's last tile)
                for (int c = c_first ^ ((int)((it - 1) & flip_groups) << 4); c < Rp; c += 32) {
                    float lv[16];
                    tmem_ld16(tmem + lane_addr + col_l + l_sel * Rp + c, lv);
                    tmem_wait_ld();
                    float mine = 0.f;
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float y = lv[e];
#pragma unroll
                        for (int o = 16; o; o >>= 1) y += __shfl_xor_sync(0xffffffffu, y, o);
                        mine = (lane == e) ? y : mine;
                    }
                    if (lane < 16) sh->wpart[quarter][c + lane] = mine;
                }
                softmax_bar_sync();
                if (st < Rp) sh->fscale[st] = (sh->wpart[0][st] + sh->wpart[1][st]) + (sh->wpart[2][st] + sh->wpart[3][st]);
                ok = W.wait(&sh->pv_done[(it - 1) & 1], ((it - 1) >> 1) & 1, 13) && ok;
                // multi-layer kernel: the slot set of this layer was used kLayerRing layers ago; the merge warp says when
                // every CTA has finished reading it (long ago, as a rule)
                if (kMulti && !whole_unit && st == 0) ok = W.wait_shared_gt(&sh->slots_free_upto, layer, 16) && ok;
                tc_fence_after();
                softmax_bar_sync();
                {
                    const int unit = b * Hkv + hk;
                    // partial: a workspace slot, or (clustered) this CTA's ring memory, idle once the last PV has completed
                    float *slot = clustered ? reinterpret_cast<float *>(ring)
                                            : slot_set + (size_t)(slot_bias * unit + my_cta) * slot_float_count(R, D);
                    const int Rpad = slot_rows_padded(R);
                    const bool direct = whole_unit && !clustered;
                    // per row, by one thread: lse or the partial's (m, l); fscale becomes the factor of the row's outputs
                    if (st < Rp) {
                        const int r = st;
                        const float l = sh->fscale[r];
                        const float m_ref = -sh->mneg[r];   // -inf while nothing was visible
                        float factor = 0.f;
                        if (r < R && ok) {
                            if (direct) {
                                factor = l > 0.f ? 1.f / l : 0.f;
                                if (lse_g) lse_g[sh->rowoff[r]] = l > 0.f ? m_ref * kLn2 + logf(l) : -INFINITY;
                            } else {
                                factor = (m_ref == -INFINITY) ? 0.f : 1.f;
                                slot[r] = (m_ref == -INFINITY) ? -INFINITY : m_ref * kLn2;   // natural-log domain for the combine
                                slot[Rpad + r] = (m_ref == -INFINITY) ? 0.f : l;
                            }
                        }
                        sh->fscale[r] = factor;
                    }
                    softmax_bar_sync();
                    // the outputs: straight-line body, predicated stores
                    const bool store_ok = d_active && ok;
                    if (direct) {
                        for (int c = c_first; c < Rp; c += 32) {
                            float ov[16];
                            tmem_ld16(tmem + lane_addr + col_o + c, ov);
                            tmem_wait_ld();
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 f = *reinterpret_cast<const float4 *>(&sh->fscale[c + 4 * e4]);
                                const int4 ro = *reinterpret_cast<const int4 *>(&sh->rowoff[c + 4 * e4]);
                                const float fv[4] = {f.x, f.y, f.z, f.w};
                                const int rv4[4] = {ro.x, ro.y, ro.z, ro.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (store_ok && rv4[e] >= 0) og[(size_t)rv4[e] * D + d] = __float2bfloat16_rn(ov[4 * e4 + e] * fv[e]);
                            }
                        }
                    } else {
                        float *so = slot + 2 * Rpad + d;
                        for (int c = c_first; c < Rp; c += 32) {
                            float ov[16];
                            tmem_ld16(tmem + lane_addr + col_o + c, ov);
                            tmem_wait_ld();
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 f = *reinterpret_cast<const float4 *>(&sh->fscale[c + 4 * e4]);
                                const float fv[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int r = c + 4 * e4 + e;
                                    if (store_ok && r < R) {
                                        // multi-layer kernel: the partial is read back by a merge warp within a few
                                        // layers; ask L2 to keep it rather than write it out under the KV stream
                                        if (kMulti) st_global_f32_hint(so + (size_t)r * D, fv[e] == 0.f ? 0.f : ov[4 * e4 + e], keep_pol);
                                        else so[(size_t)r * D] = fv[e] == 0.f ? 0.f : ov[4 * e4 + e];
                                    }
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                softmax_bar_sync();   // tables and tensor memory are rewritten by the next segment
                if (kMulti && !whole_unit) {
                    // the partial is in memory (every thread stored before the barrier): tell the merge warp
                    ++n_partials;
                    if (st == 0) st_release_cta_shared(&sh->seg_done, n_partials);
                }
                t += n;
                ++seg;
            }
        }
    }

    // ---- teardown
    tc_fence_before();
    __syncthreads();
    if (clustered) {
        // Every thread of every CTA of the cluster gets here, whatever happened before, so the barriers complete.
        const int u = blockIdx.x / cluster_size, rank = blockIdx.x % cluster_size;
        const int b = u / Hkv, hk = u % Hkv;
        const int Rpad = slot_rows_padded(R);
        float *mine = reinterpret_cast<float *>(ring);
        long long t_begin, t_end;
        range_of((int)blockIdx.x, t_begin, t_end);
        if (t_begin == t_end || sh->abort) {   // no tiles for this CTA, or it gave up (its loads have landed): an empty partial
            for (int r = tid; r < R; r += kThreads) { mine[r] = -INFINITY; mine[Rpad + r] = 0.f; }
        }
        cluster_sync_all();
        if (sh->tile_prefix[b + 1] == sh->tile_prefix[b]) {
            // a sequence shorter than q_len is skipped: its outputs are defined as zero (rows of this unit, by rank 0)
            if (rank == 0) {
                for (int x = tid; x < R * D; x += kThreads) {
                    const int r = x / D;
                    const size_t ro = (size_t)(b * p.q_len + r / G) * p.n_q_heads + hk * G + r % G;
                    ((__nv_bfloat16 *)set.out[0])[ro * D + x % D] = __float2bfloat16_rn(0.f);
                    if (set.lse[0] && x % D == 0) set.lse[0][ro] = -INFINITY;
                }
            }
        } else {
            // rows r = rank, rank + cluster_size, ... of the unit are merged here, one warp per row
            constexpr int V = D / 32;
            const uint32_t local = smem_u32(mine);
            for (int r = rank + cluster_size * warp; r < R; r += cluster_size * (kThreads / 32)) {
                float M = -INFINITY, L = 0.f, acc[V];
#pragma unroll
                for (int x = 0; x < V; ++x) acc[x] = 0.f;
                for (int c0 = 0; c0 < cluster_size; c0 += 8) {
                    float m[8], l[8], v[8][V];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t peer = cluster_map(local, (uint32_t)min(c0 + j, cluster_size - 1));
                        m[j] = ld_cluster_f32(peer + 4 * r);
                        l[j] = ld_cluster_f32(peer + 4 * (Rpad + r));
                        const uint32_t oa = peer + 4 * (2 * Rpad + r * D + lane * V);
                        if (V == 4) {
                            const float4 t4 = ld_cluster_v4(oa);
                            v[j][0] = t4.x; v[j][1] = t4.y; v[j][V - 2] = t4.z; v[j][V - 1] = t4.w;
                        } else {
                            const float2 t2 = ld_cluster_v2(oa);
                            v[j][0] = t2.x; v[j][1] = t2.y;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (c0 + j >= cluster_size || m[j] == -INFINITY) continue;
                        const float m_new = fmaxf(M, m[j]);
                        const float f_old = (M == -INFINITY) ? 0.f : expf(M - m_new), f_new = expf(m[j] - m_new);
                        L = L * f_old + l[j] * f_new;
#pragma unroll
                        for (int x = 0; x < V; ++x) acc[x] = acc[x] * f_old + v[j][x] * f_new;
                        M = m_new;
                    }
                }
                const size_t ro = (size_t)(b * p.q_len + r / G) * p.n_q_heads + hk * G + r % G;
                const float inv = L > 0.f ? 1.f / L : 0.f;
                __nv_bfloat16 *o = (__nv_bfloat16 *)set.out[0] + ro * D + lane * V;
                if (V == 4) {
                    __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv), h1 = __floats2bfloat162_rn(acc[V - 2] * inv, acc[V - 1] * inv);
                    *reinterpret_cast<uint2 *>(o) = make_uint2(*reinterpret_cast<uint32_t *>(&h0), *reinterpret_cast<uint32_t *>(&h1));
                } else {
                    __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
                    *reinterpret_cast<uint32_t *>(o) = *reinterpret_cast<uint32_t *>(&h0);
                }
                if (set.lse[0] && lane == 0) set.lse[0][ro] = L > 0.f ? M + logf(L) : -INFINITY;
            }
        }
        cluster_sync_all();   // nobody leaves while a peer may still read its shared memory
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
    }
}

// Merge of the per-CTA partials of one output row (b, t, h); rows whose unit was covered by a single CTA were
// written by it and are skipped.  One CTA of 8 warps per row.  Warp w takes the contributors c = w, w+8, ... and
// merges them online (running max, sum, D/32 output columns per lane); every global load of a pass is independent
// of the others, so a pass costs one memory round trip.  The eight warp results are merged through shared memory.
constexpr int kCombineThreads = 256;
template <int D>
__global__ void __launch_bounds__(kCombineThreads) attn_tc_combine_kernel(const AttnParams p, const int main_grid) {
    constexpr int V = D / 32;   // output columns per lane
    __shared__ float w_m[8], w_l[8];
    __shared__ float w_acc[8][D];
    __shared__ int2 s_info;
    const int R = p.rows, G = p.group, Hkv = p.n_kv_heads;
    const int row = blockIdx.x, tid = threadIdx.x, w = tid >> 5, lane = tid & 31;
    const int h = row % p.n_q_heads, t = (row / p.n_q_heads) % p.q_len, b = row / (p.n_q_heads * p.q_len);
    const int hk = h / G, r = t * G + (h % G);
    __nv_bfloat16 *out = (__nv_bfloat16 *)p.out + (size_t)row * D;
    if (main_grid > 0) {
        // Unit-aligned split with at most 32 units: which partials belong to this row's unit follows from the lengths
        // alone.  The lengths are an input of the call, complete before the main kernel let this one be launched, so
        // the table is worked out here while the main kernel is still running, instead of being read after it.
        if (w == 0) {
            const int U = p.batch * Hkv;
            const int kvl = lane < p.batch ? (p.kv_len ? __ldcg(p.kv_len + lane) : p.max_kv_len) : 0;
            const int nt = lane < p.batch ? seq_tiles(kvl, p.q_len) : 0;
            int sum = nt;
#pragma unroll
            for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            const int my_tiles = __shfl_sync(0xffffffffu, nt, lane < U ? lane / Hkv : 0);
            int all;
            const int2 mine = aligned_split_warp(lane, U, main_grid, lane < U ? my_tiles : 0, (long long)sum * Hkv, all);
            const int2 pick = make_int2(__shfl_sync(0xffffffffu, mine.x, b * Hkv + hk), __shfl_sync(0xffffffffu, mine.y, b * Hkv + hk));
            if (lane == 0) s_info = pick;
        }
        __syncthreads();
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int2 info = main_grid > 0 ? s_info : reinterpret_cast<const int2 *>(p.counters)[b * Hkv + hk];   // first slot, contributors
    const int n = info.y;
    if (n == 0) {   // a sequence shorter than q_len is skipped: its outputs are defined as zero
        if (tid < D) out[tid] = __float2bfloat16_rn(0.f);
        if (p.lse && tid == 0) p.lse[row] = -INFINITY;
        return;
    }
    if (n == 1) return;
    const size_t slot_floats = slot_float_count(R, D);
    const int Rp = slot_rows_padded(R);
    const float *base = p.partials + (size_t)info.x * slot_floats;
    float M = -INFINITY, L = 0.f, acc[V];
#pragma unroll
    for (int x = 0; x < V; ++x) acc[x] = 0.f;
    for (int c0 = w; c0 < n; c0 += 32) {
        float m[4], l[4], v[4][V];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = min(c0 + 8 * j, n - 1);    // clamped; a repeated contributor is dropped below
            const float *sl = base + (size_t)c * slot_floats;
            m[j] = sl[r];
            l[j] = sl[Rp + r];
            if (V == 4) {
                const float4 t4 = *reinterpret_cast<const float4 *>(sl + 2 * Rp + (size_t)r * D + lane * V);
                v[j][0] = t4.x; v[j][1] = t4.y; v[j][V - 2] = t4.z; v[j][V - 1] = t4.w;
            } else {
                const float2 t2 = *reinterpret_cast<const float2 *>(sl + 2 * Rp + (size_t)r * D + lane * V);
                v[j][0] = t2.x; v[j][1] = t2.y;
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (c0 + 8 * j >= n || m[j] == -INFINITY) continue;
            const float m_new = fmaxf(M, m[j]);
            const float f_old = (M == -INFINITY) ? 0.f : expf(M - m_new), f_new = expf(m[j] - m_new);
            L = L * f_old + l[j] * f_new;
#pragma unroll
            for (int x = 0; x < V; ++x) acc[x] = acc[x] * f_old + v[j][x] * f_new;
            M = m_new;
        }
    }
    if (lane == 0) { w_m[w] = M; w_l[w] = L; }
#pragma unroll
    for (int x = 0; x < V; ++x) w_acc[w][lane * V + x] = acc[x];
    __syncthreads();
    if (tid < D) {
        float Mt = -INFINITY;
#pragma unroll
        for (int k = 0; k < 8; ++k) Mt = fmaxf(Mt, w_m[k]);
        float Lt = 0.f, o = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float f = (w_m[k] == -INFINITY) ? 0.f : expf(w_m[k] - Mt);
            Lt += w_l[k] * f;
            o += w_acc[k][tid] * f;
        }
        out[tid] = __float2bfloat16_rn(Lt > 0.f ? o / Lt : 0.f);
        if (p.lse && tid == 0) p.lse[row] = Lt > 0.f ? Mt + logf(Lt) : -INFINITY;
    }
}

// ---- host side -----------------------------------------------------------------------------------------------------
EncodeTiledFn tensor_map_encoder() {
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
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kPageSize};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return HIPPO_OK;
}

bool attn_tc_supported(const AttnParams &p, int dtype) {
    return dtype == HIPPO_DTYPE_BF16 && (p.head_dim == 64 || p.head_dim == 128) && p.batch <= kTcMaxBatch &&
           p.rows <= kMaxRows;
}

// Cluster size for the one-cluster-per-unit mode, or 0 for the split modes.  `pages` = pages of the longest unit,
// `total_pages` = pages of all units (exact when the caller passed the lengths on the host, else units * pages);
// max_active[cs] = clusters of cs CTAs of this kernel that the device keeps resident at once.  The cluster mode
// needs no second kernel, but all clusters must be resident together, a unit gets at most 16 SMs and the longest
// unit sets the time, so long caches with few units and ragged batches stay on the split path.
static int choose_cluster_size(int units, int pages, long long total_pages, int total_rows, const int *max_active) {
    // costs in pages per CTA (ranges are cut on page boundaries); the second kernel of the split modes is worth ten, and
    // one more for every 128 output rows it merges (measured: 8 ragged sequences of 168 rows, 35 pages per CTA in the split
    // mode against 50 in the cluster mode, 46.4 us against 43.7 us)
    int best = 0, best_cost = (int)((total_pages + kNumSMs - 1) / kNumSMs) + 10 + total_rows / 128;
    for (int cs = 2; cs <= 16 && 2 * cs <= pages + 1; ++cs) {
        if (units > max_active[cs]) continue;
        const int cost = ceil_div(pages, cs);
        if (cost < best_cost || (cost == best_cost && best == 0)) { best = cs; best_cost = cost; }
    }
    return best;
}

// Pages of the longest unit and of all units together, from the host copy of the lengths when there is one.
static void plan_pages(const AttnParams &p, int &longest, long long &total) {
    const int bound = ceil_div(p.max_kv_len, kPageSize);
    longest = bound;
    total = (long long)p.batch * p.n_kv_heads * bound;
    if (p.kv_len_host) {
        longest = 0;
        total = 0;
        for (int b = 0; b < p.batch; ++b) {
            int kvl = p.kv_len_host[b];
            if (kvl > p.max_kv_len) kvl = p.max_kv_len;
            const int pg = kvl < p.q_len ? 0 : ceil_div(kvl, kPageSize);
            if (pg > longest) longest = pg;
            total += (long long)pg * p.n_kv_heads;
        }
        if (longest < 1) longest = 1;
    }
}

struct TcLaunchShape { int Rp, spare_cols, tmem_cols; TcSmemPlan plan; };
template <int D>
static int32_t tc_launch_shape(const AttnParams &p, TcLaunchShape &s) {
    s.Rp = (p.rows + 15) & ~15;
    s.plan = tc_smem_plan(D, s.Rp);
    if (s.plan.slots < 3) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "attention: shared memory too small for %d packed rows", p.rows);
    // tensor-memory columns: S^T x 2, O^T, partial row sums; a second set of sums when 512 columns allow it
    s.spare_cols = 5 * s.Rp <= 512 ? s.Rp : 0;
    s.tmem_cols = 32;
    while (s.tmem_cols < 4 * s.Rp + s.spare_cols) s.tmem_cols *= 2;
    return HIPPO_OK;
}

template <int D>
static int32_t launch_tc(const AttnParams &p, int grid, cudaStream_t stream) {
    LayerSetT<1> set;
    const long long rows = (long long)p.n_pages * p.n_kv_heads * kPageSize;
    int32_t rc = make_map(&set.k[0], p.k_pages, rows, D);
    if (rc != HIPPO_OK) return rc;
    rc = make_map(&set.v[0], p.v_pages, rows, D);
    if (rc != HIPPO_OK) return rc;
    set.q[0] = p.q; set.out[0] = p.out; set.lse[0] = p.lse;
    MultiCtl mc = {};
    TcLaunchShape sh;
    rc = tc_launch_shape<D>(p, sh);
    if (rc != HIPPO_OK) return rc;
    const TcSmemPlan &plan = sh.plan;
    static PerDeviceOnce attr_set;
    int dev;
    if (attr_set.needed(dev)) {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<D, 1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        attr_set.mark(dev);
    }
    const int units = p.batch * p.n_kv_heads;
    // resident clusters per cluster size, asked once per ring size (the only launch parameter that moves it); every
    // device of this library's only target has the same answer, so one table serves them all
    static int max_active[kMaxSlots + 1][17];
    static std::atomic<bool> have_active[kMaxSlots + 1];
    if (!have_active[plan.slots].load(std::memory_order_acquire)) {
        for (int c = 2; c <= 16; ++c) {
            cudaLaunchConfig_t q = {};
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = (unsigned)c; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
            q.gridDim = dim3((unsigned)(c * kNumSMs)); q.blockDim = dim3(kTcThreads); q.dynamicSmemBytes = (size_t)plan.total;
            q.attrs = qa; q.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<D, 1>, &q) != cudaSuccess) { n = 0; (void)cudaGetLastError(); }
            max_active[plan.slots][c] = n;
        }
        have_active[plan.slots].store(true, std::memory_order_release);
    }
    int longest;
    long long total_pages;
    plan_pages(p, longest, total_pages);
    const int cs = p.num_splits > 0 ? 0 : choose_cluster_size(units, longest, total_pages, p.batch * p.q_len * p.n_q_heads, max_active[plan.slots]);
    // Both kernels are launched with programmatic stream serialization and wait (griddepcontrol.wait) before they
    // touch memory, so stream order is kept while launch latency overlaps the previous kernel's tail.
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = (size_t)plan.total;
    cfg.stream = stream;
    cfg.attrs = attr;
    if (cs > 1) {
        // one cluster per unit; the partial of a CTA (m, l, O) must fit in its ring memory
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cs;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
        cfg.gridDim = dim3((unsigned)(units * cs));
        if (slot_float_count(p.rows, D) * sizeof(float) <= (size_t)plan.slots * kBlockN * D * 2 &&
            cudaLaunchKernelEx(&cfg, attn_tc_kernel<D, 1>, p, set, mc, sh.Rp, plan.slots, sh.tmem_cols, cs, sh.spare_cols) == cudaSuccess) {
            count_launches(1);
            return HIPPO_OK;
        }
        (void)cudaGetLastError();   // clusters of this size cannot be scheduled here: use the split modes
    }
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)grid);
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_tc_kernel<D, 1>, p, set, mc, sh.Rp, plan.slots, sh.tmem_cols, 0, sh.spare_cols));
    count_launches(1);
    cfg.gridDim = dim3((unsigned)(p.batch * p.q_len * p.n_q_heads));
    cfg.blockDim = dim3(kCombineThreads);
    cfg.dynamicSmemBytes = 0;
    // unit-aligned split by one warp (see the kernel): the combine kernel derives the slot table itself
    const int derive = (units <= grid && units <= 32) ? grid : 0;
    HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_tc_combine_kernel<D>, p, derive));
    count_launches(1);
    return HIPPO_OK;
}

// Grid of the split modes: one CTA per SM, never more CTAs than pages (bound from the host-side length bound; the
// kernel derives the exact partition from kv_len on the device).
static int split_grid(const AttnParams &p, int sms) {
    const long long max_tiles = (long long)p.batch * p.n_kv_heads * ceil_div(p.max_kv_len, kPageSize);
    long long grid = p.num_splits > 0 ? (long long)p.num_splits * p.batch * p.n_kv_heads : sms;
    if (grid > max_tiles) grid = max_tiles;
    if (grid > kExtraSlots) grid = kExtraSlots;
    if (grid < 1) grid = 1;
    return (int)grid;
}

int32_t launch_attn_tc(const AttnParams &p, cudaStream_t stream) {
    const int grid = split_grid(p, kNumSMs);
    if (p.head_dim == 128) return launch_tc<128>(p, grid, stream);
    return launch_tc<64>(p, grid, stream);
}

// ---- several layers in one launch -----------------------------------------------------------------------------------
bool attn_tc_layers_supported(const AttnParams &p, int dtype) {
    return attn_tc_supported(p, dtype) && p.batch * p.n_kv_heads <= kMaxAlignedUnits;
}

AttnLayersWsLayout attn_layers_ws_layout(int n_layers, int batch, int q_len, int n_q_heads, int n_kv_heads, int head_dim) {
    AttnLayersWsLayout L;
    const AttnWsLayout one = attn_ws_layout(batch, q_len, n_q_heads, n_kv_heads, head_dim);
    const size_t units = (size_t)batch * n_kv_heads;
    L.counters_off = one.counters_off;
    L.done_off = L.counters_off + one.counters_bytes;
    L.done_bytes = align_up(((size_t)n_layers * units + (size_t)n_layers) * sizeof(int32_t), 256);
    L.partials_off = L.done_off + L.done_bytes;
    L.slot_floats = one.slot_floats;
    L.slots_per_set = units + kNumSMs;
    L.total = L.partials_off + align_up((size_t)kLayerRing * L.slots_per_set * L.slot_floats * sizeof(float), 256);
    if (L.total < one.total) L.total = one.total;   // shapes outside this kernel run layer by layer on the single-layer paths
    return L;
}

template <int D>
static int32_t launch_tc_layers(AttnParams p, int n_layers, const void *const *q, const hippo_kv_cache_t *kv, void *const *out,
                                float *const *lse, int max_ctas, void *workspace, cudaStream_t stream) {
    constexpr int NL = kLayersPerLaunch;
    TcLaunchShape sh;
    int32_t rc = tc_launch_shape<D>(p, sh);
    if (rc != HIPPO_OK) return rc;
    static PerDeviceOnce attr_set;
    static std::atomic<int> sm_count[kMaxDevices];
    int dev;
    if (attr_set.needed(dev)) {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<D, NL>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        if (dev >= 0) {
            int n = 0;
            HIPPO_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
            sm_count[dev].store(n, std::memory_order_relaxed);
        }
        attr_set.mark(dev);
    }
    // the CTAs wait for one another's partials, so all of them must be resident together: one per SM at most
    int sms = dev >= 0 ? sm_count[dev].load(std::memory_order_relaxed) : 1;
    if (sms > kNumSMs) sms = kNumSMs;
    if (max_ctas > 0 && sms > max_ctas) sms = max_ctas;    // the caller leaves the other SMs to concurrent kernels
    if (sms < 1) sms = 1;
    p.num_splits = 0;
    // Short caches: with fewer than about seven pages per CTA and layer a CTA spends longer merging (every output row
    // gathers one partial per contributing CTA) than streaming, so the grid shrinks with the work, to a whole number of
    // CTAs per unit where it can.  Measured at 6,400 keys, 4 kv heads, 42 packed rows, per layer: 19.1 us on 148 CTAs,
    // 17.3 on 72, 15.0 on 64, 14.6 on 56, 17.1 on 48.
    {
        int longest;
        long long total_pages;
        plan_pages(p, longest, total_pages);
        long long by_work = total_pages / 7;
        const int units_all = p.batch * p.n_kv_heads;
        if (by_work > units_all) by_work -= by_work % units_all;
        if (by_work < sms) sms = (int)(by_work < 1 ? 1 : by_work);
    }
    const int grid = split_grid(p, sms);
    const AttnLayersWsLayout L = attn_layers_ws_layout(n_layers, p.batch, p.q_len, p.n_q_heads, p.n_kv_heads, D);
    const int units = p.batch * p.n_kv_heads;
    p.header = (WsHeader *)workspace;
    p.counters = (int32_t *)((char *)workspace + L.counters_off);
    p.partials = (float *)((char *)workspace + L.partials_off);
    MultiCtl mc;
    mc.done = (int *)((char *)workspace + L.done_off);
    mc.merged = mc.done + (size_t)n_layers * units;
    mc.ring_floats = (long long)(L.slots_per_set * L.slot_floats);
    mc.rot = 0;
    for (int cand : {41, 43, 47, 53, 1}) {   // a stride that is coprime with the grid visits every range
        int a = grid, b = cand % grid;
        while (b) { const int t = a % b; a = b; b = t; }
        if (grid > 1 && a == 1) { mc.rot = cand % grid; break; }
    }
    HIPPO_CUDA_TRY(cudaMemsetAsync(mc.done, 0, L.done_bytes, stream));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kTcThreads + 32);
    cfg.gridDim = dim3((unsigned)grid);
    cfg.dynamicSmemBytes = (size_t)sh.plan.total;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    for (int l0 = 0; l0 < n_layers; l0 += NL) {
        LayerSetT<NL> set;
        memset(&set, 0, sizeof(set));
        mc.layer0 = l0;
        mc.n_layers = n_layers - l0 < NL ? n_layers - l0 : NL;
        for (int i = 0; i < mc.n_layers; ++i) {
            const hippo_kv_cache_t &c = kv[l0 + i];
            const long long rows = (long long)c.n_pages * p.n_kv_heads * kPageSize;
            rc = make_map(&set.k[i], c.k_pages, rows, D);
            if (rc != HIPPO_OK) return rc;
            rc = make_map(&set.v[i], c.v_pages, rows, D);
            if (rc != HIPPO_OK) return rc;
            set.q[i] = q[l0 + i];
            set.out[i] = out[l0 + i];
            set.lse[i] = lse ? lse[l0 + i] : nullptr;
        }
        HIPPO_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_tc_kernel<D, NL>, p, set, mc, sh.Rp, sh.plan.slots, sh.tmem_cols, 0, sh.spare_cols));
        count_launches(1);
    }
    return HIPPO_OK;
}

int32_t launch_attn_tc_layers(const AttnParams &p, int n_layers, const void *const *q, const hippo_kv_cache_t *kv,
                              void *const *out, float *const *lse, int max_ctas, void *workspace, cudaStream_t stream) {
    if (p.head_dim == 128) return launch_tc_layers<128>(p, n_layers, q, kv, out, lse, max_ctas, workspace, stream);
    return launch_tc_layers<64>(p, n_layers, q, kv, out, lse, max_ctas, workspace, stream);
}

}  // namespace hippo
