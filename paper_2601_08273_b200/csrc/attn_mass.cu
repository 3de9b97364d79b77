// hippo_attention_mass: global semantic relevance of the visual tokens (Section 5.1, Eq. 2), one layer per call.
//
//   mass[b][j] += weight * sum over heads h and text rows i of  softmax_j( scale * q[b][i][h] . K[b][j][h / G] ),
//   the softmax taken over the visual keys j < n_visual[b] only.
//
// The normaliser of a row needs all keys, the score of a key needs all rows, so the logits are formed twice, both
// times on the tensor cores (bf16, head_dim 64 or 128), and never stored:
//   pass 1 (row statistics)  S   [128 rows x 128 keys] = Q_block . K_tile^T    thread = row: running max and sum of
//                                                                                exponentials over its CTA's key tiles
//   merge                     the key splits of a row -> t = -(max + log2 sum)
//   pass 2 (column sums)      S^T [128 keys x 128 rows] = K_tile . Q_block^T    thread = key: sum over the rows of
//                                                                                2^(s + t_row)
//   reduce                    mass += weight * (sum of the KV heads' column sums), in a fixed order
// Both passes are one kernel: a "resident" tile is the A operand (the Q block in pass 1, the key tile in pass 2) and
// the other operand streams through a ring of shared-memory slots; the accumulator tile lives in tensor memory,
// double buffered, and a consumer thread owns one tensor-memory lane (a row of the accumulator), so neither pass
// needs a cross-thread reduction.  The packed rows of a KV head are r = i * G + g (text row i, head hk * G + g); a
// block takes T = floor(128 / G) text rows, fetched with one 4-D TMA box per 64 columns straight into the
// 128-byte-swizzled operand layout.  Keys come in 128-key tiles = two 64-token pages, as in the attention kernels.
//
// CTA = 18 warps: warp 0 TMA producer, warp 1 MMA issuer and tensor-memory owner, warps 2-17 consumers (a warp reads
// its quarter of the tensor-memory lanes and one 32-column slice of the tile).
// The work is bound by the exponentials (one per row and key in each pass), not by the MMAs or by memory.
// Every mbarrier wait is bounded; on expiry the CTA records HIPPO_ERR_TIMEOUT in the workspace header and exits.
//
// Other shapes and fp32 storage run on a plain CUDA-core path (one warp per row, one thread per key).
#include <cuda.h>
#include <math.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace hippo {

constexpr int kMassSlices = 4;            // column slices of an accumulator tile, one consumer warp each per lane quarter
constexpr int kMassSliceCols = 32;
constexpr int kMassConsumers = 128 * kMassSlices;
constexpr int kMassThreads = 64 + kMassConsumers;
constexpr int kMassSlots = 3;            // ring of streamed tiles
constexpr int kMassTile = 128;           // rows and keys per accumulator tile
constexpr int kMassMaxBatch = 64;        // per-sequence lengths travel in the kernel parameters
constexpr int kMassMaxSplits = 64;
constexpr int kMassMaxRows = 3072;       // l_txt * group: the pass-2 table of a KV head lives in shared memory
constexpr float kMassLog2e = 1.4426950408889634f;
constexpr unsigned long long kMassWaitLimitNs = 2000000000ull;

struct MassParams {
    int batch, l_txt, n_q_heads, n_kv_heads, group, head_dim;
    int t_per_block;       // T: text rows per row block
    int rows_per_block;    // T * G
    int n_row_blocks;      // ceil(l_txt / T)
    int r_tot;             // l_txt * G packed rows per KV head
    int splits;            // key splits of this launch
    int stat_splits;       // key splits of pass 1 (layout of `stats`)
    int sum_nv;            // total visual tokens
    int max_pages_per_seq;
    float sl2;             // softmax scale * log2(e)
    float scale;
    float weight;
    const int32_t *page_table;
    const void *q;
    const void *k_pages;
    float2 *stats;         // [batch * n_kv_heads][stat_splits][r_tot]: (max in the log2 domain, sum of 2^(x - max))
    float2 *table;         // CUDA-core path: [batch * n_kv_heads][r_tot] (-max, 1 / sum), natural-log domain
    float *table_log2;     // tensor-core path, same memory: [batch * n_kv_heads][r_tot] -(max + log2 sum), log2 domain
    float *colsum;         // [n_kv_heads][sum_nv]
    float *mass;           // [sum_nv]
    WsHeader *header;
    int n_visual[kMassMaxBatch];
    int offset[kMassMaxBatch];   // first token of each sequence in the concatenated mass array
};

struct MassShared {
    unsigned long long full[kMassSlots], empty[kMassSlots], res_full[2], res_free[2], s_full[2], s_free[2], drain;
    long long wait_limit;   // the header's wait limit (0: the built-in one), read once
    uint32_t tmem_base;
    volatile int abort;
};

// Polling part of a bounded wait.  The limit is kMassWaitLimitNs unless the workspace header carries another one (a
// debugging aid, read once per CTA into shared memory): then the waits poll without suspending and look at the clock
// after every poll.  A drain wait guards the exit of the CTA (loads in flight, tensor-core work in flight): it keeps the
// built-in limit and does not give up because another wait did.
__device__ __noinline__ bool mass_wait_slow(MassShared *sh, WsHeader *hdr, uint32_t b, uint32_t parity, int site, bool draining) {
    const unsigned long long t0 = global_ns();
    const long long user = draining ? 0 : sh->wait_limit;
    const unsigned long long limit = user > 0 ? (unsigned long long)user : kMassWaitLimitNs;
    for (uint32_t i = 1;; ++i) {
        if (user > 0 ? mbar_test_wait(b, parity) : mbar_try_wait(b, parity)) return true;
        if (user > 0 || (i & 31) == 0) {
            if (!draining && sh->abort) return false;
            if (global_ns() - t0 > limit) {
                sh->abort = 1;
                if (atomicCAS(&hdr->status, 0, (int)HIPPO_ERR_TIMEOUT) == 0) hdr->where = 100 + site;
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mass_wait(MassShared *sh, WsHeader *hdr, unsigned long long *bar, uint32_t parity, int site,
                                          bool draining = false) {
    const uint32_t b = smem_u32(bar);
    if ((!draining && sh->wait_limit > 0) ? mbar_test_wait(b, parity) : mbar_try_wait(b, parity)) return true;
    return mass_wait_slow(sh, hdr, b, parity, site, draining);
}

// PASS 0: row statistics (resident Q block, streamed key tiles).  PASS 1: column sums (resident key tile, streamed Q blocks).
// Pass 0 keeps one resident tile and a ring of two, so that two CTAs share an SM: the maximum phase of one runs beside
// the exponentials of the other.  Pass 1 changes its resident tile per outer step and double-buffers it.
template <int PASS> struct MassBuffers {
    static constexpr int kRes = PASS == 0 ? 1 : 2;
    static constexpr int kSlots = PASS == 0 ? 2 : kMassSlots;
    static constexpr int kCtasPerSm = PASS == 0 ? 2 : 1;
};

template <int D, int PASS>
__global__ void __launch_bounds__(kMassThreads, MassBuffers<PASS>::kCtasPerSm)
mass_tc_kernel(const MassParams p, const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap q_map) {
    constexpr int kChunks = D / 64;                       // 64-column (128-byte) swizzle chunks per row
    constexpr int kChunkBytes = kMassTile * 128;          // one chunk of a 128-row tile
    constexpr int kTileBytes = kChunks * kChunkBytes;
    constexpr int kPageChunkBytes = kPageSize * 128;      // one chunk of one page
    constexpr int kRes = MassBuffers<PASS>::kRes, kSlots = MassBuffers<PASS>::kSlots;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *res = base;                                  // [2] resident tiles: [chunk][128 rows][128 B], 128-byte swizzle
    uint8_t *ring = res + kRes * kTileBytes;              // [kSlots] streamed tiles, same layout
    float *tab = (float *)(ring + kSlots * kTileBytes);   // pass 1 only: -(max + log2 sum) of the KV head's rows
    const int tab_entries = PASS == 1 ? ((p.r_tot + kMassSliceCols + 15) & ~15) : 0;
    float2 *part = (float2 *)(tab + tab_entries);           // [2][kMassSlices][128]: the slices' partial results
    MassShared *sh = (MassShared *)(part + 2 * kMassSlices * kMassTile);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = p.group, Hkv = p.n_kv_heads, T = p.t_per_block, TG = p.rows_per_block;
    int bid = blockIdx.x;
    const int split = bid % p.splits; bid /= p.splits;
    int rb = 0;
    if (PASS == 0) { rb = bid % p.n_row_blocks; bid /= p.n_row_blocks; }
    const int hk = bid % Hkv, b = bid / Hkv;
    const int unit = b * Hkv + hk;
    const int nv = p.n_visual[b];
    const int nkt = (nv + kMassTile - 1) / kMassTile;
    const int kt0 = (int)((long long)split * nkt / p.splits), kt1 = (int)((long long)(split + 1) * nkt / p.splits);
    // outer loop: resident tiles; inner loop: streamed tiles
    const int o0 = PASS == 0 ? rb : kt0, o1 = PASS == 0 ? rb + 1 : kt1;
    const int i0 = PASS == 0 ? kt0 : 0, i1 = PASS == 0 ? kt1 : p.n_row_blocks;

    if (o1 <= o0 || i1 <= i0) {
        // nothing to stream: a pass-0 CTA still owes its rows an empty partial
        if (PASS == 0 && tid < TG && rb * TG + tid < p.r_tot)
            p.stats[((size_t)unit * p.stat_splits + split) * p.r_tot + rb * TG + tid] = make_float2(-INFINITY, 0.f);
        return;
    }

    // ---- set-up
    if (tid >= 32 && tid < 32 + kSlots) mbar_init(smem_u32(&sh->full[tid - 32]), 1);
    else if (tid >= 40 && tid < 40 + kSlots) mbar_init(smem_u32(&sh->empty[tid - 40]), 1);
    else if (tid >= 48 && tid < 50) mbar_init(smem_u32(&sh->res_full[tid - 48]), 1);
    else if (tid >= 50 && tid < 52) mbar_init(smem_u32(&sh->res_free[tid - 50]), 1);
    else if (tid >= 52 && tid < 54) mbar_init(smem_u32(&sh->s_full[tid - 52]), 1);
    else if (tid >= 54 && tid < 56) mbar_init(smem_u32(&sh->s_free[tid - 54]), kMassConsumers);
    else if (tid == 56) mbar_init(smem_u32(&sh->drain), 1);
    else if (tid == 57) { sh->abort = 0; sh->wait_limit = p.header->wait_limit_ns; }
    if (tid == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&k_map) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Rows of a tile that no load ever writes (the last 128 - T*G rows of a Q block, a missing second page) must hold
    // finite numbers: clear all tile buffers once.
    for (int x = tid; x < (kRes + kSlots) * kTileBytes / 16; x += kMassThreads) reinterpret_cast<uint4 *>(res)[x] = make_uint4(0, 0, 0, 0);
    if (PASS == 1) {
        const float *src = p.table_log2 + (size_t)unit * p.r_tot;
        for (int x = tid; x < tab_entries; x += kMassThreads) tab[x] = x < p.r_tot ? src[x] : -INFINITY;
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    WsHeader *hdr = p.header;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            auto load_keys = [&](uint8_t *dst, int kt, uint32_t bar) {
                const int pages_b = (nv + kPageSize - 1) / kPageSize;
                const int np = min(2, pages_b - 2 * kt);
                mbar_expect_tx(bar, np * kChunks * kPageChunkBytes);
                for (int q = 0; q < np; ++q) {
                    const int row = (page_of(p.page_table, p.max_pages_per_seq, b, 2 * kt + q) * Hkv + hk) * kPageSize;
#pragma unroll
                    for (int c = 0; c < kChunks; ++c)
                        tma_load_2d(smem_u32(dst) + c * kChunkBytes + q * kPageChunkBytes, &k_map, c * 64, row, bar);
                }
            };
            auto load_rows = [&](uint8_t *dst, int blk, uint32_t bar) {
                mbar_expect_tx(bar, kChunks * TG * 128);
#pragma unroll
                for (int c = 0; c < kChunks; ++c) tma_load_4d(smem_u32(dst) + c * kChunkBytes, &q_map, c * 64, hk * G, blk * T, b, bar);
            };
            RingPos rp{0, 0};
            uint32_t issued = 0, res_issued = 0;
            bool ok = true;
            for (int o = o0; o < o1 && ok; ++o) {
                const int rbuf = (o - o0) % kRes;
                ok = mass_wait(sh, hdr, &sh->res_free[rbuf], ((((o - o0) / kRes) & 1) ^ 1), 1);
                if (!ok) break;
                if (PASS == 0) load_rows(res + rbuf * kTileBytes, o, smem_u32(&sh->res_full[rbuf]));
                else load_keys(res + rbuf * kTileBytes, o, smem_u32(&sh->res_full[rbuf]));
                ++res_issued;
                for (int i = i0; i < i1; ++i, rp.advance(kSlots), ++issued) {
                    ok = mass_wait(sh, hdr, &sh->empty[rp.slot], rp.phase ^ 1, 2);
                    if (!ok) break;
                    if (PASS == 0) load_keys(ring + rp.slot * kTileBytes, i, smem_u32(&sh->full[rp.slot]));
                    else load_rows(ring + rp.slot * kTileBytes, i, smem_u32(&sh->full[rp.slot]));
                }
            }
            // every load that was issued must have landed before the CTA may exit
            const int back = issued < (uint32_t)kSlots ? (int)issued : kSlots;
            for (int k = 0; k < back; ++k) {
                if (rp.slot == 0) { rp.slot = kSlots - 1; rp.phase ^= 1; } else --rp.slot;
                mass_wait(sh, hdr, &sh->full[rp.slot], rp.phase, 3, true);
            }
            for (uint32_t k = res_issued > (uint32_t)kRes ? res_issued - kRes : 0; k < res_issued; ++k)
                mass_wait(sh, hdr, &sh->res_full[k % kRes], (k / kRes) & 1, 4, true);
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            const uint32_t idesc = instr_desc(kMassTile, kMassTile, false, false);   // both operands K-major
            const uint64_t adesc0 = smem_desc(smem_u32(res), 16, 1024, 2);
            const uint64_t bdesc0 = smem_desc(smem_u32(ring), 16, 1024, 2);
            RingPos rp{0, 0};
            uint32_t it = 0;
            bool ok = true;
            for (int o = o0; o < o1 && ok; ++o) {
                const int rbuf = (o - o0) % kRes;
                ok = mass_wait(sh, hdr, &sh->res_full[rbuf], ((o - o0) / kRes) & 1, 5);
                for (int i = i0; i < i1 && ok; ++i, ++it, rp.advance(kSlots)) {
                    const int j = it & 1;
                    ok = mass_wait(sh, hdr, &sh->full[rp.slot], rp.phase, 6);
                    if (!ok) break;
                    if (it >= 2) { ok = mass_wait(sh, hdr, &sh->s_free[j], ((it - 2) >> 1) & 1, 7); if (!ok) break; }
                    tc_fence_after();
                    const uint64_t ad = adesc0 + (uint64_t)((uint32_t)(rbuf * kTileBytes) >> 4);
                    const uint64_t bd = bdesc0 + (uint64_t)((uint32_t)(rp.slot * kTileBytes) >> 4);
#pragma unroll
                    for (int c = 0; c < kChunks; ++c)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t off = (uint64_t)((c * kChunkBytes + ks * 32) >> 4);
                            tc_mma(tmem + j * kMassTile, ad + off, bd + off, idesc, (c | ks) ? 1u : 0u);
                        }
                    tc_commit(smem_u32(&sh->s_full[j]));
                    tc_commit(smem_u32(&sh->empty[rp.slot]));
                }
                if (ok) tc_commit(smem_u32(&sh->res_free[rbuf]));
            }
            // all tensor-core work of this CTA must be complete before tensor memory is released
            tc_commit(smem_u32(&sh->drain));
            mass_wait(sh, hdr, &sh->drain, 0, 8, true);
        }
    } else {
        // ================= consumers =================
        // A thread owns one tensor-memory lane (a row of the accumulator tile) and one 32-column slice of it; the four
        // slices of a lane run on four warps of the same scheduler, which hides the tensor-memory and MUFU latencies.
        // Control flow is the same for all consumer warps whatever `ok` is: they meet at one named barrier per outer step.
        const int quarter = warp & 3, slice = (warp - 2) >> 2;
        const int L = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const float sl2 = p.sl2;
        const int c0 = slice * kMassSliceCols;
        uint32_t it = 0;
        bool ok = true;
        for (int o = o0; o < o1; ++o) {
            float m = -INFINITY, l = 0.f, acc = 0.f;
            for (int i = i0; i < i1; ++i, ++it) {
                const int j = it & 1;
                if (ok) ok = mass_wait(sh, hdr, &sh->s_full[j], (it >> 1) & 1, 9);
                if (!ok) continue;
                tc_fence_after();
                // columns: keys of tile i (pass 0) / packed rows of block i (pass 1)
                const int ncols = PASS == 0 ? min(kMassTile, nv - i * kMassTile) : min(TG, p.r_tot - i * TG);
                const int mine = min(kMassSliceCols, ncols - c0);      // valid columns of this slice
                if (mine > 0) {
                    float sv[kMassSliceCols];
                    const uint32_t s_addr = tmem + lane_addr + j * kMassTile + c0;
                    tmem_ld16(s_addr, sv);
                    tmem_ld16(s_addr + 16, sv + 16);
                    tmem_wait_ld();
                    if (PASS == 0) {
                        float tmax = -INFINITY;
                        if (mine == kMassSliceCols) {
                            float t4[4] = {sv[0], sv[1], sv[2], sv[3]};     // four short chains instead of one long one
#pragma unroll
                            for (int e = 4; e < kMassSliceCols; ++e) t4[e & 3] = fmaxf(t4[e & 3], sv[e]);
                            tmax = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
                        } else {
#pragma unroll
                            for (int e = 0; e < kMassSliceCols; ++e) tmax = fmaxf(tmax, e < mine ? sv[e] : -INFINITY);
                        }
                        const float m_new = fmaxf(m, tmax * sl2);
                        l *= ex2_approx(m - m_new);     // m = -inf at first: factor 0
                        m = m_new;
                        const float mneg = -m_new;
                        float add0 = 0.f, add1 = 0.f;
                        if (mine == kMassSliceCols) {
                            float add2 = 0.f, add3 = 0.f;
#pragma unroll
                            for (int e = 0; e < kMassSliceCols; e += 4) {
                                add0 += ex2_approx(fmaf(sv[e], sl2, mneg));
                                add1 += ex2_approx(fmaf(sv[e + 1], sl2, mneg));
                                add2 += ex2_approx(fmaf(sv[e + 2], sl2, mneg));
                                add3 += ex2_approx(fmaf(sv[e + 3], sl2, mneg));
                            }
                            add0 += add2; add1 += add3;
                        } else {
#pragma unroll
                            for (int e = 0; e < kMassSliceCols; ++e) {
                                const float pe = ex2_approx(fmaf(sv[e], sl2, mneg));
                                add0 += e < mine ? pe : 0.f;
                            }
                        }
                        l += add0 + add1;
                    } else {
                        // 2^(s * scale * log2e - max_r) / sum_r = 2^(s * sl2 + t_r): one table entry per column
                        const float *tb = tab + i * TG + c0;
                        float a0 = 0.f, a1 = 0.f;
                        if (mine == kMassSliceCols && ((i * TG) & 3) == 0) {
                            float a2 = 0.f, a3 = 0.f;
                            const float4 *tb4 = reinterpret_cast<const float4 *>(tb);   // 16-byte aligned here
#pragma unroll
                            for (int e = 0; e < kMassSliceCols; e += 4) {
                                const float4 t = tb4[e >> 2];
                                a0 += ex2_approx(fmaf(sv[e], sl2, t.x));
                                a1 += ex2_approx(fmaf(sv[e + 1], sl2, t.y));
                                a2 += ex2_approx(fmaf(sv[e + 2], sl2, t.z));
                                a3 += ex2_approx(fmaf(sv[e + 3], sl2, t.w));
                            }
                            a0 += a2; a1 += a3;
                        } else if (mine == kMassSliceCols) {
#pragma unroll
                            for (int e = 0; e < kMassSliceCols; e += 2) {
                                a0 += ex2_approx(fmaf(sv[e], sl2, tb[e]));
                                a1 += ex2_approx(fmaf(sv[e + 1], sl2, tb[e + 1]));
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < kMassSliceCols; ++e) {
                                const float pe = ex2_approx(fmaf(sv[e], sl2, tb[e]));
                                a0 += e < mine ? pe : 0.f;
                            }
                        }
                        acc += a0 + a1;
                    }
                }
                tc_fence_before();
                mbar_arrive(smem_u32(&sh->s_free[j]));
            }
            // the four slices of a lane meet in shared memory (double buffered over the outer steps)
            float2 *pt = part + ((o - o0) & 1) * (kMassSlices * kMassTile);
            pt[slice * kMassTile + L] = PASS == 0 ? make_float2(m, l) : make_float2(acc, 0.f);
            asm volatile("bar.sync 1, %0;" ::"n"(kMassConsumers) : "memory");
            if (slice == 0 && ok && !sh->abort) {
                if (PASS == 0) {
                    float M = m;
#pragma unroll
                    for (int q = 1; q < kMassSlices; ++q) M = fmaxf(M, pt[q * kMassTile + L].x);
                    float Ls = 0.f;
#pragma unroll
                    for (int q = 0; q < kMassSlices; ++q) {
                        const float2 v = pt[q * kMassTile + L];
                        if (v.y > 0.f) Ls += v.y * ex2_approx(v.x - M);
                    }
                    if (L < TG && o * TG + L < p.r_tot)
                        p.stats[((size_t)unit * p.stat_splits + split) * p.r_tot + o * TG + L] = make_float2(M, Ls);
                } else {
                    float sum = acc;
#pragma unroll
                    for (int q = 1; q < kMassSlices; ++q) sum += pt[q * kMassTile + L].x;
                    const int key = o * kMassTile + L;
                    if (key < nv) p.colsum[(size_t)hk * p.sum_nv + p.offset[b] + key] = sum;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
    }
}

// One thread per packed row of a KV head: merge the key splits of pass 1 into t = -(max + log2 sum).
__global__ void mass_merge_kernel(const MassParams p) {
    const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)p.batch * p.n_kv_heads * p.r_tot;
    if (x >= total) return;
    const int r = (int)(x % p.r_tot);
    const int unit = (int)(x / p.r_tot);
    const float2 *src = p.stats + (size_t)unit * p.stat_splits * p.r_tot + r;
    float M = -INFINITY;
    for (int s = 0; s < p.stat_splits; ++s) M = fmaxf(M, src[(size_t)s * p.r_tot].x);
    float Lsum = 0.f;
    for (int s = 0; s < p.stat_splits; ++s) {
        const float2 v = src[(size_t)s * p.r_tot];
        if (v.y > 0.f) Lsum += v.y * exp2f(v.x - M);
    }
    p.table_log2[x] = Lsum > 0.f ? -(M + log2f(Lsum)) : -INFINITY;
}

// mass += weight * (column sums of the KV heads, added in head order)
__global__ void mass_reduce_kernel(const MassParams p) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= p.sum_nv) return;
    float s = 0.f;
    for (int hk = 0; hk < p.n_kv_heads; ++hk) s += p.colsum[(size_t)hk * p.sum_nv + x];
    p.mass[x] += p.weight * s;
}

// ---- CUDA-core path: any head_dim, fp32 or bf16 storage ---------------------------------------------------------------
// One warp per (sequence, head, text row): natural-log-domain maximum and sum over the visual keys -> table.
template <typename T>
__global__ void mass_generic_stats_kernel(const MassParams p) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int rows = p.batch * p.n_q_heads * p.l_txt;
    if (warp >= rows) return;
    const int i = warp % p.l_txt, h = (warp / p.l_txt) % p.n_q_heads, b = warp / (p.l_txt * p.n_q_heads);
    const int hk = h / p.group, g = h % p.group, D = p.head_dim, nv = p.n_visual[b];
    const T *q = (const T *)p.q + (((size_t)b * p.l_txt + i) * p.n_q_heads + h) * D;
    float m = -INFINITY, l = 0.f;
    for (int j = lane; j < nv; j += 32) {
        const int pg = page_of(p.page_table, p.max_pages_per_seq, b, j / kPageSize);
        const T *k = (const T *)p.k_pages + (((size_t)pg * p.n_kv_heads + hk) * kPageSize + j % kPageSize) * D;
        float a = 0.f;
        for (int d = 0; d < D; ++d) a = fmaf(to_float(q[d]), to_float(k[d]), a);
        a *= p.scale;
        const float mn = fmaxf(m, a);
        l = l * expf(m - mn) + expf(a - mn);
        m = mn;
    }
    for (int o = 16; o; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
        const float mn = fmaxf(m, m2);
        if (mn != -INFINITY) l = l * expf(m - mn) + l2 * expf(m2 - mn);
        m = mn;
    }
    if (lane == 0) p.table[(size_t)(b * p.n_kv_heads + hk) * p.r_tot + i * p.group + g] = l > 0.f ? make_float2(-m, 1.f / l) : make_float2(0.f, 0.f);
}

// One thread per (sequence, KV head, visual key): sum over the head group's rows.
template <typename T>
__global__ void mass_generic_sum_kernel(const MassParams p) {
    const int hk = blockIdx.y % p.n_kv_heads, b = blockIdx.y / p.n_kv_heads;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int nv = p.n_visual[b], D = p.head_dim;
    if (j >= nv) return;
    const int pg = page_of(p.page_table, p.max_pages_per_seq, b, j / kPageSize);
    const T *k = (const T *)p.k_pages + (((size_t)pg * p.n_kv_heads + hk) * kPageSize + j % kPageSize) * D;
    const float2 *tb = p.table + (size_t)(b * p.n_kv_heads + hk) * p.r_tot;
    float acc = 0.f;
    for (int i = 0; i < p.l_txt; ++i)
        for (int g = 0; g < p.group; ++g) {
            const T *q = (const T *)p.q + (((size_t)b * p.l_txt + i) * p.n_q_heads + hk * p.group + g) * D;
            float a = 0.f;
            for (int d = 0; d < D; ++d) a = fmaf(to_float(q[d]), to_float(k[d]), a);
            const float2 t = tb[i * p.group + g];
            acc += expf(fmaf(a, p.scale, t.x)) * t.y;
        }
    p.colsum[(size_t)hk * p.sum_nv + p.offset[b] + j] = acc;
}

// ---- host side ---------------------------------------------------------------------------------------------------------
struct MassPlan {
    bool tc;
    int T, TG, RB, r_tot, stat_splits, sum_splits, max_nkt;
    size_t stats_off, table_off, colsum_off, total;
};

// Key splits for `items` equal work items of `tiles` key tiles each (every key tile costing `inner` accumulator
// tiles): the CTAs run one per SM in waves, so the cost is waves x (accumulator tiles per CTA + a fixed start-up).
static int mass_best_splits(int items, int tiles, int inner, int ctas_per_sm) {
    int best = 1;
    long long best_cost = -1;
    const int room = kNumSMs * ctas_per_sm;
    for (int s = 1; s <= tiles && s <= kMassMaxSplits; ++s) {
        const long long waves = ((long long)items * s + room - 1) / room;
        const long long cost = waves * ((long long)ceil_div(tiles, s) * inner + 4);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

static MassPlan mass_plan(int batch, const int32_t *n_visual, int l_txt, int n_q_heads, int n_kv_heads, int head_dim, int dtype) {
    MassPlan pl;
    const int G = n_q_heads / n_kv_heads;
    pl.r_tot = l_txt * G;
    pl.tc = dtype == HIPPO_DTYPE_BF16 && (head_dim == 64 || head_dim == 128) && G <= kMassTile && pl.r_tot <= kMassMaxRows;
    pl.T = G <= kMassTile ? kMassTile / G : 1;
    if (pl.T > l_txt) pl.T = l_txt;
    pl.TG = pl.T * G;
    pl.RB = ceil_div(l_txt, pl.T);
    long long sum_nv = 0;
    int max_nv = 0;
    for (int b = 0; b < batch; ++b) { sum_nv += n_visual[b]; if (n_visual[b] > max_nv) max_nv = n_visual[b]; }
    pl.max_nkt = ceil_div(max_nv > 0 ? max_nv : 1, kMassTile);
    const int units = batch * n_kv_heads;
    pl.stat_splits = pl.tc ? mass_best_splits(units * pl.RB, pl.max_nkt, 1, MassBuffers<0>::kCtasPerSm) : 1;
    pl.sum_splits = mass_best_splits(units, pl.max_nkt, pl.RB, MassBuffers<1>::kCtasPerSm);
    pl.stats_off = kWsHeaderBytes;
    pl.table_off = align_up(pl.stats_off + (size_t)units * pl.stat_splits * pl.r_tot * sizeof(float2), 256);
    pl.colsum_off = align_up(pl.table_off + (size_t)units * pl.r_tot * sizeof(float2), 256);
    pl.total = align_up(pl.colsum_off + (size_t)n_kv_heads * (size_t)sum_nv * sizeof(float), 256);
    return pl;
}

static int32_t make_q_map(CUtensorMap *m, const void *q, int batch, int l_txt, int n_q_heads, int D, int G, int T) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)n_q_heads, (cuuint64_t)l_txt, (cuuint64_t)batch};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)n_q_heads * D * 2, (cuuint64_t)l_txt * n_q_heads * D * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)T, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(q), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled (text queries) failed (%d)", (int)r);
    return HIPPO_OK;
}

static int32_t make_k_map(CUtensorMap *m, const void *pool, long long rows, int D) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)kPageSize};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(HIPPO_ERR_CUDA, "cuTensorMapEncodeTiled (keys) failed (%d)", (int)r);
    return HIPPO_OK;
}

template <int D>
static int32_t launch_mass_tc(MassParams &p, const MassPlan &pl, long long pool_rows, cudaStream_t s) {
    CUtensorMap km, qm;
    int32_t rc = make_k_map(&km, p.k_pages, pool_rows, D);
    if (rc != HIPPO_OK) return rc;
    rc = make_q_map(&qm, p.q, p.batch, p.l_txt, p.n_q_heads, D, p.group, pl.T);
    if (rc != HIPPO_OK) return rc;
    const size_t tile = (size_t)kMassTile * D * 2, fixed = 1024 + 2 * kMassSlices * kMassTile * sizeof(float2) + sizeof(MassShared) + 64;
    const size_t smem0 = fixed + (MassBuffers<0>::kRes + MassBuffers<0>::kSlots) * tile;
    const size_t smem1 = fixed + (MassBuffers<1>::kRes + MassBuffers<1>::kSlots) * tile +
                         (size_t)((p.r_tot + kMassSliceCols + 15) & ~15) * sizeof(float);
    static PerDeviceOnce attr_set;
    int dev;
    if (attr_set.needed(dev)) {
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(mass_tc_kernel<D, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        HIPPO_CUDA_TRY(cudaFuncSetAttribute(mass_tc_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr_set.mark(dev);
    }
    const int units = p.batch * p.n_kv_heads;
    p.splits = pl.stat_splits;
    mass_tc_kernel<D, 0><<<(unsigned)(units * pl.RB * pl.stat_splits), kMassThreads, smem0, s>>>(p, km, qm);
    HIPPO_CUDA_TRY(cudaGetLastError());
    const long long rows = (long long)units * p.r_tot;
    mass_merge_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, s>>>(p);
    HIPPO_CUDA_TRY(cudaGetLastError());
    p.splits = pl.sum_splits;
    mass_tc_kernel<D, 1><<<(unsigned)(units * pl.sum_splits), kMassThreads, smem1, s>>>(p, km, qm);
    HIPPO_CUDA_TRY(cudaGetLastError());
    count_launches(3);
    return HIPPO_OK;
}

template <typename T>
static int32_t launch_mass_generic(const MassParams &p, int max_nv, cudaStream_t s) {
    const long long rows = (long long)p.batch * p.n_q_heads * p.l_txt;
    mass_generic_stats_kernel<T><<<(unsigned)((rows * 32 + 255) / 256), 256, 0, s>>>(p);
    HIPPO_CUDA_TRY(cudaGetLastError());
    dim3 g((unsigned)ceil_div(max_nv, 128), (unsigned)(p.batch * p.n_kv_heads));
    mass_generic_sum_kernel<T><<<g, 128, 0, s>>>(p);
    HIPPO_CUDA_TRY(cudaGetLastError());
    count_launches(2);
    return HIPPO_OK;
}

}  // namespace hippo

using namespace hippo;

extern "C" size_t hippo_attention_mass_workspace_bytes(int32_t batch, const int32_t *n_visual, int32_t l_txt,
                                                       int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype) {
    if (batch <= 0 || batch > kMassMaxBatch || !n_visual || l_txt <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 ||
        n_q_heads % n_kv_heads || head_dim <= 0)
        return 0;
    for (int b = 0; b < batch; ++b) if (n_visual[b] < 0) return 0;
    return mass_plan(batch, n_visual, l_txt, n_q_heads, n_kv_heads, head_dim, dtype).total;
}

extern "C" int32_t hippo_attention_mass(int32_t batch, const int32_t *n_visual, int32_t l_txt, int32_t n_q_heads,
                                        const void *q_txt, const hippo_kv_cache_t *kv, float softmax_scale, float weight,
                                        float *mass, void *workspace, size_t workspace_bytes, void *stream) {
    const char *who = "hippo_attention_mass";
    if (!kv) return fail(HIPPO_ERR_INVALID_ARG, "%s: null kv cache descriptor", who);
    if (kv->struct_size != sizeof(hippo_kv_cache_t))
        return fail(HIPPO_ERR_INVALID_ARG, "%s: kv struct_size %u != %zu", who, kv->struct_size, sizeof(hippo_kv_cache_t));
    if (kv->dtype != HIPPO_DTYPE_FP32 && kv->dtype != HIPPO_DTYPE_BF16) return fail(HIPPO_ERR_INVALID_ARG, "%s: unknown dtype %d", who, kv->dtype);
    if (!kv->k_pages) return fail(HIPPO_ERR_INVALID_ARG, "%s: null key pool", who);
    if (kv->n_kv_heads <= 0 || kv->head_dim <= 0 || kv->n_pages <= 0 || kv->max_pages_per_seq <= 0)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: non-positive cache dimension", who);
    if ((uintptr_t)kv->k_pages & 127) return fail(HIPPO_ERR_INVALID_ARG, "%s: key pool must be 128-byte aligned", who);
    if (batch <= 0 || l_txt <= 0 || n_q_heads <= 0) return fail(HIPPO_ERR_INVALID_ARG, "%s: non-positive size", who);
    if (batch > kMassMaxBatch) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: batch %d > %d", who, batch, kMassMaxBatch);
    if (!n_visual || !q_txt || !mass || !workspace) return fail(HIPPO_ERR_INVALID_ARG, "%s: null pointer", who);
    if (n_q_heads % kv->n_kv_heads) return fail(HIPPO_ERR_INVALID_ARG, "%s: n_q_heads %% n_kv_heads != 0", who);
    if ((uintptr_t)q_txt & 15) return fail(HIPPO_ERR_INVALID_ARG, "%s: q_txt must be 16-byte aligned", who);
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale) || !isfinite(weight)) return fail(HIPPO_ERR_INVALID_ARG, "%s: bad scale or weight", who);
    long long sum_nv = 0;
    int max_nv = 0;
    for (int b = 0; b < batch; ++b) {
        if (n_visual[b] < 0) return fail(HIPPO_ERR_INVALID_ARG, "%s: n_visual[%d] < 0", who, b);
        if ((long long)n_visual[b] > (long long)kv->max_pages_per_seq * kPageSize)
            return fail(HIPPO_ERR_INVALID_ARG, "%s: n_visual[%d] exceeds max_pages_per_seq*%d", who, b, kPageSize);
        sum_nv += n_visual[b];
        if (n_visual[b] > max_nv) max_nv = n_visual[b];
    }
    if (sum_nv > 0x7fffffffLL / 4) return fail(HIPPO_ERR_UNSUPPORTED_SHAPE, "%s: too many visual tokens", who);
    if (!kv->page_table && (long long)batch * kv->max_pages_per_seq > kv->n_pages)
        return fail(HIPPO_ERR_INVALID_ARG, "%s: identity page mapping needs batch*max_pages_per_seq <= n_pages", who);
    const MassPlan pl = mass_plan(batch, n_visual, l_txt, n_q_heads, kv->n_kv_heads, kv->head_dim, kv->dtype);
    if (workspace_bytes < pl.total) return fail(HIPPO_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu bytes", who, workspace_bytes, pl.total);
    if ((uintptr_t)workspace & 255) return fail(HIPPO_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", who);
    if (sum_nv == 0) return HIPPO_OK;

    MassParams p;
    p.batch = batch; p.l_txt = l_txt; p.n_q_heads = n_q_heads; p.n_kv_heads = kv->n_kv_heads;
    p.group = n_q_heads / kv->n_kv_heads; p.head_dim = kv->head_dim;
    p.t_per_block = pl.T; p.rows_per_block = pl.TG; p.n_row_blocks = pl.RB; p.r_tot = pl.r_tot;
    p.splits = 1; p.stat_splits = pl.stat_splits; p.sum_nv = (int)sum_nv; p.max_pages_per_seq = kv->max_pages_per_seq;
    p.scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kv->head_dim);
    p.sl2 = p.scale * kMassLog2e;
    p.weight = weight;
    p.page_table = kv->page_table; p.q = q_txt; p.k_pages = kv->k_pages;
    p.stats = (float2 *)((char *)workspace + pl.stats_off);
    p.table = (float2 *)((char *)workspace + pl.table_off);
    p.table_log2 = (float *)p.table;
    p.colsum = (float *)((char *)workspace + pl.colsum_off);
    p.mass = mass;
    p.header = (WsHeader *)workspace;
    int off = 0;
    for (int b = 0; b < kMassMaxBatch; ++b) {
        p.n_visual[b] = b < batch ? n_visual[b] : 0;
        p.offset[b] = off;
        off += p.n_visual[b];
    }
    cudaStream_t s = (cudaStream_t)stream;
    int32_t rc;
    if (pl.tc) {
        const long long pool_rows = (long long)kv->n_pages * kv->n_kv_heads * kPageSize;
        rc = kv->head_dim == 128 ? launch_mass_tc<128>(p, pl, pool_rows, s) : launch_mass_tc<64>(p, pl, pool_rows, s);
    } else if (kv->dtype == HIPPO_DTYPE_FP32) {
        rc = launch_mass_generic<float>(p, max_nv, s);
    } else {
        rc = launch_mass_generic<__nv_bfloat16>(p, max_nv, s);
    }
    if (rc != HIPPO_OK) return rc;
    mass_reduce_kernel<<<(unsigned)((sum_nv + 255) / 256), 256, 0, s>>>(p);
    HIPPO_CUDA_TRY(cudaGetLastError());
    count_launches(1);
    return HIPPO_OK;
}
