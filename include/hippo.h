/*
 * hippo.h - C ABI of the B200 (sm_100a) hot path of one HIPPO video speculative-decoding step.
 *
 * Five operations, each a hand-written CUDA kernel family:
 *   hippo_select_tokens     semantic-aware visual-token preservation (Section 5.1, Eq. 3-7 + top-k)
 *   hippo_gather_kv         one-time pruning of the draft model's KV cache (Limitations (i))
 *   hippo_draft_attention   draft decode attention over the pruned KV (Section 3.2, drafting phase)
 *   hippo_verify_attention  target verification attention, gamma+1 query tokens (Section 3.2)
 *   hippo_accept            lossless speculative acceptance (Section 3.2, Eq. 1 and the resampling rule)
 * and, upstream of the selection, hippo_attention_mass (global semantic relevance, Section 5.1, Eq. 2).
 *
 * Conventions
 *   - Every call returns a hippo_status_t (0 = HIPPO_OK, negative = error).  Arguments are validated on the
 *     host before anything is enqueued; on an error nothing has been launched.
 *   - Pointers are DEVICE pointers unless the comment says "host".  The caller owns every buffer, including
 *     workspaces (size them with the *_workspace_bytes helpers; 256-byte aligned).  The library allocates
 *     no device memory.  Between calls it keeps a per-thread error string, cached kernel attributes, and - for
 *     hippo_accept_noalloc alone - a fixed scratch array in its image (HIPPO_ACCEPT_NOALLOC_SCRATCH_BYTES on every
 *     GPU that loads the library) with that array's cached address.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*) and the call returns without synchronising.
 *     Calls on different streams may overlap if they use different workspaces and outputs.
 *   - Device-side waits are bounded (2 s).  If one gives up, the kernel records it in the first word of the
 *     workspace, waits for its own copies and tensor-core work in flight, frees its tensor memory and exits;
 *     hippo_workspace_status() reports it after the stream has drained.  Results of that call are undefined.
 *   - dtype: HIPPO_DTYPE_FP32 or HIPPO_DTYPE_BF16 storage; accumulation is fp32 (attention) or fp64
 *     (selection scores, acceptance).
 */
#ifndef HIPPO_H_
#define HIPPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HIPPO_VERSION 101
#define HIPPO_PAGE_SIZE 64          /* tokens per KV page */
#define HIPPO_MAX_PACKED_ROWS 128   /* q_len * (n_q_heads / n_kv_heads) must not exceed this */

typedef enum hippo_status {
    HIPPO_OK = 0,
    HIPPO_ERR_INVALID_ARG = -1,         /* null pointer, negative size, inconsistent shapes */
    HIPPO_ERR_UNSUPPORTED_SHAPE = -2,   /* valid in principle, not built (e.g. head_dim not a multiple of 32) */
    HIPPO_ERR_WORKSPACE_TOO_SMALL = -3,
    HIPPO_ERR_CUDA = -4,                /* a CUDA runtime/driver call failed; see hippo_last_error() */
    HIPPO_ERR_TIMEOUT = -5,             /* a bounded device-side wait gave up (reported by hippo_workspace_status) */
    HIPPO_ERR_UNIMPLEMENTED = -6
} hippo_status_t;

typedef enum hippo_dtype { HIPPO_DTYPE_FP32 = 0, HIPPO_DTYPE_BF16 = 1 } hippo_dtype_t;

typedef enum hippo_accept_mode { HIPPO_ACCEPT_SAMPLE = 0, HIPPO_ACCEPT_GREEDY = 1 } hippo_accept_mode_t;
/* optional flags OR-ed into the mode of the sampling acceptance: force one of its two launch forms (same arithmetic, same
 * results; without a flag the library picks the faster one for the shape) */
#define HIPPO_ACCEPT_ONE_LAUNCH 16      /* one kernel, its CTAs meet at two counters in the workspace header */
#define HIPPO_ACCEPT_THREE_LAUNCHES 32  /* three chained kernels */

/* selection rules of hippo_select_tokens_policy */
typedef enum hippo_select_policy {
    HIPPO_SELECT_HOLISTIC = 0,            /* Section 5.1: the k best of the fused score over the whole sequence */
    HIPPO_SELECT_UNIFORM_PER_FRAME = 1,   /* the same budget for every frame, the best of the fused score inside each */
    HIPPO_SELECT_RANDOM = 2,              /* the k best by a caller-supplied random key per token */
    HIPPO_SELECT_FRAMES = 3               /* whole frames at a regular stride */
} hippo_select_policy_t;

/* score_mask bits for hippo_select_tokens (Eq. 7 sums the enabled terms) */
#define HIPPO_SCORE_ATTN 1u
#define HIPPO_SCORE_TEMP 2u
#define HIPPO_SCORE_SPA 4u
#define HIPPO_SCORE_ALL 7u

/*
 * Paged KV cache of ONE layer.  K and V are separate pools of fixed-size pages:
 *     k_pages, v_pages : [n_pages][n_kv_heads][HIPPO_PAGE_SIZE][head_dim]   (dtype elements, dense)
 * so one (page, head) block is a contiguous HIPPO_PAGE_SIZE x head_dim tile.  Token t of sequence b lives in
 * page  page_table[b * max_pages_per_seq + t / 64]  at slot  t % 64.  A contiguous cache is the special case
 * page_table == NULL, which means page id = b * max_pages_per_seq + t / 64.  Page ids must lie in
 * [0, n_pages); slots past a sequence's length may hold anything (they are never used).
 * Pools must be 128-byte aligned.
 */
typedef struct hippo_kv_cache {
    uint32_t struct_size;        /* sizeof(hippo_kv_cache_t), for versioning */
    int32_t dtype;               /* hippo_dtype_t */
    int32_t n_kv_heads;
    int32_t head_dim;
    int32_t n_pages;             /* pages in each pool */
    int32_t max_pages_per_seq;   /* row length of page_table */
    void *k_pages;
    void *v_pages;
    const int32_t *page_table;   /* device int32 [batch][max_pages_per_seq], or NULL for the identity mapping */
} hippo_kv_cache_t;

/* ---- helpers ------------------------------------------------------------------------------------------------ */

int32_t hippo_version(void);
const char *hippo_status_string(int32_t status);
/* Text of the last error raised on the calling host thread (empty string if none). */
const char *hippo_last_error(void);
/* Kernels launched by this library in this process so far (host-side counter, all threads). */
uint64_t hippo_launch_count(void);
/* Synchronises `stream`, then reads the status word that kernels keep in the first bytes of `workspace`:
 * HIPPO_OK, or HIPPO_ERR_TIMEOUT if a bounded device-side wait gave up since hippo_workspace_reset(). */
int32_t hippo_workspace_status(const void *workspace, void *stream);
/* Zeroes the header of a workspace (status word, wait limit and arrival counters); enqueued on `stream`.  Must be
 * called once on a fresh workspace before its first use by the attention calls, and after a reported time-out. */
int32_t hippo_workspace_reset(void *workspace, size_t workspace_bytes, void *stream);
/* Debugging aid: replaces the 2 s limit of the bounded device-side waits of the tensor-core attention and
 * attention-mass kernels that use this workspace by `limit_ns` nanoseconds (0 restores the default).  The waits that
 * guard a kernel's exit (its own copies and tensor-core work in flight) keep the 2 s limit.  Synchronises `stream`.
 * With a limit of a few microseconds a healthy kernel gives up on its first wait: this is how the time-out path
 * (status word, clean exit, reset) can be exercised without anything being stuck. */
int32_t hippo_workspace_set_wait_limit(void *workspace, int64_t limit_ns, void *stream);

/* Measurement aid (no counterpart in the paper): one pass of 16-byte loads over `bytes` bytes at `buffer`, summed into
 * `sink` (256 bytes of device memory, 256-byte aligned; contents are a checksum of no interest).  Timed by the caller,
 * it gives the bandwidth a read-only kernel reaches on this device, the natural ceiling of the attention kernels. */
int32_t hippo_read_probe(const void *buffer, size_t bytes, void *sink, void *stream);

/* ---- global semantic relevance: Section 5.1, Eq. 2 ------------------------------------------------------------ */
/*
 * The attention mass that hippo_select_tokens takes as `attn_mass`, from the prefilled target cache: for every
 * text query row i and attention head h, S_i = softmax over the VISUAL keys j < n_visual[b] of
 * scale * q_txt[b][i][h] . K[b][j][h / G]; Eq. 2 is the mean of [S_i]_j over layers, heads and text rows.
 * One call handles one layer and ADDS its share:
 *     mass[off_b + j] += weight * sum_{h, i} [S_i^(h)]_j        off_b = sum(n_visual[0..b))
 * so zeroing `mass` and calling once per layer with weight = 1 / (n_layers * n_q_heads * l_txt) yields Eq. 2.
 * The visual tokens are positions [0, n_visual[b]) of sequence b in the cache (text and generated tokens follow);
 * only the key pool is read.
 *   n_visual  host int32 [batch], each >= 0; batch <= 64      q_txt  [batch][l_txt][n_q_heads][head_dim], kv dtype
 *   softmax_scale  0 selects 1/sqrt(head_dim)                  mass   fp32 [sum n_visual], read and written
 * bf16 with head_dim 64 or 128 and l_txt * G <= 3072 runs on the tensor cores (logits formed twice, never stored);
 * other shapes and fp32 run on the CUDA cores.  Sums are added in a fixed order: results are reproducible.
 * The workspace needs no reset for this call unless a time-out was reported.
 */
size_t hippo_attention_mass_workspace_bytes(int32_t batch, const int32_t *n_visual, int32_t l_txt, int32_t n_q_heads,
                                            int32_t n_kv_heads, int32_t head_dim, int32_t dtype);
int32_t hippo_attention_mass(int32_t batch, const int32_t *n_visual, int32_t l_txt, int32_t n_q_heads,
                             const void *q_txt, const hippo_kv_cache_t *kv, float softmax_scale, float weight,
                             float *mass, void *workspace, size_t workspace_bytes, void *stream);

/* ---- selection: Section 5.1 --------------------------------------------------------------------------------- */
/*
 * For each of `batch` sequences scores its visual tokens and keeps the k best.
 *   Eq. 3-4  s_temp = 1 - mean cosine similarity with the same grid cell in the adjacent frames that contain it
 *   Eq. 5-6  s_spa  = population variance of the token's row of the crop's cosine-similarity matrix (diagonal 1);
 *            crops are crop_h x crop_w tiles anchored at the grid origin and clipped at the grid edge
 *   Eq. 7    fused = z(attn_mass) + z(s_spa) + z(s_temp), z = per-frame standardisation (population sigma;
 *            a frame with constant score contributes 0); only the terms enabled in score_mask are added
 *   top-k    over the whole sequence, ordered by (fused as fp32 descending, index ascending)
 * Layout: tokens are frame-major, row-major inside the grid_h x grid_w grid; a sequence whose length is not a
 * multiple of grid_h*grid_w has a partial last frame holding the first cells.  Sequences are concatenated:
 * sequence b starts at token offset sum(n_visual[0..b)).
 *   n_visual  host int32 [batch], each >= 1          k         host int32 [batch], 0 <= k[b] <= n_visual[b]
 *   embeds    [sum n_visual][embed_dim] dtype         attn_mass fp32 [sum n_visual]
 *   kept_idx  out int32: sequence b's k[b] indices (relative to its own start, ascending) are written at element
 *             offset kept_offsets[b]; kept_offsets (host int32 [batch]) may be NULL, meaning sum(k[0..b)).  Explicit
 *             offsets let the caller interleave other entries (e.g. always-kept text positions) in the same list.
 *   fused_score out fp32 [sum n_visual]
 * Scores are accumulated in fp64.  embed_dim must be a multiple of 8; crop_h*crop_w <= 32.
 */
size_t hippo_select_workspace_bytes(int32_t batch, const int32_t *n_visual, int32_t grid_h, int32_t grid_w,
                                    int32_t crop_h, int32_t crop_w);
int32_t hippo_select_tokens(int32_t batch, const int32_t *n_visual, int32_t grid_h, int32_t grid_w, int32_t crop_h,
                            int32_t crop_w, int32_t embed_dim, int32_t dtype, const void *embeds,
                            const float *attn_mass, const int32_t *k, const int32_t *kept_offsets,
                            uint32_t score_mask, int32_t *kept_idx, float *fused_score, void *workspace,
                            size_t workspace_bytes, void *stream);

/*
 * hippo_select_tokens under another selection rule.  The paper contrasts its holistic top-k with uniform pruning across
 * frames guided by the target's attention (related work on video speculative decoding) and, in its exploration of
 * pruning criteria (Section 6), with randomly sampled tokens and with whole frames dropped at regular temporal intervals;
 * it names these rules without spelling them out, so the definitions below are this library's reading.  Rules only:
 * the comparison systems themselves are not part of the library.
 *   HIPPO_SELECT_HOLISTIC           exactly hippo_select_tokens.
 *   HIPPO_SELECT_UNIFORM_PER_FRAME  the fused score as above (score_mask = HIPPO_SCORE_ATTN gives attention-guided uniform
 *                                   pruning); frame f of F keeps floor(k / F) tokens, the first k mod F frames one more;
 *                                   a frame with fewer tokens than its budget (a partial last frame) keeps them all and
 *                                   the shortfall goes, one token at a time in frame order, to frames that still have room;
 *                                   inside a frame the best by (fused as fp32 descending, index ascending).
 *   HIPPO_SELECT_RANDOM             random_keys (fp32 [sum n_visual], drawn by the caller) take the place of the fused
 *                                   score: the k best keys over the sequence, lower index first among equal keys.
 *                                   fused_score receives the keys.  embeds and attn_mass are not read and may be NULL.
 *   HIPPO_SELECT_FRAMES             with T = grid_h * grid_w, Fc = n_visual / T complete frames and m = ceil(k / T):
 *                                   frames floor(i * Fc / m), i = 0 .. m-1, whole, the last of them cut to its first cells
 *                                   when k is not a multiple of T; if k >= Fc * T (or Fc = 0) the first k tokens.
 *                                   Nothing is scored: embeds, attn_mass and fused_score are not touched and may be NULL.
 * All other arguments, the output order (ascending per sequence) and the workspace are those of hippo_select_tokens.
 */
int32_t hippo_select_tokens_policy(int32_t batch, const int32_t *n_visual, int32_t grid_h, int32_t grid_w, int32_t crop_h,
                                   int32_t crop_w, int32_t embed_dim, int32_t dtype, const void *embeds,
                                   const float *attn_mass, const int32_t *k, const int32_t *kept_offsets,
                                   uint32_t score_mask, int32_t policy, const float *random_keys, int32_t *kept_idx,
                                   float *fused_score, void *workspace, size_t workspace_bytes, void *stream);

/* ---- gather: pruning the draft KV cache (Limitations (i); the experimental set-up drops the pruned tokens'
 *      features from the draft model's input) ------------------------------------------------------------------- */
/*
 * For every layer l < n_layers, sequence b and i in [keep_offsets[b], keep_offsets[b+1]):
 *     dst token (i - keep_offsets[b]) of sequence b  :=  src token keep_idx[i] of sequence b      (K and V, all heads)
 * `src` / `dst` describe layer 0; layer l's pools start src_layer_stride_bytes * l (dst_layer_stride_bytes * l)
 * bytes further on.  Page tables are shared by all layers.  keep_idx holds positions in the source sequence
 * (the kept visual tokens and every always-kept position such as text), ascending per sequence to preserve
 * order; the kernel does not require ascending order.  src and dst must not overlap and must agree in dtype,
 * n_kv_heads and head_dim (head_dim * element size a multiple of 16 bytes).
 * Indices are read on the device and checked there before any address is formed from them: a source position
 * outside [0, src max_pages_per_seq * 64), a destination position beyond dst max_pages_per_seq * 64 (a sequence
 * keeping more than its destination holds), or a page id outside [0, n_pages) of its pool.  Such an entry is
 * skipped (nothing is read or written for it) and *bad_index is set to 1.  A source position inside the page
 * capacity but past the sequence's length copies whatever the slot holds.
 *   keep_idx      int32 [total_keep]          keep_offsets  int32 [batch + 1] (device), keep_offsets[0] = 0
 *   total_keep    host copy of keep_offsets[batch]; must not exceed batch * dst max_pages_per_seq * 64
 *   bad_index     optional device int32, zeroed by the caller; NULL: bad entries are skipped silently
 */
int32_t hippo_gather_kv(int32_t n_layers, const hippo_kv_cache_t *src, size_t src_layer_stride_bytes,
                        const hippo_kv_cache_t *dst, size_t dst_layer_stride_bytes, int32_t batch,
                        const int32_t *keep_idx, const int32_t *keep_offsets, int32_t total_keep,
                        int32_t *bad_index, void *stream);

/* ---- attention: Section 3.2 (drafting phase / verification phase) ------------------------------------------ */
/*
 * out[b][t][h] = softmax_j( scale * q[b][t][h] . K[b][j][h / G] ) V[b][j][h / G],   G = n_q_heads / n_kv_heads,
 * over the keys j <= kv_len[b] - q_len + t: the q_len query tokens are the LAST q_len positions of the
 * kv_len[b]-token context (their own K/V are already in the cache), every earlier key is visible.
 * The verification call is q_len = gamma + 1 rows against the full-length video cache, the draft call q_len = 1
 * against the short pruned cache.  Both names compute the same function for any q_len >= 1 and pick the kernel from
 * the shape: up to 8 packed rows over at most 1,024 keys run as one cluster of CTAs with a page each (latency-bound);
 * anything larger streams K/V tiles through one persistent CTA per SM.
 *   q        [batch][q_len][n_q_heads][head_dim] dtype        out  same shape and dtype as q
 *   kv_len   int32 [batch] (device), q_len <= kv_len[b] <= max_kv_len;  a sequence with kv_len[b] < q_len is skipped.
 *            NULL means the lengths are known on the host and all equal max_kv_len: the kernels then start their
 *            loads without the round trip for the length
 *   kv_len_host  optional HOST copy of kv_len (NULL: none).  Used only to plan the launch: with the real lengths of a
 *            ragged batch the work split is chosen from the total number of pages instead of batch * the longest;
 *            the kernels still read kv_len on the device, and results depend on it only through the order of the
 *            floating-point sums
 *   max_kv_len  host upper bound used to size the launch; <= max_pages_per_seq * 64
 *   softmax_scale  0 selects 1/sqrt(head_dim)
 *   num_splits  0 = automatic
 *   lse      optional fp32 [batch][q_len][n_q_heads], natural-log sum of exponentials of the scaled logits
 * bf16 with head_dim 64 or 128 runs on the tensor cores with TMA-staged tiles; fp32 (any head_dim that is a
 * multiple of 32, <= 256) runs on the CUDA cores.  q_len * G <= HIPPO_MAX_PACKED_ROWS.
 * The workspace header must have been zeroed once with hippo_workspace_reset().
 */
size_t hippo_attention_workspace_bytes(int32_t batch, int32_t q_len, int32_t n_q_heads, int32_t n_kv_heads,
                                       int32_t head_dim);
int32_t hippo_verify_attention(int32_t batch, int32_t q_len, int32_t n_q_heads, const void *q,
                               const hippo_kv_cache_t *kv, const int32_t *kv_len, const int32_t *kv_len_host,
                               int32_t max_kv_len, float softmax_scale, int32_t num_splits, void *out, float *lse,
                               void *workspace, size_t workspace_bytes, void *stream);
int32_t hippo_draft_attention(int32_t batch, int32_t q_len, int32_t n_q_heads, const void *q,
                              const hippo_kv_cache_t *kv, const int32_t *kv_len, const int32_t *kv_len_host,
                              int32_t max_kv_len, float softmax_scale, int32_t num_splits, void *out, float *lse,
                              void *workspace, size_t workspace_bytes, void *stream);

/*
 * The verification attention of SEVERAL layers in one launch (Section 3.2, verification phase; the target model's
 * verification pass runs this op once per layer over that layer's cache).  Same function as n_layers calls of
 * hippo_verify_attention:  out_layers[l] = attention(q_layers[l], kv_layers[l])  for l in [0, n_layers).
 * The persistent CTAs walk the layers: barriers, tensor memory and the work split are set up once, the loads of
 * layer l + 1 start while the softmax of layer l finishes, and the partial results of a layer are merged by a spare
 * warp of every CTA while the next layer streams, so no kernel boundary and no second kernel separate two layers.
 * All layers share batch, q_len, heads, head_dim, dtype, kv_len and the page table (kv_layers[l].page_table must be the
 * same pointer for every l, as must max_pages_per_seq; pools and n_pages may differ).
 *   q_layers, out_layers   HOST arrays [n_layers] of DEVICE pointers, each [batch][q_len][n_q_heads][head_dim]
 *   kv_layers              HOST array [n_layers] of descriptors
 *   lse_layers             NULL, or HOST array [n_layers] of DEVICE pointers (entries may be NULL)
 *   kv_len, kv_len_host, max_kv_len, softmax_scale   as for hippo_verify_attention
 *   max_ctas               0: one CTA per SM.  Otherwise an upper bound of the grid: the launch holds its SMs (all of their
 *                          shared memory) from the first layer to the last, so a caller that wants kernels of another
 *                          stream to run beside it - the draft model's, Section 5.2 - leaves them some SMs this way
 * The host arrays are read before the call returns.  The call enqueues one memset of its counters and one kernel
 * per 64 layers.  The workspace is larger than a single-layer one (three sets of partial-result slots and per-layer
 * counters): size it with hippo_verify_attention_layers_workspace_bytes.  bf16 with head_dim 64 or 128 and at most
 * 256 (sequence, kv head) units use the multi-layer kernel; every other shape is run layer by layer on the
 * single-layer paths, with the same results.  Because the CTAs of the launch wait for one another's partial results,
 * the grid never exceeds the number of SMs; the waits are bounded like every other.
 */
size_t hippo_verify_attention_layers_workspace_bytes(int32_t n_layers, int32_t batch, int32_t q_len, int32_t n_q_heads,
                                                     int32_t n_kv_heads, int32_t head_dim);
int32_t hippo_verify_attention_layers(int32_t n_layers, int32_t batch, int32_t q_len, int32_t n_q_heads,
                                      const void *const *q_layers, const hippo_kv_cache_t *kv_layers,
                                      const int32_t *kv_len, const int32_t *kv_len_host, int32_t max_kv_len,
                                      float softmax_scale, int32_t max_ctas, void *const *out_layers, float *const *lse_layers,
                                      void *workspace, size_t workspace_bytes, void *stream);

/* ---- acceptance: Section 3.2, Eq. 1 -------------------------------------------------------------------------- */
/*
 * Row alignment: target row j in [0, gamma] and draft row j in [0, gamma) both predict draft token x_{j+1};
 * target row gamma is the bonus row.  P_j, Q_j = softmax of the logit rows (temperature 1).
 *   for j = 0 .. gamma-1: accept x_{j+1} iff u_accept[j] * Q_j[x] < P_j[x]   (probability min(1, P/Q), Eq. 1)
 *   n = number accepted before the first rejection
 *   n < gamma : emit a token drawn from norm(max(0, P_n - Q_n));   n == gamma : from P_gamma
 *   the draw is the inverse CDF in ascending token id with u_resample[b]: smallest t with cumsum_t > u * total
 * Softmax normalisers, probabilities and CDFs are evaluated in fp64.
 * mode HIPPO_ACCEPT_GREEDY (the decoding mode of the paper's experiments, Appendix "More Details of Experiment
 * Setups"): x_{j+1} is kept iff it equals the arg-max of target row j (lowest token id on ties); the emitted token
 * is the arg-max of target row n.  draft_logits, u_accept and u_resample are not read and may be NULL.
 *   target_logits fp32 [batch][gamma+1][vocab]     draft_logits fp32 [batch][gamma][vocab]
 *   draft_tokens  int32 [batch][gamma]; a token outside [0, vocab) is never looked up and counts as rejected
 *   u_accept fp32 [batch][gamma]                    u_resample fp32 [batch]
 *   n_accepted    out int32 [batch]                 out_tokens out int32 [batch][gamma+1]: accepted draft tokens,
 *                                                   then the drawn token, then -1
 */
size_t hippo_accept_workspace_bytes(int32_t batch, int32_t gamma, int32_t vocab);
int32_t hippo_accept(int32_t batch, int32_t gamma, int32_t vocab, const float *target_logits,
                     const float *draft_logits, const int32_t *draft_tokens, const float *u_accept,
                     const float *u_resample, int32_t mode, int32_t *n_accepted, int32_t *out_tokens,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * hippo_accept for callers that cannot hand over a workspace.  (No counterpart in the paper: this is a packaging
 * variant of hippo_accept, same inputs, same outputs, same arithmetic, both modes.)
 *
 * Who needs it: code that reaches the acceptance step without any means of allocating device memory - a decode
 * loop whose memory was given in full to an engine's pool at start-up, a plug-in whose host forbids cudaMalloc
 * because it synchronises the device, glue code that holds only the logits.  The scratch that hippo_accept takes
 * from its `workspace` argument comes here from an array built into the library image:
 * HIPPO_ACCEPT_NOALLOC_SCRATCH_BYTES bytes of device memory on every GPU that loads libhippo.so, occupied until
 * the process exits whether or not this function is ever called.
 *
 *   - Nothing is allocated or freed, on the device or through any library, by this call.
 *   - Sizes whose scratch would not fit (hippo_accept_workspace_bytes(batch, gamma, vocab) >
 *     HIPPO_ACCEPT_NOALLOC_SCRATCH_BYTES) are refused with HIPPO_ERR_WORKSPACE_TOO_SMALL before anything is
 *     launched; hippo_last_error() gives both numbers.  The array covers batch 8, gamma 8 at a 152,064-entry
 *     vocabulary; larger problems must use hippo_accept.
 *   - The first call on each device looks up the array's device address (with that device current) and caches
 *     it.  Make that first call ahead of time, outside any stream capture.
 *   - All calls on one device share the one array and it keeps whatever the last call left in it.  The kernels
 *     overwrite every word before reading it, so no clearing is needed, but two calls that may run at the same
 *     time on the GPU (different streams without an ordering between them) race on it and corrupt each other's
 *     result.  Order them, or give one of them hippo_accept with its own workspace.
 */
#define HIPPO_ACCEPT_NOALLOC_SCRATCH_BYTES (1024u * 1024u)
int32_t hippo_accept_noalloc(int32_t batch, int32_t gamma, int32_t vocab, const float *target_logits,
                             const float *draft_logits, const int32_t *draft_tokens, const float *u_accept,
                             const float *u_resample, int32_t mode, int32_t *n_accepted, int32_t *out_tokens,
                             void *stream);

/* ---- decoding schedule: Section 5.2 (video parallel speculative decoding) -------------------------------------- */
/*
 * Host-only bookkeeping of the adaptive schedule; nothing here touches the GPU.  A round is planned, the caller
 * launches what the plan says on its draft and verification streams, reads the accepted count back and commits it.
 *   optimistic round   (previous batch accepted in full): verify the current batch (`verify_tokens` draft tokens,
 *                      q_len = verify_tokens + 1) WHILE drafting the next `draft_during` = gamma tokens.  All accepted:
 *                      the batch is emitted and the new tokens become the current batch.  Otherwise the accepted
 *                      tokens and the target's replacement are emitted, the new tokens are dropped, and the next
 *                      round is conservative.
 *   conservative round (after a rejection): draft x_1 first (`draft_before` = 1), then verify x_1 WHILE drafting
 *                      x_2..x_gamma (`draft_during` = gamma - 1).  x_1 rejected: stop drafting at once
 *                      (`abort_on_reject`), emit the replacement, stay conservative.  x_1 accepted: emit it; the
 *                      remaining tokens are the batch of an optimistic round (with gamma = 1 nothing remains: the
 *                      target's bonus token is emitted too and the mode stays conservative).
 * Synchronous draft-target prefill: the draft model keeps decoding while the target prefills;
 * hippo_vpsd_prefill_buffer gives floor((prefill_target - prefill_draft) / t_draft) tokens, and a non-empty buffer
 * handed to hippo_vpsd_init is the batch of a first optimistic round.
 * The paper gives the two modes in words only; the emission and hand-over rules above are this library's reading.
 */
typedef enum hippo_vpsd_mode { HIPPO_VPSD_OPTIMISTIC = 0, HIPPO_VPSD_CONSERVATIVE = 1 } hippo_vpsd_mode_t;

typedef struct hippo_vpsd_state {
    uint32_t struct_size;       /* set by hippo_vpsd_init */
    int32_t gamma;
    int32_t mode;               /* hippo_vpsd_mode_t of the next round */
    int32_t batch;              /* draft tokens waiting for verification at the start of the next round */
    int64_t rounds;             /* statistics since init */
    int64_t tokens_emitted;
    int64_t tokens_drafted;
    int64_t tokens_discarded;   /* drafted tokens that never reached the output */
} hippo_vpsd_state_t;

typedef struct hippo_vpsd_round {
    int32_t mode;
    int32_t draft_before;       /* draft tokens to produce before the verification starts */
    int32_t verify_tokens;      /* draft tokens the target verifies this round */
    int32_t draft_during;       /* draft tokens to produce while the target verifies */
    int32_t abort_on_reject;    /* 1: stop drafting as soon as the verdict is a rejection */
} hippo_vpsd_round_t;

typedef struct hippo_vpsd_outcome {
    int32_t accepted;           /* as committed */
    int32_t emitted;            /* tokens appended to the output this round */
    int32_t target_token;       /* 1: the last emitted token comes from the target (replacement or bonus) */
    int32_t keep_drafted;       /* how many of the tokens drafted during the round form the next batch */
    int32_t next_mode;
} hippo_vpsd_outcome_t;

/* All host pointers.  Status codes as everywhere; the two *_time functions return model time in the caller's unit. */
int32_t hippo_vpsd_prefill_buffer(double prefill_target, double prefill_draft, double t_draft);
int32_t hippo_vpsd_init(hippo_vpsd_state_t *state, int32_t gamma, int32_t buffered_tokens);
int32_t hippo_vpsd_plan(const hippo_vpsd_state_t *state, hippo_vpsd_round_t *round);
/* n_accepted in [0, verify_tokens]; drafted_during = tokens actually drafted beside the verification (less than
 * round->draft_during only after an abort). */
int32_t hippo_vpsd_commit(hippo_vpsd_state_t *state, const hippo_vpsd_round_t *round, int32_t n_accepted,
                          int32_t drafted_during, hippo_vpsd_outcome_t *outcome);
/* Duration of a round when one draft pass costs t_draft and one target pass t_target (the paper's latency
 * example, Section 4.2, uses the same two constants): max(t_target, draft_during * t_draft) after the
 * draft_before passes; a conservative round whose x_1 is rejected ends at the verdict. */
double hippo_vpsd_round_time(const hippo_vpsd_round_t *round, int32_t n_accepted, double t_draft, double t_target);
/* Serial speculative decoding for comparison: gamma draft passes, then one target pass (Section 4.2). */
double hippo_vpsd_serial_round_time(int32_t gamma, double t_draft, double t_target);

#ifdef __cplusplus
}
#endif
#endif /* HIPPO_H_ */
