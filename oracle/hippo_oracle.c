/*
 * CPU oracle for the HIPPO speculative-decoding hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, double-precision restatement of what the path computes, written from the paper's
 * definitions.  It shares no code with the CUDA library and must never be linked into, imported by or
 * executed from the product path; only the tests, the smoke check and the benchmark's CPU-baseline
 * leg call it.  No blocking, fusion or reordering beyond what the equations state; the only
 * concession to run time is an OpenMP "parallel for" over independent units (tokens, crops, rows,
 * sequences).
 *
 * Inputs are fp32 arrays holding the storage-rounded values (bf16 values widened exactly), so the
 * oracle and the GPU see identical numbers.  All arithmetic below is in double.
 *
 * Pin status (see the CPU test-suite):
 *   selection scores  - pinned by closed forms, invariants and a hand-worked case; the crop tiling,
 *                       the population sigma and the partial-last-frame rule are readings of the
 *                       paper, so parity with the authors' own code is unpinned.
 *   top-k, gather     - pinned (library sort / exact copy identities).
 *   attention         - pinned (library softmax-attention, closed forms).
 *   attention mass    - pinned (hand-worked case, closed forms, library softmax, invariants).
 *   acceptance        - pinned (losslessness identity by enumeration and by seeded simulation); the two
 *                       margins it reports are pinned by hand-worked cases and by the measured
 *                       decision boundaries.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------------------------------------
 * Selection: Section 5.1 "Semantic-aware Token Preservation", Eq. 3-7.
 * Tokens are frame-major, row-major inside the frame's grid_h x grid_w patch grid.  The last frame
 * may be partial: it then holds the first (n_visual mod grid_h*grid_w) cells.
 * ---------------------------------------------------------------------------------------------- */

static double dot_ff(const float *a, const float *b, int d) {
    double s = 0.0;
    for (int i = 0; i < d; ++i) s += (double)a[i] * (double)b[i];
    return s;
}

static int frame_tokens(int n_visual, int tpf, int f) {
    int left = n_visual - f * tpf;
    return left < tpf ? (left < 0 ? 0 : left) : tpf;
}

/* Per-frame standardisation (text below Eq. 6): s_hat = (s - mu_f) / sigma_f with the population
 * standard deviation.  A frame whose score is constant gets s_hat = 0. */
static void znorm_per_frame(const double *s, double *z, int n_visual, int tpf) {
    int F = (n_visual + tpf - 1) / tpf;
    for (int f = 0; f < F; ++f) {
        int n = frame_tokens(n_visual, tpf, f);
        const double *x = s + (size_t)f * tpf;
        double mu = 0.0;
        for (int i = 0; i < n; ++i) mu += x[i];
        mu /= n;
        double var = 0.0;
        for (int i = 0; i < n; ++i) var += (x[i] - mu) * (x[i] - mu);
        var /= n;
        double floor_ = 1e-24 * (mu * mu > 1.0 ? mu * mu : 1.0);
        if (var <= floor_) {
            for (int i = 0; i < n; ++i) z[(size_t)f * tpf + i] = 0.0;
        } else {
            double sd = sqrt(var);
            for (int i = 0; i < n; ++i) z[(size_t)f * tpf + i] = (x[i] - mu) / sd;
        }
    }
}

/* Eq. 3-4: s_temp = 1 - mean over the adjacent frames f' (those that exist and contain the cell)
 * of cos(v^f, v^f') at the same grid cell.  No neighbour, or a zero vector: cosine taken as 0. */
static void temporal_scores(int n_visual, int tpf, int d, const float *E, double *s_temp) {
    int F = (n_visual + tpf - 1) / tpf;
#pragma omp parallel for schedule(dynamic, 16)
    for (int j = 0; j < n_visual; ++j) {
        int f = j / tpf, c = j % tpf;
        const float *v = E + (size_t)j * d;
        double nv = sqrt(dot_ff(v, v, d));
        double sum = 0.0;
        int cnt = 0;
        for (int df = -1; df <= 1; df += 2) {
            int g = f + df;
            if (g < 0 || g >= F) continue;
            if (c >= frame_tokens(n_visual, tpf, g)) continue;
            const float *w = E + ((size_t)g * tpf + c) * d;
            double nw = sqrt(dot_ff(w, w, d));
            double cs = (nv > 0.0 && nw > 0.0) ? dot_ff(v, w, d) / (nv * nw) : 0.0;
            sum += cs;
            ++cnt;
        }
        double sp = cnt ? sum / cnt : 0.0;
        s_temp[j] = 1.0 - sp;
    }
}

/* Eq. 5-6: per crop of M tokens, S = E_hat E_hat^T on L2-normalised embeddings (diagonal exactly 1);
 * s_spa(j) = (1/M) sum_k (S_jk - mu_j)^2, mu_j = (1/M) sum_k S_jk, both sums including k = j.
 * Crops are non-overlapping crop_h x crop_w tiles anchored at the grid origin, clipped at the grid
 * edge and at the end of a partial frame; M is the number of tokens actually in the crop. */
static void spatial_scores(int n_visual, int gh, int gw, int ch, int cw, int d, const float *E, double *s_spa) {
    int tpf = gh * gw;
    int F = (n_visual + tpf - 1) / tpf;
    int cy = (gh + ch - 1) / ch, cx = (gw + cw - 1) / cw;
    int n_crops = F * cy * cx;
    int Mmax = ch * cw;
#pragma omp parallel
    {
        double *Eh = (double *)malloc((size_t)Mmax * d * sizeof(double));
        double *S = (double *)malloc((size_t)Mmax * Mmax * sizeof(double));
        int *tok = (int *)malloc((size_t)Mmax * sizeof(int));
#pragma omp for schedule(dynamic, 1)
        for (int c = 0; c < n_crops; ++c) {
            int f = c / (cy * cx), r = c % (cy * cx);
            int y0 = (r / cx) * ch, x0 = (r % cx) * cw;
            int nf = frame_tokens(n_visual, tpf, f);
            int M = 0;
            for (int y = y0; y < y0 + ch && y < gh; ++y)
                for (int x = x0; x < x0 + cw && x < gw; ++x)
                    if (y * gw + x < nf) tok[M++] = f * tpf + y * gw + x;
            for (int a = 0; a < M; ++a) {
                const float *v = E + (size_t)tok[a] * d;
                double nv = sqrt(dot_ff(v, v, d));
                for (int i = 0; i < d; ++i) Eh[(size_t)a * d + i] = nv > 0.0 ? (double)v[i] / nv : 0.0;
            }
            for (int a = 0; a < M; ++a)
                for (int b = 0; b < M; ++b) {
                    if (a == b) { S[a * Mmax + b] = 1.0; continue; }
                    double s = 0.0;
                    for (int i = 0; i < d; ++i) s += Eh[(size_t)a * d + i] * Eh[(size_t)b * d + i];
                    S[a * Mmax + b] = s;
                }
            for (int a = 0; a < M; ++a) {
                double mu = 0.0;
                for (int b = 0; b < M; ++b) mu += S[a * Mmax + b];
                mu /= M;
                double var = 0.0;
                for (int b = 0; b < M; ++b) var += (S[a * Mmax + b] - mu) * (S[a * Mmax + b] - mu);
                s_spa[tok[a]] = var / M;
            }
        }
        free(Eh); free(S); free(tok);
    }
}

/* Eq. 7: fused = z(attn) + z(spa) + z(temp); score_mask bit0 = attn, bit1 = temp, bit2 = spa.
 * Outputs (each [n_visual], any may be NULL except fused): raw s_temp, s_spa and the fused score. */
int oracle_select_scores(int n_visual, int grid_h, int grid_w, int crop_h, int crop_w, int d,
                         const float *embeds, const float *attn_mass, unsigned score_mask,
                         double *s_temp_out, double *s_spa_out, double *fused) {
    if (n_visual <= 0 || grid_h <= 0 || grid_w <= 0 || crop_h <= 0 || crop_w <= 0 || d <= 0 || !fused) return -1;
    int tpf = grid_h * grid_w;
    double *raw = (double *)malloc((size_t)n_visual * sizeof(double));
    double *z = (double *)malloc((size_t)n_visual * sizeof(double));
    if (!raw || !z) { free(raw); free(z); return -2; }
    for (int j = 0; j < n_visual; ++j) fused[j] = 0.0;
    if (score_mask & 1u) {
        for (int j = 0; j < n_visual; ++j) raw[j] = (double)attn_mass[j];
        znorm_per_frame(raw, z, n_visual, tpf);
        for (int j = 0; j < n_visual; ++j) fused[j] += z[j];
    }
    if ((score_mask & 4u) || s_spa_out) {
        spatial_scores(n_visual, grid_h, grid_w, crop_h, crop_w, d, embeds, raw);
        if (s_spa_out) memcpy(s_spa_out, raw, (size_t)n_visual * sizeof(double));
        if (score_mask & 4u) {
            znorm_per_frame(raw, z, n_visual, tpf);
            for (int j = 0; j < n_visual; ++j) fused[j] += z[j];
        }
    }
    if ((score_mask & 2u) || s_temp_out) {
        temporal_scores(n_visual, tpf, d, embeds, raw);
        if (s_temp_out) memcpy(s_temp_out, raw, (size_t)n_visual * sizeof(double));
        if (score_mask & 2u) {
            znorm_per_frame(raw, z, n_visual, tpf);
            for (int j = 0; j < n_visual; ++j) fused[j] += z[j];
        }
    }
    free(raw); free(z);
    return 0;
}

/* "retain the top-k visual tokens" (end of Section 5.1): the k best over the whole sequence, ordered by
 * (score descending, index ascending); indices returned ascending.  *kth_score = score of the worst
 * kept token (the threshold). */
typedef struct { double s; int32_t i; } scored_t;
static int cmp_scored(const void *a, const void *b) {
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);
}
static int cmp_i32(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}
int oracle_topk(int n, const double *score, int k, int32_t *kept_idx, double *kth_score) {
    if (n < 0 || k < 0 || k > n) return -1;
    scored_t *t = (scored_t *)malloc((size_t)(n > 0 ? n : 1) * sizeof(scored_t));
    if (!t) return -2;
    for (int i = 0; i < n; ++i) { t[i].s = score[i]; t[i].i = i; }
    qsort(t, (size_t)n, sizeof(scored_t), cmp_scored);
    for (int i = 0; i < k; ++i) kept_idx[i] = t[i].i;
    if (kth_score) *kth_score = k > 0 ? t[k - 1].s : INFINITY;
    qsort(kept_idx, (size_t)k, sizeof(int32_t), cmp_i32);
    free(t);
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Other selection rules, for comparison with the holistic rule above.  The paper names them without
 * spelling them out: uniform pruning across all frames (related work, the attention-guided selection
 * of an earlier video speculative-decoding method), randomly sampled tokens and whole frames dropped at
 * regular temporal intervals (Section 6, exploration of pruning criteria).  The readings taken:
 *   policy 0  holistic    the k best over the whole sequence (oracle_topk).
 *   policy 1  per frame   every frame gets the same budget: floor(k / F) tokens, the first k mod F frames
 *                         one more; a frame that holds fewer tokens than its budget (a partial last
 *                         frame) keeps them all and the shortfall goes, one token at a time in frame
 *                         order, to the frames that still have room.  Inside a frame the best tokens by
 *                         (score descending, index ascending).
 *   policy 2  random      the k best by a caller-supplied key per token (the caller draws the keys): the
 *                         same rule as policy 0 with the keys as scores.
 *   policy 3  frames      whole frames at a regular stride: with m = ceil(k / T) frames to keep out of the
 *                         Fc complete frames (T tokens each), frame floor(i * Fc / m) for i = 0..m-1; when k
 *                         is not a multiple of T the last kept frame gives only its first cells.  If k
 *                         reaches Fc * T (or there is no complete frame) the complete frames are all kept
 *                         and the rest comes from the first cells of the partial frame.
 * score: [n] (ignored by policy 3).  frame_budget (may be NULL): [F] tokens kept per frame, for policy 1.
 * ---------------------------------------------------------------------------------------------- */
int oracle_select_policy(int policy, int n, int tokens_per_frame, const double *score, int k, int32_t *kept_idx,
                         int32_t *frame_budget) {
    if (n <= 0 || tokens_per_frame <= 0 || k < 0 || k > n) return -1;
    int T = tokens_per_frame, F = (n + T - 1) / T;
    if (policy == 0 || policy == 2) return oracle_topk(n, score, k, kept_idx, NULL);
    if (policy == 1) {
        int *budget = (int *)malloc((size_t)F * sizeof(int));
        if (!budget) return -2;
        int given = 0;
        for (int f = 0; f < F; ++f) {
            int want = k / F + (f < k % F ? 1 : 0), have = frame_tokens(n, T, f);
            budget[f] = want < have ? want : have;
            given += budget[f];
        }
        while (given < k)
            for (int f = 0; f < F && given < k; ++f)
                if (budget[f] < frame_tokens(n, T, f)) { ++budget[f]; ++given; }
        int out = 0;
        for (int f = 0; f < F; ++f) {
            int have = frame_tokens(n, T, f);
            int rc = oracle_topk(have, score + (size_t)f * T, budget[f], kept_idx + out, NULL);
            if (rc != 0) { free(budget); return rc; }
            for (int i = 0; i < budget[f]; ++i) kept_idx[out + i] += f * T;
            out += budget[f];
            if (frame_budget) frame_budget[f] = budget[f];
        }
        free(budget);
        return 0;
    }
    if (policy == 3) {
        int Fc = n / T, out = 0;
        if (Fc == 0 || (long)k >= (long)Fc * T) {
            for (int i = 0; i < k; ++i) kept_idx[i] = i;      /* all complete frames, then the first cells of the rest */
            return 0;
        }
        int m = (k + T - 1) / T;
        for (int i = 0; i < m; ++i) {
            int f = (int)((long)i * Fc / m);
            int take = k - out < T ? k - out : T;
            for (int c = 0; c < take; ++c) kept_idx[out++] = f * T + c;
        }
        return 0;
    }
    return -1;
}

/* ------------------------------------------------------------------------------------------------
 * Gather: "one-time pruning of the draft model's KV cache" (Limitations (i)); removing the pruned
 * video features (experimental set-up).  dst[l][i][h][:] = src[l][keep[i]][h][:].
 * src [n_layers][n_src][row], dst [n_layers][n_keep][row], row = h_kv * d_h elements of elem_bytes.
 * ---------------------------------------------------------------------------------------------- */
int oracle_gather_kv(int n_layers, int n_src, int n_keep, int row_bytes, const int32_t *keep,
                     const unsigned char *src, unsigned char *dst) {
    for (int i = 0; i < n_keep; ++i)
        if (keep[i] < 0 || keep[i] >= n_src) return -1;
    for (int l = 0; l < n_layers; ++l)
        for (int i = 0; i < n_keep; ++i)
            memcpy(dst + ((size_t)l * n_keep + i) * row_bytes, src + ((size_t)l * n_src + keep[i]) * row_bytes,
                   (size_t)row_bytes);
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Attention (draft decode and target verification, Section 3.2): softmax(q K^T * scale) V under
 * grouped-query attention, query head h reading KV head h / (H_q / H_kv).  The q_len query rows are
 * the last q_len positions of the kv_len-long context: row t sees keys j <= kv_len - q_len + t.
 * q [B][q_len][H_q][D]; k, v [B][max_kv][H_kv][D]; out double [..][D]; lse natural-log.
 * ---------------------------------------------------------------------------------------------- */
static void attention_row(int b, int t, int h, int q_len, int Hq, int Hkv, int D, int max_kv, int kv_len,
                          const float *q, const float *k, const float *v, double scale, double *out, double *lse) {
    int G = Hq / Hkv, hk = h / G;
    int n = kv_len - q_len + t + 1;
    if (n <= 0) {
        for (int i = 0; i < D; ++i) out[i] = 0.0;
        if (lse) *lse = -INFINITY;
        return;
    }
    const float *qr = q + (((size_t)b * q_len + t) * Hq + h) * D;
    double *a = (double *)malloc((size_t)n * sizeof(double));
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        const float *kr = k + (((size_t)b * max_kv + j) * Hkv + hk) * D;
        a[j] = scale * dot_ff(qr, kr, D);
        if (a[j] > m) m = a[j];
    }
    double l = 0.0;
    for (int j = 0; j < n; ++j) { a[j] = exp(a[j] - m); l += a[j]; }
    for (int i = 0; i < D; ++i) out[i] = 0.0;
    for (int j = 0; j < n; ++j) {
        const float *vr = v + (((size_t)b * max_kv + j) * Hkv + hk) * D;
        double p = a[j] / l;
        for (int i = 0; i < D; ++i) out[i] += p * (double)vr[i];
    }
    if (lse) *lse = m + log(l);
    free(a);
}

int oracle_attention(int B, int q_len, int Hq, int Hkv, int D, int max_kv, const int32_t *kv_len,
                     const float *q, const float *k, const float *v, double scale, double *out, double *lse) {
    if (B <= 0 || q_len <= 0 || Hkv <= 0 || Hq % Hkv || D <= 0) return -1;
    long total = (long)B * q_len * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < total; ++r) {
        int h = (int)(r % Hq), t = (int)((r / Hq) % q_len), b = (int)(r / ((long)Hq * q_len));
        attention_row(b, t, h, q_len, Hq, Hkv, D, max_kv, kv_len[b], q, k, v, scale, out + (size_t)r * D,
                      lse ? lse + r : NULL);
    }
    return 0;
}

/* The same definition for a chosen list of (b, t, h) rows only (spot checks at full problem size). */
int oracle_attention_rows(int n_sel, const int32_t *sel_b, const int32_t *sel_t, const int32_t *sel_h, int q_len,
                          int Hq, int Hkv, int D, int max_kv, const int32_t *kv_len, const float *q, const float *k,
                          const float *v, double scale, double *out, double *lse) {
    if (q_len <= 0 || Hkv <= 0 || Hq % Hkv || D <= 0) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_sel; ++r)
        attention_row(sel_b[r], sel_t[r], sel_h[r], q_len, Hq, Hkv, D, max_kv, kv_len[sel_b[r]], q, k, v, scale,
                      out + (size_t)r * D, lse ? lse + r : NULL);
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Global semantic relevance (Section 5.1, Eq. 2).  For every layer l, attention head h and text query
 * row i the cross-modal attention row is S_i = softmax over the N_v visual keys of scale * q_i . k_j
 * (head h reads KV head h / (H_q / H_kv)); the score of visual token j is the mean of [S]_ij over
 * layers, heads and text rows.  The softmax runs over the visual keys only: S_attn is defined as an
 * L_txt x N_v matrix.
 * q_txt [n_layers][B][L_txt][H_q][D]; k_vid [n_layers][B][max_nv][H_kv][D]; n_visual [B];
 * mass double [B][max_nv] (entries at and beyond n_visual[b] are set to 0).
 * ---------------------------------------------------------------------------------------------- */
int oracle_attention_mass(int n_layers, int B, int L_txt, int Hq, int Hkv, int D, int max_nv, const int32_t *n_visual,
                          const float *q_txt, const float *k_vid, double scale, double *mass) {
    if (n_layers <= 0 || B <= 0 || L_txt <= 0 || Hkv <= 0 || Hq % Hkv || D <= 0 || max_nv <= 0) return -1;
    int G = Hq / Hkv;
    double *head_sum = (double *)malloc((size_t)Hq * max_nv * sizeof(double));   /* sum over text rows, one head */
    if (!head_sum) return -2;
    for (size_t x = 0; x < (size_t)B * max_nv; ++x) mass[x] = 0.0;
    for (int b = 0; b < B; ++b) {
        int nv = n_visual[b];
        if (nv <= 0) continue;
        if (nv > max_nv) { free(head_sum); return -1; }
        for (int l = 0; l < n_layers; ++l) {
            const float *ql = q_txt + ((size_t)l * B + b) * L_txt * Hq * D;
            const float *kl = k_vid + ((size_t)l * B + b) * max_nv * Hkv * D;
#pragma omp parallel for schedule(dynamic, 1)
            for (int h = 0; h < Hq; ++h) {
                int hk = h / G;
                double *acc = head_sum + (size_t)h * max_nv;
                double *a = (double *)malloc((size_t)nv * sizeof(double));
                for (int j = 0; j < nv; ++j) acc[j] = 0.0;
                for (int i = 0; i < L_txt; ++i) {
                    const float *qr = ql + ((size_t)i * Hq + h) * D;
                    double m = -INFINITY, z = 0.0;
                    for (int j = 0; j < nv; ++j) {
                        a[j] = scale * dot_ff(qr, kl + ((size_t)j * Hkv + hk) * D, D);
                        if (a[j] > m) m = a[j];
                    }
                    for (int j = 0; j < nv; ++j) { a[j] = exp(a[j] - m); z += a[j]; }
                    for (int j = 0; j < nv; ++j) acc[j] += a[j] / z;
                }
                free(a);
            }
            for (int h = 0; h < Hq; ++h)
                for (int j = 0; j < nv; ++j) mass[(size_t)b * max_nv + j] += head_sum[(size_t)h * max_nv + j];
        }
        for (int j = 0; j < nv; ++j) mass[(size_t)b * max_nv + j] /= (double)n_layers * Hq * L_txt;
    }
    free(head_sum);
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Speculative acceptance (Section 3.2, Eq. 1 and the resampling rule below it).
 * Row alignment: target row j in [0, gamma] and draft row j in [0, gamma) both predict draft token
 * x_{j+1}; target row gamma is the bonus row.  P_j, Q_j = softmax of the logit rows.
 *   accept x_{j+1} with probability min(1, P_j[x]/Q_j[x]): tested as u_acc[j] * Q_j[x] < P_j[x];
 *   first rejection at n: draw from norm(max(0, P_n - Q_n)); none: draw the bonus token from P_gamma.
 * The draw is an inverse CDF in ascending token id with the single uniform u_res: the smallest t with
 * sum_{t'<=t} w_t' > u_res * Z.
 * target_logits [B][gamma+1][V], draft_logits [B][gamma][V], draft_tokens [B][gamma],
 * n_accepted [B], out_tokens [B][gamma+1] (unused tail = -1).
 * margin_accept[b]: min over the tests made of |u*Q - P| / P;  margin_cdf[b]: distance of u_res*Z to the
 * nearer edge of the chosen token's CDF interval, relative to Z.  Either may be NULL.
 * ---------------------------------------------------------------------------------------------- */
static void softmax_row(const float *logit, int V, double *p) {
    double m = -INFINITY;
    for (int t = 0; t < V; ++t) if ((double)logit[t] > m) m = (double)logit[t];
    double z = 0.0;
    for (int t = 0; t < V; ++t) { p[t] = exp((double)logit[t] - m); z += p[t]; }
    for (int t = 0; t < V; ++t) p[t] /= z;
}

int oracle_accept(int B, int gamma, int V, const float *target_logits, const float *draft_logits,
                  const int32_t *draft_tokens, const float *u_accept, const float *u_resample, int32_t *n_accepted,
                  int32_t *out_tokens, double *margin_accept, double *margin_cdf) {
    if (B <= 0 || gamma < 0 || V <= 0) return -1;
    for (long i = 0; i < (long)B * gamma; ++i)
        if (draft_tokens[i] < 0 || draft_tokens[i] >= V) return -1;
#pragma omp parallel
    {
        double *P = (double *)malloc((size_t)V * sizeof(double));
        double *Q = (double *)malloc((size_t)V * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (int b = 0; b < B; ++b) {
            const float *tl = target_logits + (size_t)b * (gamma + 1) * V;
            const float *dl = draft_logits + (size_t)b * gamma * V;
            const int32_t *x = draft_tokens + (size_t)b * gamma;
            int32_t *out = out_tokens + (size_t)b * (gamma + 1);
            for (int j = 0; j <= gamma; ++j) out[j] = -1;
            double mg = INFINITY;
            int n = 0;
            for (; n < gamma; ++n) {
                softmax_row(tl + (size_t)n * V, V, P);
                softmax_row(dl + (size_t)n * V, V, Q);
                double u = (double)u_accept[(size_t)b * gamma + n];
                double lhs = u * Q[x[n]], rhs = P[x[n]];
                double rel = rhs > 0.0 ? fabs(lhs - rhs) / rhs : INFINITY;
                if (rel < mg) mg = rel;
                if (!(lhs < rhs)) break; /* rejected: P and Q now hold row n */
                out[n] = x[n];
            }
            double z = 0.0;
            if (n < gamma) {
                for (int t = 0; t < V; ++t) { double w = P[t] - Q[t]; Q[t] = w > 0.0 ? w : 0.0; z += Q[t]; }
                if (!(z > 0.0)) { for (int t = 0; t < V; ++t) { Q[t] = P[t]; } z = 0.0; for (int t = 0; t < V; ++t) z += Q[t]; }
            } else {
                softmax_row(tl + (size_t)gamma * V, V, Q);
                for (int t = 0; t < V; ++t) z += Q[t];
            }
            double target = (double)u_resample[b] * z, cum = 0.0, prev = 0.0;
            int tok = -1, last_pos = -1;
            for (int t = 0; t < V; ++t) {
                if (Q[t] > 0.0) last_pos = t;
                prev = cum;
                cum += Q[t];
                if (cum > target) { tok = t; break; }
            }
            if (tok < 0) { tok = last_pos; prev = cum; }
            out[n] = tok;
            n_accepted[b] = n;
            if (margin_accept) margin_accept[b] = mg;
            if (margin_cdf) {
                double lo = fabs(target - prev), hi = fabs(cum - target);
                margin_cdf[b] = (lo < hi ? lo : hi) / z;
            }
        }
        free(P); free(Q);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------------
 * Greedy verification: the decoding mode of the paper's experiments (Appendix "More Details of
 * Experiment Setups": answers are generated "following greedy decoding").  With greedy decoding the
 * target's token at a position is the arg-max of its logit row, so a draft token is kept iff it
 * equals that arg-max; at the first mismatch n the target's own arg-max is emitted instead, and if all
 * gamma tokens match, the arg-max of the bonus row gamma.  Ties: the lowest token id.  No uniforms.
 * ---------------------------------------------------------------------------------------------- */
int oracle_accept_greedy(int B, int gamma, int V, const float *target_logits, const int32_t *draft_tokens,
                         int32_t *n_accepted, int32_t *out_tokens) {
    if (B <= 0 || gamma < 0 || V <= 0) return -1;
    for (int b = 0; b < B; ++b) {
        const float *tl = target_logits + (size_t)b * (gamma + 1) * V;
        int32_t *out = out_tokens + (size_t)b * (gamma + 1);
        for (int j = 0; j <= gamma; ++j) out[j] = -1;
        int n = 0;
        for (;;) {
            const float *row = tl + (size_t)n * V;
            int best = 0;
            for (int t = 1; t < V; ++t) if (row[t] > row[best]) best = t;
            if (n < gamma && draft_tokens[(size_t)b * gamma + n] == best) { out[n] = best; ++n; continue; }
            out[n] = best;
            break;
        }
        n_accepted[b] = n;
    }
    return 0;
}
