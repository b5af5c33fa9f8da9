/*
 * CPU oracle for the prefill-stage dual-attention vision-token filter of MustDrop
 * (arXiv 2411.10803, Sec. 3.4 "Dual-Attention Filtering Guided by Language").
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the filter
 * computes, written from the paper's equations.  It shares no code with the CUDA library
 * and must never sit on a product path: only tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it.
 *
 * Arithmetic: bf16 inputs are converted exactly to double; logits, softmax, head mean,
 * column sum and column max run in double and are rounded once to fp32.  The selection
 * arithmetic (dual criteria -> one score per token) runs in fp32, one IEEE operation per
 * step, because it decides integers (which tokens are kept) and the kernel takes the same
 * decision in fp32.
 *
 * Pins (tests/test_oracle_*.py): softmax rows sum to one; an independent float64
 * restatement with a library softmax; closed forms (identical keys -> harmonic numbers,
 * one dominant key); rank-one logits with a hand-computed softmax; inequalities and
 * permutation equivariances; brute-force subset enumeration, nesting, pairwise order and
 * mode equivalence for the selection; identity compaction.
 * Parity unpinned (the paper prints no values for them): the default thresholds
 * gamma = 1/M and alpha = 2/L, and the exact-budget rule, which are readings of the text.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Text-row attention map of ONE request (Eq. 1 restricted to the text queries).
 *   q_text [H][N][D], k [H][L][D] as bf16 bits.
 *   z[h][i][l] = scale * sum_d q[h][i][d] * k[h][l][d]
 *   visible(i,l) = !causal || l <= txt_start + i   (the model's own prefill mask; the text
 *                  query i sits at sequence position txt_start + i, Sec. 3.1 "Prefilling")
 *   p[h][i][l]  = softmax over the visible l; 0 where not visible.
 * p_out [H][N][L] doubles.  Returns 0, or -1 on a bad argument.
 */
int mustdrop_oracle_attention(const uint16_t *q_text, const uint16_t *k, int H, int N, int L, int D,
                              int txt_start, int causal, double scale, double *p_out)
{
    if (!q_text || !k || !p_out || H <= 0 || N <= 0 || L <= 0 || D <= 0) return -1;
    if (scale == 0.0) scale = 1.0 / sqrt((double)D);
    double *z = (double *)malloc(sizeof(double) * (size_t)L);
    if (!z) return -1;
    for (int h = 0; h < H; ++h) {
        for (int i = 0; i < N; ++i) {
            const uint16_t *qrow = q_text + ((size_t)h * N + i) * D;
            int last = causal ? txt_start + i : L - 1; /* last visible key */
            if (last > L - 1) last = L - 1;
            double zmax = -INFINITY;
            for (int l = 0; l <= last; ++l) {
                const uint16_t *krow = k + ((size_t)h * L + l) * D;
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
                z[l] = scale * acc;
                if (z[l] > zmax) zmax = z[l];
            }
            double denom = 0.0;
            for (int l = 0; l <= last; ++l) denom += exp(z[l] - zmax);
            double *prow = p_out + ((size_t)h * N + i) * L;
            for (int l = 0; l < L; ++l) prow[l] = (l <= last) ? exp(z[l] - zmax) / denom : 0.0;
        }
    }
    free(z);
    return 0;
}

/*
 * Importance scores of a batch (Eq. 8 and Eq. 10 on the head-averaged text->vision attention).
 *   a[i][j] = (1/H) sum_h p[h][i][vis_start + j]          one scalar per (text, vision) pair
 *   G[j]    = sum_{i<N} a[i][j]                            Eq. 8 (the paper's V_j)
 *   I[j]    = max_{i<N} a[i][j]                            Eq. 10, max over the text tokens
 * q_text [B][H][N][D], k [B][H][L][D] bf16 bits; g_out, i_out fp32 [B][M];
 * a_out nullable, double [B][N][M].
 */
int mustdrop_oracle_score(const uint16_t *q_text, const uint16_t *k, int B, int H, int N, int L, int D,
                          int vis_start, int M, int txt_start, int causal, double scale,
                          float *g_out, float *i_out, double *a_out)
{
    if (!q_text || !k || !g_out || !i_out) return -1;
    if (B <= 0 || M <= 0 || vis_start < 0 || vis_start + M > txt_start || txt_start + N > L) return -1;
    double *p = (double *)malloc(sizeof(double) * (size_t)H * N * L);
    double *a = (double *)malloc(sizeof(double) * (size_t)N * M);
    if (!p || !a) { free(p); free(a); return -1; }
    for (int b = 0; b < B; ++b) {
        const uint16_t *qb = q_text + (size_t)b * H * N * D;
        const uint16_t *kb = k + (size_t)b * H * L * D;
        if (mustdrop_oracle_attention(qb, kb, H, N, L, D, txt_start, causal, scale, p)) { free(p); free(a); return -1; }
        for (int i = 0; i < N; ++i)
            for (int j = 0; j < M; ++j) {
                double s = 0.0;
                for (int h = 0; h < H; ++h) s += p[((size_t)h * N + i) * L + vis_start + j];
                a[(size_t)i * M + j] = s / (double)H;
            }
        for (int j = 0; j < M; ++j) {
            double g = 0.0, mx = -INFINITY;
            for (int i = 0; i < N; ++i) {
                double v = a[(size_t)i * M + j];
                g += v;
                if (v > mx) mx = v;
            }
            g_out[(size_t)b * M + j] = (float)g;
            i_out[(size_t)b * M + j] = (float)mx;
        }
        if (a_out) memcpy(a_out + (size_t)b * N * M, a, sizeof(double) * (size_t)N * M);
    }
    free(p);
    free(a);
    return 0;
}

/*
 * The other reading of Eq. 10 over heads (the paper does not say how heads enter): the maximum
 * over text tokens is taken per head and the maxima are averaged,
 *   I[j] = (1/H) sum_h max_i p^h[i][vis_start + j],
 * instead of the maximum of the head mean.  G (Eq. 8) is linear in the heads and is unchanged.
 */
int mustdrop_oracle_score_per_head(const uint16_t *q_text, const uint16_t *k, int B, int H, int N, int L, int D,
                                   int vis_start, int M, int txt_start, int causal, double scale,
                                   float *g_out, float *i_out)
{
    if (!q_text || !k || !g_out || !i_out) return -1;
    if (B <= 0 || M <= 0 || vis_start < 0 || vis_start + M > txt_start || txt_start + N > L) return -1;
    double *p = (double *)malloc(sizeof(double) * (size_t)H * N * L);
    if (!p) return -1;
    for (int b = 0; b < B; ++b) {
        const uint16_t *qb = q_text + (size_t)b * H * N * D;
        const uint16_t *kb = k + (size_t)b * H * L * D;
        if (mustdrop_oracle_attention(qb, kb, H, N, L, D, txt_start, causal, scale, p)) { free(p); return -1; }
        for (int j = 0; j < M; ++j) {
            double g = 0.0, isum = 0.0;
            for (int h = 0; h < H; ++h) {
                double mx = -INFINITY;
                for (int i = 0; i < N; ++i) {
                    double v = p[((size_t)h * N + i) * L + vis_start + j];
                    g += v;
                    if (v > mx) mx = v;
                }
                isum += mx;
            }
            g_out[(size_t)b * M + j] = (float)(g / (double)H);
            i_out[(size_t)b * M + j] = (float)(isum / (double)H);
        }
    }
    free(p);
    return 0;
}

/* ---- selection ------------------------------------------------------------------------- */

enum { MODE_BUDGET = 0, MODE_THRESHOLD = 1 };
enum { CRIT_DUAL = 0, CRIT_GLOBAL_ONLY = 1, CRIT_INDIVIDUAL_ONLY = 2 };

typedef struct { float s; int32_t j; } scored_t;

/* order: larger score first, then smaller index */
static int by_score_desc_index_asc(const void *pa, const void *pb)
{
    const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
    return (a->j > b->j) - (a->j < b->j);
}

/*
 * Dual criteria, key set and selection for a batch.
 *   T    = fp32( sum_j (double) G[j] )            right-hand sum of Eq. 9
 *   gt   = gamma * T                              (fp32 multiply)
 *   D    = { j : G[j] <= gt }                     Eq. 9
 *   j is dropped iff j in D and I[j] < alpha (Eq. 10) and j not in O (Sec. 3.3, the key
 *   set is always retained).                      -> THRESHOLD mode, as printed.
 *   With one common factor t on both thresholds the rule reads "keep iff s[j] >= t" with
 *   s[j] = max(G[j]/gt, I[j]/alpha) (strictness at equality aside); BUDGET mode keeps O and
 *   then the tokens with the largest s (lower index first among equals) until exactly
 *   `budget` tokens are kept.  GLOBAL_ONLY / INDIVIDUAL_ONLY use one criterion (Table 4).
 *   gamma == 0 -> 1/M, alpha == 0 -> 2/L (fp32 divisions); seq_len is only used for that default.
 * key_idx int32 [B][key_max] vision-relative; entries outside [0,M) and repeats are ignored.
 * kept_idx int32 [B][cap], cap = budget (BUDGET) or M (THRESHOLD), ascending; kept_cnt [B].
 * s_out nullable fp32 [B][M]; t_out nullable fp32 [B].
 */
int mustdrop_oracle_select(const float *G, const float *I, int B, int M, int seq_len,
                           const int32_t *key_idx, const int32_t *key_cnt, int key_max,
                           int mode, int criteria, int budget, float gamma, float alpha,
                           int32_t *kept_idx, int32_t *kept_cnt, float *s_out, float *t_out)
{
    if (!G || !I || !kept_idx || !kept_cnt || B <= 0 || M <= 0) return -1;
    if (mode == MODE_BUDGET && (budget < 0 || budget > M)) return -1;
    if (gamma == 0.0f) gamma = 1.0f / (float)M;
    if (alpha == 0.0f) alpha = 2.0f / (float)seq_len;
    const int cap = (mode == MODE_BUDGET) ? budget : M;
    unsigned char *is_key = (unsigned char *)malloc((size_t)M);
    unsigned char *keep = (unsigned char *)malloc((size_t)M);
    scored_t *cand = (scored_t *)malloc(sizeof(scored_t) * (size_t)M);
    float *s = (float *)malloc(sizeof(float) * (size_t)M);
    if (!is_key || !keep || !cand || !s) { free(is_key); free(keep); free(cand); free(s); return -1; }
    for (int b = 0; b < B; ++b) {
        const float *g = G + (size_t)b * M, *in = I + (size_t)b * M;
        double tsum = 0.0;
        for (int j = 0; j < M; ++j) tsum += (double)g[j];
        const float T = (float)tsum;
        volatile float gt_v = gamma * T; /* volatile: one rounded fp32 product, never fused */
        const float gt = gt_v;
        memset(is_key, 0, (size_t)M);
        int n_key = 0;
        if (key_idx && key_cnt && key_max > 0) {
            int c = key_cnt[b] < key_max ? key_cnt[b] : key_max;
            for (int t = 0; t < c; ++t) {
                int32_t j = key_idx[(size_t)b * key_max + t];
                if (j >= 0 && j < M && !is_key[j]) { is_key[j] = 1; ++n_key; }
            }
        }
        for (int j = 0; j < M; ++j) {
            volatile float gj = g[j] / gt;
            volatile float rj = in[j] / alpha;
            float v;
            if (criteria == CRIT_GLOBAL_ONLY) v = gj;
            else if (criteria == CRIT_INDIVIDUAL_ONLY) v = rj;
            else v = (gj > rj) ? gj : rj;
            s[j] = v;
        }
        if (mode == MODE_THRESHOLD) {
            for (int j = 0; j < M; ++j) {
                int in_d = (g[j] <= gt);          /* Eq. 9 */
                int small = (in[j] < alpha);      /* Eq. 10 */
                int drop;
                if (criteria == CRIT_GLOBAL_ONLY) drop = in_d;
                else if (criteria == CRIT_INDIVIDUAL_ONLY) drop = small;
                else drop = in_d && small;
                keep[j] = (unsigned char)(is_key[j] || !drop);
            }
        } else {
            int n_cand = 0;
            for (int j = 0; j < M; ++j) {
                keep[j] = is_key[j];
                if (!is_key[j]) { cand[n_cand].s = s[j]; cand[n_cand].j = j; ++n_cand; }
            }
            qsort(cand, (size_t)n_cand, sizeof(scored_t), by_score_desc_index_asc);
            int want = budget - n_key;
            if (want > n_cand) want = n_cand;
            for (int t = 0; t < want; ++t) keep[cand[t].j] = 1;
        }
        int cnt = 0;
        for (int j = 0; j < M; ++j)
            if (keep[j]) { if (cnt < cap) kept_idx[(size_t)b * cap + cnt] = j; ++cnt; }
        kept_cnt[b] = cnt;
        if (s_out) memcpy(s_out + (size_t)b * M, s, sizeof(float) * (size_t)M);
        if (t_out) t_out[b] = T;
    }
    free(is_key); free(keep); free(cand); free(s);
    return 0;
}

/*
 * Gather-compaction (the pruned tokens leave the hidden sequence and the KV cache; Table 3
 * counts "vision tokens in the KV cache").  Byte copies of 2-byte elements:
 *   hidden_out[b][r][:]   = hidden[b][vis_start + kept[b][r]][:]
 *   k_out[b][h][r][:]     = k[b][h][vis_start + kept[b][r]][:]     (v likewise)
 * hidden [B][L][hid], k,v [B][H][L][D]; outputs [B][cap][hid], [B][H][cap][D]; rows
 * r >= kept_cnt[b] are left untouched.
 */
int mustdrop_oracle_compact(const int32_t *kept_idx, const int32_t *kept_cnt, int B, int cap,
                            int H, int L, int D, int hid, int vis_start,
                            const uint16_t *hidden, const uint16_t *k, const uint16_t *v,
                            uint16_t *hidden_out, uint16_t *k_out, uint16_t *v_out)
{
    if (!kept_idx || !kept_cnt) return -1;
    for (int b = 0; b < B; ++b) {
        int cnt = kept_cnt[b] < cap ? kept_cnt[b] : cap;
        for (int r = 0; r < cnt; ++r) {
            int row = vis_start + kept_idx[(size_t)b * cap + r];
            if (row < 0 || row >= L) return -1;
            if (hidden && hidden_out)
                memcpy(hidden_out + ((size_t)b * cap + r) * hid, hidden + ((size_t)b * L + row) * hid,
                       sizeof(uint16_t) * (size_t)hid);
            for (int h = 0; h < H; ++h) {
                size_t src = (((size_t)b * H + h) * L + row) * D;
                size_t dst = (((size_t)b * H + h) * cap + r) * D;
                if (k && k_out) memcpy(k_out + dst, k + src, sizeof(uint16_t) * (size_t)D);
                if (v && v_out) memcpy(v_out + dst, v + src, sizeof(uint16_t) * (size_t)D);
            }
        }
    }
    return 0;
}
