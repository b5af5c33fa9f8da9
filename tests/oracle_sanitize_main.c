/* Harness for tests/test_oracle_sanitizers.py: runs the C oracle on exactly-sized heap buffers of
 * several small ragged shapes (every edge the loops have: one token, one head, keys after the text
 * span, full and causal masks, keep-all, a key set with repeated and out-of-range entries), so
 * that a build with -fsanitize=address,undefined reports any read or write outside a buffer and
 * any undefined arithmetic.  Prints a checksum; exit status 0 when every call was accepted. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

int mustdrop_oracle_score(const uint16_t *, const uint16_t *, int, int, int, int, int, int, int, int, int, double,
                          float *, float *, double *);
int mustdrop_oracle_score_per_head(const uint16_t *, const uint16_t *, int, int, int, int, int, int, int, int, int,
                                   double, float *, float *);
int mustdrop_oracle_select(const float *, const float *, int, int, int, const int32_t *, const int32_t *, int, int,
                           int, int, float, float, int32_t *, int32_t *, float *, float *);
int mustdrop_oracle_compact(const int32_t *, const int32_t *, int, int, int, int, int, int, int, const uint16_t *,
                            const uint16_t *, const uint16_t *, uint16_t *, uint16_t *, uint16_t *);

static uint32_t rng = 12345u;
static uint16_t rand_bf16(void) {   /* a bf16 in about [-2, 2): sign, exponent 124..127, random mantissa */
    rng = rng * 1664525u + 1013904223u;
    const uint32_t r = rng >> 8;
    return (uint16_t)(((r & 1u) << 15) | ((124u + ((r >> 1) & 3u)) << 7) | ((r >> 3) & 0x7Fu));
}

static int run(int B, int H, int N, int M, int vis_start, int gap, int tail, int D, int hid, int causal, int key_max,
               int budget, int mode, double *sum) {
    const int txt_start = vis_start + M + gap, L = txt_start + N + tail;
    const int cap = mode == 0 ? budget : M;
    uint16_t *q = malloc(sizeof(uint16_t) * (size_t)B * H * N * D), *k = malloc(sizeof(uint16_t) * (size_t)B * H * L * D);
    uint16_t *v = malloc(sizeof(uint16_t) * (size_t)B * H * L * D), *hd = malloc(sizeof(uint16_t) * (size_t)B * L * hid);
    float *G = malloc(sizeof(float) * (size_t)B * M), *I = malloc(sizeof(float) * (size_t)B * M);
    float *G2 = malloc(sizeof(float) * (size_t)B * M), *I2 = malloc(sizeof(float) * (size_t)B * M);
    float *s = malloc(sizeof(float) * (size_t)B * M), *T = malloc(sizeof(float) * (size_t)B);
    double *a = malloc(sizeof(double) * (size_t)B * N * M);
    int32_t *key_idx = malloc(sizeof(int32_t) * (size_t)B * (key_max ? key_max : 1)), *key_cnt = malloc(sizeof(int32_t) * (size_t)B);
    int32_t *kept = malloc(sizeof(int32_t) * (size_t)B * (cap ? cap : 1)), *cnt = malloc(sizeof(int32_t) * (size_t)B);
    uint16_t *ho = malloc(sizeof(uint16_t) * (size_t)B * (cap ? cap : 1) * hid);
    uint16_t *ko = malloc(sizeof(uint16_t) * (size_t)B * H * (cap ? cap : 1) * D), *vo = malloc(sizeof(uint16_t) * (size_t)B * H * (cap ? cap : 1) * D);
    for (size_t x = 0; x < (size_t)B * H * N * D; ++x) q[x] = rand_bf16();
    for (size_t x = 0; x < (size_t)B * H * L * D; ++x) { k[x] = rand_bf16(); v[x] = rand_bf16(); }
    for (size_t x = 0; x < (size_t)B * L * hid; ++x) hd[x] = rand_bf16();
    for (int b = 0; b < B; ++b) {
        key_cnt[b] = key_max;
        for (int x = 0; x < key_max; ++x)   /* in range, repeated, and (every fourth) out of range */
            key_idx[b * key_max + x] = (x % 4 == 3) ? M + x : (x * 7 + b) % M;
    }
    int rc = 0;
    rc |= mustdrop_oracle_score(q, k, B, H, N, L, D, vis_start, M, txt_start, causal, 0.0, G, I, a);
    rc |= mustdrop_oracle_score_per_head(q, k, B, H, N, L, D, vis_start, M, txt_start, causal, 0.0, G2, I2);
    rc |= mustdrop_oracle_select(G, I, B, M, L, key_max ? key_idx : NULL, key_max ? key_cnt : NULL, key_max, mode, 0, budget,
                                 0.0f, 0.0f, kept, cnt, s, T);
    rc |= mustdrop_oracle_compact(kept, cnt, B, cap, H, L, D, hid, vis_start, hd, k, v, ho, ko, vo);
    for (int b = 0; b < B; ++b) {
        *sum += T[b] + cnt[b];
        for (int j = 0; j < M; ++j) *sum += G[b * M + j] + I2[b * M + j];
    }
    free(q); free(k); free(v); free(hd); free(G); free(I); free(G2); free(I2); free(s); free(T); free(a);
    free(key_idx); free(key_cnt); free(kept); free(cnt); free(ho); free(ko); free(vo);
    return rc;
}

int main(void) {
    double sum = 0.0;
    int rc = 0;
    /*        B  H  N   M  vs gap tail  D  hid causal keys budget mode */
    rc |= run(1, 1, 1,  1, 0, 0, 0,  8,  8, 1, 0,  1, 0, &sum);
    rc |= run(2, 3, 5, 17, 2, 0, 0, 16, 24, 1, 4,  6, 0, &sum);
    rc |= run(2, 2, 4, 23, 0, 3, 5, 16, 16, 0, 8, 23, 0, &sum);   /* keys behind the text span; keep all */
    rc |= run(3, 1, 7, 40, 1, 0, 2,  8, 40, 1, 5,  0, 1, &sum);   /* threshold mode: capacity M */
    rc |= run(1, 4, 9, 64, 0, 0, 0, 32,  8, 1, 0, 64, 0, &sum);
    printf("checksum %.9g\n", sum);
    return rc ? 1 : 0;
}
