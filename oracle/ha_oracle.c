/*
 * CPU oracle for the HashAttention decode path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain scalar C, written from the paper's definitions; it shares no code, header,
 * table or helper with the CUDA library and is never called by it.  Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may load this file.
 *
 * What each function follows:
 *   ora_encode       Eq. 2 (phi(x) = relu(sign(F(x))), bits packed into an integer) with
 *                    F the 128x128-128x128-128x32 feed-forward net of Section 5.2
 *                    ("Efficiency"); phi_kv acts on the key only (Section 4.1, last
 *                    paragraph).  The paper gives only the shapes of F; the arithmetic
 *                    below (fp32 fused multiply-add chain, ascending input index, started
 *                    from the bias, ReLU between layers, bit o set iff output o > 0) is
 *                    this build's stated reading.
 *   ora_score        Eq. 1 and the bitcount(xor) identity under "Implementation"
 *                    (Section 4.1), reported as 32 - Hamming distance; for grouped-query
 *                    attention the group score is the maximum over the query heads that
 *                    share the KV head (reduces to Eq. 1 when the group has one head).
 *   ora_score_sum    the other way to reduce Eq. 1 over a group (the stand-alone entry ha_score_topk_sum,
 *                    not of the layer-step): the per-head scores added up, 0 .. 32 G; the score
 *                    of the G query signatures concatenated against the key signature repeated.
 *   ora_score_wide   the same score for a signature of b = 64 .. 512 bits kept as b/64 packed
 *                    64-bit integers (the setting of the SCORE-latency table, "Latency of
 *                    SCORE computation"): b - Hamming distance, one query signature against n
 *                    key signatures, counted bit by bit.
 *   ora_encode_wide  Eq. 2 at b = 64 .. 512 bits (the signature widths of the bit-width study and of the
 *                    SCORE-latency table): the same network with a last layer of 128 x b, the b sign bits packed
 *                    into b/64 64-bit integers, bit j of the signature = bit j % 64 of word j / 64 (the order that
 *                    ora_score_wide reads).  Same arithmetic as ora_encode, output by output.
 *   ora_inner_products  the comparator column of that table: the inner product of one query
 *                    with each of n keys of 128 16-bit floats (bf16 here), in float64.
 *   ora_topk         "the standard top-k on these scores" (Section 4): sort by
 *                    (score descending, token index ascending), keep min(k, n).
 *   ora_topk_windows the selection used for every method in the experiments (Section 5,
 *                    paragraph on baselines): the first n_sink and the most recent n_local
 *                    tokens are always in context, the token budget k counts the heavy
 *                    tokens retrieved in addition, by the same order, among the others.
 *   ora_gather_attn  the GATHER-ATT formula of Section 4 (softmax restricted to the index
 *                    set), with the 1/sqrt(d) factor of the SDPA definition (Section 3.1)
 *                    passed in as sm_scale.
 *   ora_dense        SDPA for one query (Section 3.1) = GATHER-ATT over all n tokens.
 *   ora_decode_step  the composition ENCODE -> SCORE -> TOPK -> GATHER-ATT for a batch
 *                    (Section 4 recipe + Section 4.1 "Implementation").
 *
 * Pins (tests/test_oracle_*.py): closed forms (identity / zero weights, single token,
 * zero query), hand-derived fixtures in tests/golden/, an O(n^2) rank definition of
 * top-k, bit-level brute force for the score, the +-1 inner-product identity and the 32-bit
 * score for the wide score, concatenated signatures and the +-1 identity for the summed score, float64 numpy for the mapping net and the inner products, and
 * torch's scaled_dot_product_attention in float64 for the attention.
 * The fp32 accumulation ORDER inside ora_encode is a definition of this build, not of
 * the paper: it is pinned only up to the float64 margin test ("parity unpinned" for
 * the order itself).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define HA_D 128      /* head dimension = input width of the mapping net */
#define HA_HID 128    /* hidden width */
#define HA_BITS 32    /* signature width b */

/* ---------------------------------------------------------------- bf16 helpers */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* double -> bf16, one round-to-nearest-even step (no intermediate float rounding). */
static uint16_t f64_to_bf16(double x) {
    if (isnan(x)) return 0x7FC0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80);
    int e;
    (void)frexp(a, &e);               /* a = m * 2^e with m in [0.5, 1) */
    int exp_unb = e - 1;              /* a = (2m) * 2^(e-1), 2m in [1, 2) */
    if (exp_unb < -126) exp_unb = -126;          /* subnormal range: fixed quantum 2^-133 */
    double quantum = ldexp(1.0, exp_unb - 7);    /* bf16 keeps 7 fraction bits */
    double q = nearbyint(a / quantum);           /* ties-to-even in the default rounding mode */
    double r = q * quantum;
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80);
    float f = (float)r;                          /* exact: r is representable in bf16 */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* ---------------------------------------------------------------- ENCODE (Eq. 2) */

/* One mapping phi_int applied to n_vec vectors.
 *   x        bf16 [n_vec][128], row r starts at x + r * x_stride (elements)
 *   w1, w2   bf16 [128][128], w3 bf16 [128][32]; y = x W + b, W indexed [in][out]
 *   b1..b3   fp32 [out] or NULL (= zeros)
 *   codes    out, uint32 [n_vec]; bit o = 1 iff z3[o] > 0
 *   z3_out   optional fp32 [n_vec][32]: the pre-sign outputs, for margin diagnostics */
void ora_encode(const uint16_t *x, int64_t n_vec, int64_t x_stride,
                const uint16_t *w1, const uint16_t *w2, const uint16_t *w3,
                const float *b1, const float *b2, const float *b3,
                uint32_t *codes, float *z3_out) {
    float *W1 = (float *)malloc(sizeof(float) * HA_D * HA_HID);
    float *W2 = (float *)malloc(sizeof(float) * HA_HID * HA_HID);
    float *W3 = (float *)malloc(sizeof(float) * HA_HID * HA_BITS);
    for (int i = 0; i < HA_D * HA_HID; ++i) W1[i] = bf16_to_f32(w1[i]);
    for (int i = 0; i < HA_HID * HA_HID; ++i) W2[i] = bf16_to_f32(w2[i]);
    for (int i = 0; i < HA_HID * HA_BITS; ++i) W3[i] = bf16_to_f32(w3[i]);

    for (int64_t r = 0; r < n_vec; ++r) {
        float h0[HA_D], h1[HA_HID], h2[HA_HID], z[HA_HID];
        const uint16_t *xr = x + r * x_stride;
        for (int k = 0; k < HA_D; ++k) h0[k] = bf16_to_f32(xr[k]);

        /* layer 1: z = b1 + sum_k h0[k] W1[k][o], ascending k, one fmaf per term */
        for (int o = 0; o < HA_HID; ++o) z[o] = b1 ? b1[o] : 0.0f;
        for (int k = 0; k < HA_D; ++k)
            for (int o = 0; o < HA_HID; ++o) z[o] = fmaf(h0[k], W1[k * HA_HID + o], z[o]);
        for (int o = 0; o < HA_HID; ++o) h1[o] = (z[o] > 0.0f) ? z[o] : 0.0f;

        /* layer 2 */
        for (int o = 0; o < HA_HID; ++o) z[o] = b2 ? b2[o] : 0.0f;
        for (int k = 0; k < HA_HID; ++k)
            for (int o = 0; o < HA_HID; ++o) z[o] = fmaf(h1[k], W2[k * HA_HID + o], z[o]);
        for (int o = 0; o < HA_HID; ++o) h2[o] = (z[o] > 0.0f) ? z[o] : 0.0f;

        /* layer 3: 32 outputs, no activation; sign -> bit */
        for (int o = 0; o < HA_BITS; ++o) z[o] = b3 ? b3[o] : 0.0f;
        for (int k = 0; k < HA_HID; ++k)
            for (int o = 0; o < HA_BITS; ++o) z[o] = fmaf(h2[k], W3[k * HA_BITS + o], z[o]);

        uint32_t code = 0;
        for (int o = 0; o < HA_BITS; ++o)
            if (z[o] > 0.0f) code |= (1u << o);
        codes[r] = code;
        if (z3_out)
            for (int o = 0; o < HA_BITS; ++o) z3_out[r * HA_BITS + o] = z[o];
    }
    free(W1); free(W2); free(W3);
}

/* Eq. 2 with a last layer of n_bits outputs (n_bits a multiple of 64): w3 bf16 [128][n_bits], b3 fp32 [n_bits] or
 * NULL; codes out, uint64 [n_vec][n_bits / 64]; z3_out optional fp32 [n_vec][n_bits].  Layers 1 and 2 and the
 * arithmetic of every output (fmaf chain, ascending input index, from the bias) are those of ora_encode. */
void ora_encode_wide(const uint16_t *x, int64_t n_vec, int64_t x_stride,
                     const uint16_t *w1, const uint16_t *w2, const uint16_t *w3,
                     const float *b1, const float *b2, const float *b3, int32_t n_bits,
                     uint64_t *codes, float *z3_out) {
    const int n_words = n_bits / 64;
    float *W1 = (float *)malloc(sizeof(float) * HA_D * HA_HID);
    float *W2 = (float *)malloc(sizeof(float) * HA_HID * HA_HID);
    float *W3 = (float *)malloc(sizeof(float) * HA_HID * (size_t)n_bits);
    float *z3 = (float *)malloc(sizeof(float) * (size_t)n_bits);
    for (int i = 0; i < HA_D * HA_HID; ++i) W1[i] = bf16_to_f32(w1[i]);
    for (int i = 0; i < HA_HID * HA_HID; ++i) W2[i] = bf16_to_f32(w2[i]);
    for (int i = 0; i < HA_HID * n_bits; ++i) W3[i] = bf16_to_f32(w3[i]);
    for (int64_t r = 0; r < n_vec; ++r) {
        float h0[HA_D], h1[HA_HID], h2[HA_HID], z[HA_HID];
        const uint16_t *xr = x + r * x_stride;
        for (int k = 0; k < HA_D; ++k) h0[k] = bf16_to_f32(xr[k]);
        for (int o = 0; o < HA_HID; ++o) z[o] = b1 ? b1[o] : 0.0f;
        for (int k = 0; k < HA_D; ++k)
            for (int o = 0; o < HA_HID; ++o) z[o] = fmaf(h0[k], W1[k * HA_HID + o], z[o]);
        for (int o = 0; o < HA_HID; ++o) h1[o] = (z[o] > 0.0f) ? z[o] : 0.0f;
        for (int o = 0; o < HA_HID; ++o) z[o] = b2 ? b2[o] : 0.0f;
        for (int k = 0; k < HA_HID; ++k)
            for (int o = 0; o < HA_HID; ++o) z[o] = fmaf(h1[k], W2[k * HA_HID + o], z[o]);
        for (int o = 0; o < HA_HID; ++o) h2[o] = (z[o] > 0.0f) ? z[o] : 0.0f;
        for (int o = 0; o < n_bits; ++o) z3[o] = b3 ? b3[o] : 0.0f;
        for (int k = 0; k < HA_HID; ++k)
            for (int o = 0; o < n_bits; ++o) z3[o] = fmaf(h2[k], W3[(size_t)k * n_bits + o], z3[o]);
        for (int w = 0; w < n_words; ++w) codes[r * n_words + w] = 0;
        for (int o = 0; o < n_bits; ++o)
            if (z3[o] > 0.0f) codes[r * n_words + o / 64] |= ((uint64_t)1 << (o % 64));
        if (z3_out)
            for (int o = 0; o < n_bits; ++o) z3_out[r * n_bits + o] = z3[o];
    }
    free(W1); free(W2); free(W3); free(z3);
}

/* ---------------------------------------------------------------- SCORE (Eq. 1) */

static int hamming32(uint32_t a, uint32_t b) {
    uint32_t x = a ^ b;
    int h = 0;
    for (int bit = 0; bit < HA_BITS; ++bit) h += (int)((x >> bit) & 1u);
    return h;
}

/* scores[i] = max over the group's query codes of (32 - Hamming(kcodes[i], qcodes[j])). */
void ora_score(const uint32_t *qcodes, int32_t group, const uint32_t *kcodes, int64_t n,
               int32_t *scores) {
    for (int64_t i = 0; i < n; ++i) {
        int best = -1;
        for (int j = 0; j < group; ++j) {
            int s = HA_BITS - hamming32(kcodes[i], qcodes[j]);
            if (s > best) best = s;
        }
        scores[i] = best;
    }
}

/* Alternative reduction over a GQA group: scores[i] = sum over the group's query codes of
 * (32 - Hamming(kcodes[i], qcodes[j])), i.e. Eq. 1 per query head added up; range 0 .. 32 * group.
 * The paper defines the score for one query head only; with group = 1 this is Eq. 1 itself. */
void ora_score_sum(const uint32_t *qcodes, int32_t group, const uint32_t *kcodes, int64_t n,
                   int32_t *scores) {
    for (int64_t i = 0; i < n; ++i) {
        int total = 0;
        for (int j = 0; j < group; ++j) total += HA_BITS - hamming32(kcodes[i], qcodes[j]);
        scores[i] = total;
    }
}

/* scores[i] = n_bits - Hamming(k_i, q) for signatures of n_words packed 64-bit integers
 * (n_bits = 64 n_words; bit j of the signature is bit j % 64 of word j / 64).  Counted one
 * bit at a time: a score is the number of positions in which the two signatures agree. */
void ora_score_wide(const uint64_t *qcode, const uint64_t *kcodes, int64_t n, int32_t n_words, int32_t *scores) {
    for (int64_t i = 0; i < n; ++i) {
        int agree = 0;
        for (int w = 0; w < n_words; ++w)
            for (int bit = 0; bit < 64; ++bit)
                agree += (int)(((kcodes[i * n_words + w] >> bit) & 1u) == ((qcode[w] >> bit) & 1u));
        scores[i] = agree;
    }
}

/* dots[i] = <q, K_i> over 128 bf16 components, accumulated in float64 (the comparator of the table). */
void ora_inner_products(const uint16_t *q, const uint16_t *K, int64_t n, int64_t row_stride, double *dots) {
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int d = 0; d < HA_D; ++d) acc += (double)bf16_to_f32(q[d]) * (double)bf16_to_f32(K[i * row_stride + d]);
        dots[i] = acc;
    }
}

/* ---------------------------------------------------------------- TOPK */

/* stable merge sort of token indices by score descending: equal scores keep index order */
static void merge_sort_desc(int32_t *a, int32_t *tmp, int64_t lo, int64_t hi, const int32_t *s) {
    if (hi - lo < 2) return;
    int64_t mid = lo + (hi - lo) / 2;
    merge_sort_desc(a, tmp, lo, mid, s);
    merge_sort_desc(a, tmp, mid, hi, s);
    int64_t i = lo, j = mid, o = lo;
    while (i < mid && j < hi) {
        if (s[a[j]] > s[a[i]]) tmp[o++] = a[j++];   /* strictly better only: ties take the left run */
        else tmp[o++] = a[i++];
    }
    while (i < mid) tmp[o++] = a[i++];
    while (j < hi) tmp[o++] = a[j++];
    memcpy(a + lo, tmp + lo, sizeof(int32_t) * (size_t)(hi - lo));
}

static int cmp_i32(const void *p, const void *q) {
    int32_t a = *(const int32_t *)p, b = *(const int32_t *)q;
    return (a > b) - (a < b);
}

/* Keep the first min(k, n) tokens of the order (score desc, index asc); emit ascending.
 * Returns the number of indices written. */
int64_t ora_topk(const int32_t *scores, int64_t n, int64_t k, int32_t *idx_out) {
    if (n <= 0 || k <= 0) return 0;
    int64_t keep = k < n ? k : n;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    for (int64_t i = 0; i < n; ++i) order[i] = (int32_t)i;
    merge_sort_desc(order, tmp, 0, n, scores);
    memcpy(idx_out, order, sizeof(int32_t) * (size_t)keep);
    qsort(idx_out, (size_t)keep, sizeof(int32_t), cmp_i32);
    free(order); free(tmp);
    return keep;
}

/* Always keep tokens [0, n_sink) and [n - n_local, n); among the other tokens keep the first
 * min(k, how many there are) of the order (score desc, index asc); emit everything ascending.
 * Returns the number of indices written (at most n).  n_sink = n_local = 0 is ora_topk. */
int64_t ora_topk_windows(const int32_t *scores, int64_t n, int64_t k, int64_t n_sink, int64_t n_local,
                         int32_t *idx_out) {
    if (n <= 0) return 0;
    if (n_sink < 0) n_sink = 0;
    if (n_local < 0) n_local = 0;
    int64_t written = 0, n_rest = 0;
    int32_t *rest = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    int32_t *tmp = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
    for (int64_t i = 0; i < n; ++i) {
        if (i < n_sink || i >= n - n_local) idx_out[written++] = (int32_t)i;   /* always in context */
        else rest[n_rest++] = (int32_t)i;
    }
    int64_t keep = k < 0 ? 0 : (k < n_rest ? k : n_rest);
    merge_sort_desc(rest, tmp, 0, n_rest, scores);
    for (int64_t i = 0; i < keep; ++i) idx_out[written++] = rest[i];
    qsort(idx_out, (size_t)written, sizeof(int32_t), cmp_i32);
    free(rest); free(tmp);
    return written;
}

/* ---------------------------------------------------------------- GATHER-ATT / SDPA */

/* One query head over an index list.
 *   q        bf16 [128]
 *   K, V     bf16 rows; token t starts at K + t * row_stride (elements)
 *   idx      token indices (NULL = 0..count-1); entries < 0 or >= n_valid are skipped
 *   out      bf16 [128], rounded once from double; lse = m + log(sum exp(l - m))
 * Empty list: out = 0, lse = -inf. */
void ora_gather_attn(const uint16_t *q, const uint16_t *K, const uint16_t *V, int64_t row_stride,
                     const int32_t *idx, int64_t count, int64_t n_valid, double sm_scale,
                     uint16_t *out, double *lse, double *out_f64) {
    double *logit = (double *)malloc(sizeof(double) * (size_t)(count > 0 ? count : 1));
    int64_t *tok = (int64_t *)malloc(sizeof(int64_t) * (size_t)(count > 0 ? count : 1));
    int64_t m_cnt = 0;
    double m = -INFINITY;
    for (int64_t c = 0; c < count; ++c) {
        int64_t t = idx ? (int64_t)idx[c] : c;
        if (t < 0 || t >= n_valid) continue;
        const uint16_t *kr = K + t * row_stride;
        double dot = 0.0;
        for (int d = 0; d < HA_D; ++d) dot += (double)bf16_to_f32(q[d]) * (double)bf16_to_f32(kr[d]);
        logit[m_cnt] = sm_scale * dot;
        tok[m_cnt] = t;
        if (logit[m_cnt] > m) m = logit[m_cnt];
        ++m_cnt;
    }
    double acc[HA_D];
    for (int d = 0; d < HA_D; ++d) acc[d] = 0.0;
    double denom = 0.0;
    for (int64_t c = 0; c < m_cnt; ++c) {
        double p = exp(logit[c] - m);
        denom += p;
        const uint16_t *vr = V + tok[c] * row_stride;
        for (int d = 0; d < HA_D; ++d) acc[d] += p * (double)bf16_to_f32(vr[d]);
    }
    for (int d = 0; d < HA_D; ++d) {
        double o = (m_cnt > 0) ? acc[d] / denom : 0.0;
        if (out) out[d] = f64_to_bf16(o);
        if (out_f64) out_f64[d] = o;
    }
    if (lse) *lse = (m_cnt > 0) ? m + log(denom) : -INFINITY;
    free(logit); free(tok);
}

void ora_dense(const uint16_t *q, const uint16_t *K, const uint16_t *V, int64_t row_stride,
               int64_t n, double sm_scale, uint16_t *out, double *lse, double *out_f64) {
    ora_gather_attn(q, K, V, row_stride, NULL, n, n, sm_scale, out, lse, out_f64);
}

uint16_t ora_f64_to_bf16(double x) { return f64_to_bf16(x); }

/* ---------------------------------------------------------------- whole decode step */

/* One layer-step for a batch (Section 4 recipe; Section 4.1 "Implementation"):
 *   for every (sequence b, KV head g): append the code of the new key at slot n_b-1,
 *   encode the group's queries, score all n_b cached codes, top-k, GATHER-ATT.
 * Layouts (all contiguous, host memory):
 *   q      bf16 [B][Hq][128]          k_new  bf16 [B][Hkv][128]
 *   K, V   bf16 [B][Hkv][n_cap][128]  kcodes u32 [B][Hkv][n_cap] (slot n_b-1 is written)
 *   wq*, wk*: per-KV-head mappings, w1/w2 [Hkv][128][128], w3 [Hkv][128][32], biases [Hkv][out] or NULL
 *   seq_lens [B], k_per_seq [B]
 *   qcodes out [B][Hq]; idx out [B][Hkv][k_max] (ascending, -1 padded); count out [B][Hkv]
 *   n_sink, n_local: tokens always kept in addition to the budget (0, 0 = plain top-k); k_max must
 *   hold the windows plus the budget
 *   out bf16 [B][Hq][128]; lse double [B][Hq]
 * One OpenMP loop over (b, g) when compiled with -fopenmp and n_threads > 1. */
void ora_decode_step(int32_t B, int32_t Hq, int32_t Hkv, int64_t n_cap, int64_t k_max,
                     const uint16_t *q, const uint16_t *k_new,
                     const uint16_t *K, const uint16_t *V, uint32_t *kcodes,
                     const uint16_t *wq1, const uint16_t *wq2, const uint16_t *wq3,
                     const float *bq1, const float *bq2, const float *bq3,
                     const uint16_t *wk1, const uint16_t *wk2, const uint16_t *wk3,
                     const float *bk1, const float *bk2, const float *bk3,
                     const int32_t *seq_lens, const int32_t *k_per_seq, double sm_scale,
                     uint32_t *qcodes, int32_t *idx, int32_t *count,
                     uint16_t *out, double *lse, int32_t n_threads, int32_t n_sink, int32_t n_local) {
    const int32_t G = Hq / Hkv;
    const int64_t units = (int64_t)B * Hkv;
    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads > 0 ? n_threads : 1)
#endif
    for (int64_t u = 0; u < units; ++u) {
        const int32_t b = (int32_t)(u / Hkv), g = (int32_t)(u % Hkv);
        const int64_t n = seq_lens[b];
        const int64_t k = k_per_seq[b];
        const uint16_t *Kh = K + ((int64_t)b * Hkv + g) * n_cap * HA_D;
        const uint16_t *Vh = V + ((int64_t)b * Hkv + g) * n_cap * HA_D;
        uint32_t *codes = kcodes + ((int64_t)b * Hkv + g) * n_cap;
        int32_t *idx_u = idx + ((int64_t)b * Hkv + g) * k_max;
        for (int64_t c = 0; c < k_max; ++c) idx_u[c] = -1;

        /* ENCODE: new key -> code cache slot n-1; the group's queries -> qcodes */
        if (k_new && n > 0)
            ora_encode(k_new + ((int64_t)b * Hkv + g) * HA_D, 1, HA_D,
                       wk1 + (int64_t)g * HA_D * HA_HID, wk2 + (int64_t)g * HA_HID * HA_HID,
                       wk3 + (int64_t)g * HA_HID * HA_BITS,
                       bk1 ? bk1 + g * HA_HID : NULL, bk2 ? bk2 + g * HA_HID : NULL,
                       bk3 ? bk3 + g * HA_BITS : NULL, codes + (n - 1), NULL);
        uint32_t *qc = qcodes + (int64_t)b * Hq + (int64_t)g * G;
        ora_encode(q + ((int64_t)b * Hq + (int64_t)g * G) * HA_D, G, HA_D,
                   wq1 + (int64_t)g * HA_D * HA_HID, wq2 + (int64_t)g * HA_HID * HA_HID,
                   wq3 + (int64_t)g * HA_HID * HA_BITS,
                   bq1 ? bq1 + g * HA_HID : NULL, bq2 ? bq2 + g * HA_HID : NULL,
                   bq3 ? bq3 + g * HA_BITS : NULL, qc, NULL);

        /* SCORE -> TOPK */
        int32_t *scores = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
        ora_score(qc, G, codes, n, scores);
        int64_t cnt = (n_sink > 0 || n_local > 0) ? ora_topk_windows(scores, n, k, n_sink, n_local, idx_u)
                                                  : ora_topk(scores, n, k, idx_u);
        count[u] = (int32_t)cnt;
        free(scores);

        /* GATHER-ATT for each query head of the group */
        for (int j = 0; j < G; ++j) {
            int64_t head = (int64_t)b * Hq + (int64_t)g * G + j;
            ora_gather_attn(q + head * HA_D, Kh, Vh, HA_D, idx_u, cnt, n, sm_scale,
                            out + head * HA_D, lse ? lse + head : NULL, NULL);
        }
    }
}

int32_t ora_max_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
